"""ctypes binding of libtlr.so: the same entry points as include/tlr.h, argument marshalling only.

Every step of the routing path runs inside the library's CUDA kernels.  torch is used
for device memory and streams.  There is no fallback: if the library is missing or a
call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_float, c_int32, c_uint32, c_void_p

import torch

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(PKG_DIR, "libtlr.so")

TLR_OK = 0
TLR_ERR_ARG, TLR_ERR_ALIGN, TLR_ERR_UNSUPPORTED, TLR_ERR_CUDA = 1, 2, 3, 4
TLR_ERR_NOMEM, TLR_ERR_TOO_MANY_ROWS, TLR_ERR_DEVICE_STATUS = 5, 6, 7
TLR_PATH_AUTO, TLR_PATH_SIMT, TLR_PATH_TC = 0, 1, 2
TLR_DEV_WAIT_TIMEOUT, TLR_DEV_NONFINITE = 1, 2
TLR_STATIC_MAX_ROWS = 1024
TLR_SCORE_CONF, TLR_SCORE_MLP = 0, 1


class TlrPlan(ctypes.Structure):
    _fields_ = [("path", c_int32), ("grid", c_int32), ("block", c_int32), ("row_units", c_int32),
                ("vocab_chunks", c_int32), ("smem_bytes", c_int32), ("launches", c_int32), ("reserved", c_int32)]


class TlrRouteOptions(ctypes.Structure):
    _fields_ = [("tau_per_row_dev", c_void_p), ("route_above", c_int32), ("seq_len", c_int32),
                ("first_routed_dev", c_void_p), ("score_source", c_int32), ("mlp_score_dev", c_void_p)]


class TlrError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (status %d)" % (where, status_string(code), code))


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libtlr.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libtlr.so not found at %s -- build it with `python -m paper_2504_07878_b200.build`"
                           % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    P = c_void_p
    lib.tlr_create.argtypes = [c_int32, c_int32, P, c_int32, POINTER(P)]
    lib.tlr_create_fp8.argtypes = [c_int32, c_int32, P, P, c_int32, POINTER(P)]
    lib.tlr_create_fp8.restype = c_int32
    lib.tlr_route.argtypes = [P, P, c_int32, c_float, P, P, P, P, P, P, P]
    lib.tlr_route_ex.argtypes = [P, P, c_int32, c_float, POINTER(TlrRouteOptions), P, P, P, P, P, P, P]
    lib.tlr_route_ex.restype = c_int32
    lib.tlr_debug_plan_tiles.argtypes = [c_int32, c_int32, c_int32, c_int32, P, c_int32, POINTER(c_int32), POINTER(TlrPlan)]
    lib.tlr_debug_plan_tiles.restype = c_int32
    lib.tlr_debug_inject.argtypes = [P, c_int32, c_uint32]
    lib.tlr_debug_inject.restype = c_int32
    lib.tlr_set_router_mlp.argtypes = [P, c_int32, P, P, P, c_float]
    lib.tlr_set_router_mlp.restype = c_int32
    lib.tlr_route_host.argtypes = [P, P, c_int32, c_float, P, P, P, P, P, P, P]
    lib.tlr_route_host_submit.argtypes = [P, P, c_int32, c_float, P]
    lib.tlr_route_host_submit.restype = c_int32
    lib.tlr_route_host_collect.argtypes = [P, P, P, P, P, P, P]
    lib.tlr_route_host_collect.restype = c_int32
    lib.tlr_shard_summary.argtypes = [P, P, c_int32, c_int32, P, P]
    lib.tlr_shard_summary.restype = c_int32
    lib.tlr_shard_finish.argtypes = [P, P, c_int32, c_int32, c_float, P, P, P, P, P, P, P]
    lib.tlr_shard_finish.restype = c_int32
    lib.tlr_shard_block_bytes.argtypes = [c_int32, c_int32]
    lib.tlr_shard_block_bytes.restype = ctypes.c_size_t
    lib.tlr_shard_attach.argtypes = [P, c_int32, c_int32, POINTER(P)]
    lib.tlr_shard_attach.restype = c_int32
    lib.tlr_shard_push.argtypes = [P, P, c_int32, c_int32, P]
    lib.tlr_shard_push.restype = c_int32
    lib.tlr_shard_finish_fused.argtypes = [P, c_int32, c_float, P, P, P, P, P, P, P]
    lib.tlr_shard_finish_fused.restype = c_int32
    lib.tlr_debug_shard_table.argtypes = [c_int32, c_int32, c_int32, POINTER(P), c_int32, POINTER(P), POINTER(P)]
    lib.tlr_debug_shard_table.restype = c_int32
    lib.tlr_rows_merge.argtypes = [P, P, P, c_int32, c_int32, P, P, P]
    lib.tlr_rows_merge.restype = c_int32
    lib.tlr_destroy.argtypes = [P]
    lib.tlr_status_string.argtypes = [c_int32]
    lib.tlr_status_string.restype = c_char_p
    lib.tlr_last_device_status.argtypes = [P, POINTER(c_uint32)]
    lib.tlr_set_path.argtypes = [P, c_int32]
    lib.tlr_plan_query.argtypes = [P, c_int32, POINTER(TlrPlan)]
    lib.tlr_set_kernel_timing.argtypes = [P, c_int32]
    lib.tlr_read_kernel_timing.argtypes = [P, POINTER(c_int32), POINTER(c_float)]
    lib.tlr_route_static.argtypes = [c_int32, c_int32, P, P, c_int32, c_float, P, P, P, P, P, P, P, P]
    lib.tlr_route_static.restype = c_int32
    for name in ("tlr_create", "tlr_route", "tlr_route_host", "tlr_destroy", "tlr_last_device_status",
                 "tlr_set_path", "tlr_plan_query", "tlr_set_kernel_timing", "tlr_read_kernel_timing"):
        getattr(lib, name).restype = c_int32
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().tlr_status_string(code).decode()


def _check(code: int, where: str):
    if code != TLR_OK:
        raise TlrError(code, where)


def _ptr(t) -> c_void_p:
    if t is None:
        return c_void_p(0)
    if isinstance(t, int):
        return c_void_p(t)
    return c_void_p(t.data_ptr())


def _stream_handle(stream) -> c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    if isinstance(stream, int):
        return c_void_p(stream)
    return c_void_p(stream.cuda_stream)


def tlr_create(d: int, V: int, W, max_n: int) -> c_void_p:
    """W: CUDA bf16 [V, d] contiguous tensor (or a raw device address).  It is borrowed, not copied."""
    ctx = c_void_p(0)
    _check(load_library().tlr_create(d, V, _ptr(W), max_n, byref(ctx)), "tlr_create")
    return ctx


def tlr_create_fp8(d: int, V: int, W_e4m3, wscale, max_n: int) -> c_void_p:
    """W_e4m3: CUDA uint8 (or float8_e4m3fn) [V, d] codes, wscale: CUDA float32 [V]; both borrowed.  Decode batches only."""
    ctx = c_void_p(0)
    _check(load_library().tlr_create_fp8(d, V, _ptr(W_e4m3), _ptr(wscale), max_n, byref(ctx)), "tlr_create_fp8")
    return ctx


def tlr_route(ctx, h, n: int, tau: float, token, conf, entropy, route_mask, routed_idx, routed_count, stream=None):
    """All tensor arguments are CUDA tensors (or raw device addresses).  Asynchronous on `stream`."""
    _check(load_library().tlr_route(ctx, _ptr(h), n, tau, _ptr(token), _ptr(conf), _ptr(entropy), _ptr(route_mask),
                                    _ptr(routed_idx), _ptr(routed_count), _stream_handle(stream)), "tlr_route")


def tlr_route_ex(ctx, h, n: int, tau: float, token, conf, entropy, route_mask, routed_idx, routed_count, stream=None,
                 tau_per_row=None, route_above: bool = False, seq_len: int = 0, first_routed=None,
                 score_source: int = 0, mlp_score=None):
    """tlr_route with per-row thresholds, the opposite polarity, the first routed position per sequence,
    and the learned router score (score_source=TLR_SCORE_MLP after tlr_set_router_mlp)."""
    opt = TlrRouteOptions(_ptr(tau_per_row), 1 if route_above else 0, int(seq_len), _ptr(first_routed),
                          int(score_source), _ptr(mlp_score))
    _check(load_library().tlr_route_ex(ctx, _ptr(h), n, tau, byref(opt), _ptr(token), _ptr(conf), _ptr(entropy),
                                       _ptr(route_mask), _ptr(routed_idx), _ptr(routed_count),
                                       _stream_handle(stream)), "tlr_route_ex")


def tlr_set_router_mlp(ctx, d_hidden: int, W1, b1, w2, b2: float):
    """Attach score(h) = sigmoid(w2 . relu(W1 h + b1) + b2); W1 bf16 [d_hidden, d], b1/w2 float [d_hidden] (CUDA)."""
    _check(load_library().tlr_set_router_mlp(ctx, d_hidden, _ptr(W1), _ptr(b1), _ptr(w2), b2), "tlr_set_router_mlp")


def tlr_route_host(ctx, h, n: int, tau: float, token, conf, entropy, route_mask, routed_idx, routed_count,
                   stream=None):
    """Same with HOST tensors (CPU, ideally pinned); copies in, routes, copies out, synchronises."""
    _check(load_library().tlr_route_host(ctx, _ptr(h), n, tau, _ptr(token), _ptr(conf), _ptr(entropy),
                                         _ptr(route_mask), _ptr(routed_idx), _ptr(routed_count),
                                         _stream_handle(stream)), "tlr_route_host")


def tlr_route_host_submit(ctx, h, n: int, tau: float, stream=None):
    """First half of tlr_route_host: enqueue copy-in, step and write-back; h (a CPU tensor, ideally pinned) must stay
    valid until the matching collect.  At most two submitted calls may be waiting."""
    _check(load_library().tlr_route_host_submit(ctx, _ptr(h), n, tau, _stream_handle(stream)), "tlr_route_host_submit")


def tlr_route_host_collect(ctx, token, conf, entropy, route_mask, routed_idx, routed_count):
    """Second half: wait for the oldest submitted call and copy its results into the given CPU tensors."""
    _check(load_library().tlr_route_host_collect(ctx, _ptr(token), _ptr(conf), _ptr(entropy), _ptr(route_mask),
                                                 _ptr(routed_idx), _ptr(routed_count)), "tlr_route_host_collect")


def tlr_shard_summary(ctx, h, n: int, v_offset: int, summary, stream=None):
    """Vocabulary-sharded step, part 1: one 16-byte summary per row over this GPU's rows of W (global indices)."""
    _check(load_library().tlr_shard_summary(ctx, _ptr(h), n, v_offset, _ptr(summary), _stream_handle(stream)),
           "tlr_shard_summary")


def tlr_shard_finish(ctx, summaries, shards: int, n: int, tau: float, token, conf, entropy, route_mask, routed_idx,
                     routed_count, stream=None):
    """Part 2: merge the gathered summaries [shards][n] and produce the six outputs of tlr_route."""
    _check(load_library().tlr_shard_finish(ctx, _ptr(summaries), shards, n, tau, _ptr(token), _ptr(conf),
                                           _ptr(entropy), _ptr(route_mask), _ptr(routed_idx), _ptr(routed_count),
                                           _stream_handle(stream)), "tlr_shard_finish")


def tlr_shard_block_bytes(max_n: int, shards: int) -> int:
    """Size of one GPU's exchange block for the fused vocabulary-sharded step."""
    return int(load_library().tlr_shard_block_bytes(max_n, shards))


def tlr_shard_attach(ctx, rank: int, shards: int, peer_blocks):
    """peer_blocks: `shards` device addresses (ints or tensors), entry g = GPU g's zeroed exchange block."""
    arr = (c_void_p * shards)(*[_ptr(b) for b in peer_blocks])
    _check(load_library().tlr_shard_attach(ctx, rank, shards, arr), "tlr_shard_attach")


def tlr_debug_shard_table(max_n: int, rank: int, shards: int, peer_blocks, parity: int):
    """Host-only: (slot addresses, flag addresses) of one rank on every peer, as tlr_shard_attach derives them."""
    blocks = (c_void_p * shards)(*[_ptr(b) for b in peer_blocks])
    slots, flags = (c_void_p * shards)(), (c_void_p * shards)()
    _check(load_library().tlr_debug_shard_table(max_n, rank, shards, blocks, parity, slots, flags),
           "tlr_debug_shard_table")
    return [int(x or 0) for x in slots], [int(x or 0) for x in flags]


def tlr_shard_push(ctx, h, n: int, v_offset: int, stream=None):
    """Projection on this rank's shard, then the summaries stored into every peer's block and the flags set."""
    _check(load_library().tlr_shard_push(ctx, _ptr(h), n, v_offset, _stream_handle(stream)), "tlr_shard_push")


def tlr_shard_finish_fused(ctx, n: int, tau: float, token, conf, entropy, route_mask, routed_idx, routed_count,
                           stream=None):
    """Waits (bounded, on the device) for every rank's flag, then merges and decides like tlr_route."""
    _check(load_library().tlr_shard_finish_fused(ctx, n, tau, _ptr(token), _ptr(conf), _ptr(entropy),
                                                 _ptr(route_mask), _ptr(routed_idx), _ptr(routed_count),
                                                 _stream_handle(stream)), "tlr_shard_finish_fused")


def tlr_rows_merge(gathered_idx, counts, row_offsets, ranks: int, cap: int, global_idx, global_count, stream=None):
    """Row-sharded batches: the ranks' routed-index lists [ranks][cap] -> one ascending list of global rows."""
    _check(load_library().tlr_rows_merge(_ptr(gathered_idx), _ptr(counts), _ptr(row_offsets), ranks, cap,
                                         _ptr(global_idx), _ptr(global_count), _stream_handle(stream)),
           "tlr_rows_merge")


def tlr_route_static(d: int, V: int, W, h, n: int, tau: float, token, conf, entropy, route_mask, routed_idx,
                     routed_count, status=None, stream=None):
    """The routing step without a context and without any device allocation (at most TLR_STATIC_MAX_ROWS rows).

    For callers that may not allocate GPU memory; the scratch is a fixed array inside the library,
    shared by all calls, so calls must not overlap on the GPU.  Make the first call on a device
    outside stream capture (it does a one-time set-up).
    """
    _check(load_library().tlr_route_static(d, V, _ptr(W), _ptr(h), n, tau, _ptr(token), _ptr(conf), _ptr(entropy),
                                           _ptr(route_mask), _ptr(routed_idx), _ptr(routed_count), _ptr(status),
                                           _stream_handle(stream)), "tlr_route_static")


def tlr_destroy(ctx):
    _check(load_library().tlr_destroy(ctx), "tlr_destroy")


def tlr_last_device_status(ctx) -> int:
    out = c_uint32(0)
    _check(load_library().tlr_last_device_status(ctx, byref(out)), "tlr_last_device_status")
    return out.value


def tlr_debug_inject(ctx, kind: int, wait_limit_ms: int = 0):
    """Test hook: kind=1 drops the W copies of the next calls so a bounded wait runs out; kind=0 restores."""
    _check(load_library().tlr_debug_inject(ctx, kind, wait_limit_ms), "tlr_debug_inject")


def tlr_debug_plan_tiles(n: int, V: int, sm_count: int = 148, mlp_hidden: int = 0):
    """Host-only: the tensor-core kernel's tile schedule as an int32 array [tiles, 5] and its plan
    (mlp_hidden > 0: with a learned router of that width inside the launch)."""
    import numpy as np
    lib = load_library()
    count, plan = c_int32(0), TlrPlan()
    _check(lib.tlr_debug_plan_tiles(n, V, sm_count, mlp_hidden, c_void_p(0), 0, byref(count), byref(plan)),
           "tlr_debug_plan_tiles")
    out = np.zeros((count.value, 5), dtype=np.int32)
    _check(lib.tlr_debug_plan_tiles(n, V, sm_count, mlp_hidden, c_void_p(out.ctypes.data), count.value, byref(count),
                                    byref(plan)), "tlr_debug_plan_tiles")
    return out, plan


def tlr_set_path(ctx, path: int):
    _check(load_library().tlr_set_path(ctx, path), "tlr_set_path")


def tlr_plan_query(ctx, n: int) -> TlrPlan:
    plan = TlrPlan()
    _check(load_library().tlr_plan_query(ctx, n, byref(plan)), "tlr_plan_query")
    return plan


def tlr_set_kernel_timing(ctx, enabled: bool):
    _check(load_library().tlr_set_kernel_timing(ctx, 1 if enabled else 0), "tlr_set_kernel_timing")


def tlr_read_kernel_timing(ctx):
    n, ms = c_int32(0), c_float(0.0)
    _check(load_library().tlr_read_kernel_timing(ctx, byref(n), byref(ms)), "tlr_read_kernel_timing")
    return n.value, ms.value


class Router:
    """Convenience owner of a context and its output tensors (allocation only; no arithmetic)."""

    def __init__(self, W: torch.Tensor, max_n: int, wscale: torch.Tensor = None):
        """W: bf16 [V, d]; or, with wscale (float32 [V]), e4m3 codes (uint8 / float8_e4m3fn) [V, d] for decode batches."""
        fp8 = wscale is not None
        ok_dtype = W.dtype in (torch.uint8, torch.float8_e4m3fn) if fp8 else W.dtype == torch.bfloat16
        if not (W.is_cuda and ok_dtype and W.dim() == 2 and W.is_contiguous()):
            raise ValueError("W must be a contiguous CUDA [V, d] tensor, bf16 or (with wscale) e4m3 codes")
        if fp8 and not (wscale.is_cuda and wscale.dtype == torch.float32 and wscale.shape == (W.shape[0],)
                        and wscale.is_contiguous()):
            raise ValueError("wscale must be a contiguous CUDA float32 [V] tensor")
        self.W = W                      # keep the borrowed matrix alive
        self.wscale = wscale
        self.V, self.d = W.shape
        self.max_n = max_n
        with torch.cuda.device(W.device):
            self.ctx = tlr_create_fp8(self.d, self.V, W, wscale, max_n) if fp8 else tlr_create(self.d, self.V, W, max_n)
            dev = W.device
            self.token = torch.empty(max_n, dtype=torch.int32, device=dev)
            self.conf = torch.empty(max_n, dtype=torch.float32, device=dev)
            self.entropy = torch.empty(max_n, dtype=torch.float32, device=dev)
            self.route_mask = torch.empty(max_n, dtype=torch.uint8, device=dev)
            self.routed_idx = torch.empty(max_n, dtype=torch.int32, device=dev)
            self.routed_count = torch.zeros(1, dtype=torch.int32, device=dev)

    def set_router_mlp(self, W1: torch.Tensor, b1: torch.Tensor, w2: torch.Tensor, b2: float):
        """Attach a learned router; the tensors are kept alive by this object."""
        self._mlp = (W1, b1, w2)
        tlr_set_router_mlp(self.ctx, W1.shape[0], W1, b1, w2, float(b2))

    def route(self, h: torch.Tensor, tau: float, stream=None, tau_per_row=None, route_above=False, seq_len=0,
              first_routed=None, score_source=0, mlp_score=None):
        """Enqueues one routing step; returns views of the output tensors (valid after the stream syncs)."""
        if not (h.is_cuda and h.dtype == torch.bfloat16 and h.dim() == 2 and h.is_contiguous()
                and h.shape[1] == self.d):
            raise ValueError("h must be a contiguous CUDA bf16 [n, d] tensor")
        n = h.shape[0]
        if tau_per_row is None and not route_above and seq_len == 0 and score_source == 0 and mlp_score is None:
            tlr_route(self.ctx, h, n, tau, self.token, self.conf, self.entropy, self.route_mask, self.routed_idx,
                      self.routed_count, stream)
        else:
            tlr_route_ex(self.ctx, h, n, tau, self.token, self.conf, self.entropy, self.route_mask, self.routed_idx,
                         self.routed_count, stream, tau_per_row=tau_per_row, route_above=route_above,
                         seq_len=seq_len, first_routed=first_routed, score_source=score_source,
                         mlp_score=mlp_score)
        return (self.token[:n], self.conf[:n], self.entropy[:n], self.route_mask[:n], self.routed_idx,
                self.routed_count)

    def prepared(self, h: torch.Tensor, tau: float, stream=None):
        """The same step as route(h, tau, stream) as a callable with its arguments marshalled once: for a decode
        loop that calls again and again with the same buffers, each call is then a single foreign call.  The
        outputs are this router's tensors, as with route()."""
        if not (h.is_cuda and h.dtype == torch.bfloat16 and h.dim() == 2 and h.is_contiguous()
                and h.shape[1] == self.d):
            raise ValueError("h must be a contiguous CUDA bf16 [n, d] tensor")
        fn = load_library().tlr_route
        args = (self.ctx, _ptr(h), int(h.shape[0]), float(tau), _ptr(self.token), _ptr(self.conf), _ptr(self.entropy),
                _ptr(self.route_mask), _ptr(self.routed_idx), _ptr(self.routed_count), _stream_handle(stream))
        keep = (h, stream, self)       # the buffers stay alive as long as the callable does

        def call():
            _check(fn(*args), "tlr_route")
            return keep[2]

        return call

    def close(self):
        if self.ctx is not None:
            tlr_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

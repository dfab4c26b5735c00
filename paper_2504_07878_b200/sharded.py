"""Vocabulary-sharded routing step over several GPUs: plumbing only (bounds, buffers, the all-gather).

One process per GPU.  Rank g keeps rows [v0, v1) of W on its GPU and calls tlr_shard_summary on them; the
16-byte per-row summaries are exchanged with one all-gather (n x 16 bytes per rank; NCCL on GPUs), and
every rank runs tlr_shard_finish on the gathered block, so every rank ends with the full decision.
All arithmetic is in the library's kernels.
"""
from __future__ import annotations

import torch

from . import binding as B

GRANULE = 32          # shard boundaries fall on multiples of this many vocabulary rows


def shard_bounds(V: int, world: int, rank: int):
    """Contiguous, near-equal split of [0, V) at multiples of GRANULE rows: rows [v0, v1) of rank `rank`."""
    if not (0 <= rank < world) or V <= 0:
        raise ValueError("bad shard request")
    granules = (V + GRANULE - 1) // GRANULE
    if granules < world:
        raise ValueError("vocabulary too small for %d shards" % world)
    g0 = granules * rank // world
    g1 = granules * (rank + 1) // world
    return g0 * GRANULE, min(V, g1 * GRANULE)


def gather_summaries(local: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather of the per-row summaries: local [n, 4] (16 bytes per row) -> [world, n, 4], rank-major."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    out = torch.empty((world,) + tuple(local.shape), dtype=local.dtype, device=local.device)
    dist.all_gather(list(out.unbind(0)), local.contiguous(), group=group)     # slot g = rank g's rows
    return out


class VocabShardedRouter:
    """Owner of one rank's context (on its rows of W), its summary buffers and the output tensors."""

    def __init__(self, W_shard: torch.Tensor, v_offset: int, max_n: int, world: int, group=None, wscale=None):
        """W_shard: this rank's rows of W, bf16 [V_local, d]; or, with wscale (float32 [V_local]), their e4m3 codes
        (decode batches of up to 64 rows, see tlr_create_fp8)."""
        fp8 = wscale is not None
        ok_dtype = W_shard.dtype in (torch.uint8, torch.float8_e4m3fn) if fp8 else W_shard.dtype == torch.bfloat16
        if not (W_shard.is_cuda and ok_dtype and W_shard.dim() == 2 and W_shard.is_contiguous()):
            raise ValueError("W_shard must be a contiguous CUDA [V_local, d] tensor, bf16 or (with wscale) e4m3 codes")
        self.W = W_shard
        self.wscale = wscale
        self.v_offset = int(v_offset)
        self.world = int(world)
        self.group = group
        self.max_n = max_n
        dev = W_shard.device
        with torch.cuda.device(dev):
            if fp8:
                self.ctx = B.tlr_create_fp8(W_shard.shape[1], W_shard.shape[0], W_shard, wscale, max_n)
            else:
                self.ctx = B.tlr_create(W_shard.shape[1], W_shard.shape[0], W_shard, max_n)
            self.summary = torch.empty((max_n, 4), dtype=torch.float32, device=dev)     # 16 bytes per row
            self.token = torch.empty(max_n, dtype=torch.int32, device=dev)
            self.conf = torch.empty(max_n, dtype=torch.float32, device=dev)
            self.entropy = torch.empty(max_n, dtype=torch.float32, device=dev)
            self.route_mask = torch.empty(max_n, dtype=torch.uint8, device=dev)
            self.routed_idx = torch.empty(max_n, dtype=torch.int32, device=dev)
            self.routed_count = torch.zeros(1, dtype=torch.int32, device=dev)

    def summarize(self, h: torch.Tensor, stream=None) -> torch.Tensor:
        n = h.shape[0]
        B.tlr_shard_summary(self.ctx, h, n, self.v_offset, self.summary, stream)
        return self.summary[:n]

    def finish(self, gathered: torch.Tensor, n: int, tau: float, stream=None):
        B.tlr_shard_finish(self.ctx, gathered, gathered.shape[0], n, tau, self.token, self.conf, self.entropy,
                           self.route_mask, self.routed_idx, self.routed_count, stream)
        return (self.token[:n], self.conf[:n], self.entropy[:n], self.route_mask[:n], self.routed_idx,
                self.routed_count)

    def route(self, h: torch.Tensor, tau: float):
        """Summary on this rank's shard, all-gather over the group, merge and decision on every rank."""
        n = h.shape[0]
        local = self.summarize(h)
        gathered = gather_summaries(local, self.group) if self.world > 1 else local.unsqueeze(0)
        return self.finish(gathered.contiguous(), n, tau)

    def close(self):
        if self.ctx is not None:
            B.tlr_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

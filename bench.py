#!/usr/bin/env python
"""Benchmark of the token-routing step (one step = one tlr_route call over one batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line.  The default workload is the batched-decode configuration
(256 sessions x 1 token, d=896, V=151936, tau=0.5) on synthetic seeded inputs.
With --gpus N > 1 (launched under torch.distributed.run) every rank routes its own
batch of the same size with its own copy of W (rows are independent units, so the
path shards with no data-path collective): weak scaling, time = max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import tlr_synth as S  # noqa: E402

METRIC = "routed-path tokens/s (rows through tlr_route per second, all six outputs)"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
RIDGE_ROWS_HBM = 256            # at or below this many rows the step is reported against the HBM roofline

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the projection kernel, from the ncu
# captures summarised under profiles/.  Only valid for the kernel source they were taken on: the
# hash of that source is recorded here and traffic is reported as null when the source differs.
NCU_TRAFFIC = {
    "kernel_sources": ["paper_2504_07878_b200/csrc/tlr_tc_kernel.cuh", "paper_2504_07878_b200/csrc/tlr_tc_ptx.cuh"],
    "sha256": "ad20ef2b7c5159246522e6c7c2b720eb8a483e50cce12ecae6fcb02813170e00",
    "bytes_per_launch": {"decode256": 274.54e6, "decode16": 274.09e6, "sweep512": 529.42e6},
}


def ncu_traffic(workload):
    import hashlib
    digest = hashlib.sha256()
    try:
        for rel in NCU_TRAFFIC["kernel_sources"]:
            with open(os.path.join(ROOT, rel), "rb") as f:
                digest.update(f.read())
    except OSError:
        return None
    if digest.hexdigest() != NCU_TRAFFIC["sha256"]:
        return None
    return NCU_TRAFFIC["bytes_per_launch"].get(workload)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def algorithmic_bytes(n, d, V, fp8=False):
    """W once + h once + the six outputs (17 bytes per row + the count); an 8-bit W is V*d bytes + V scales."""
    w_bytes = V * d + 4 * V if fp8 else 2 * V * d
    return w_bytes + 2 * n * d + 17 * n + 4


def algorithmic_flops(n, d, V):
    return 2 * n * d * V


class ClockSampler:
    """Polls NVML (SM clock, power, throttle reasons) from the host while the GPU works."""

    def __init__(self, index):
        self.samples = []
        self.reasons = set()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.max_mhz = None

    def sample(self):
        if not self.ok:
            return
        nv = self.nv
        try:
            self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
            names = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown,
                     "hw_thermal_slowdown": nv.nvmlClocksEventReasonHwThermalSlowdown,
                     "sw_thermal_slowdown": nv.nvmlClocksEventReasonSwThermalSlowdown,
                     "sw_power_cap": nv.nvmlClocksEventReasonSwPowerCap}
            for k, bit in names.items():
                if r & bit:
                    self.reasons.add(k)
        except Exception:
            pass

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(x, world, device):
    """The slowest rank's time decides the job's throughput (works on nccl and gloo groups)."""
    if world <= 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([float(x)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world, rows_per_rank, seconds_per_step):
    """Weak scaling: every rank routes its own rows_per_rank rows per step."""
    return world * rows_per_rank / seconds_per_step


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


NOMINAL_HBM_GBS = 8000.0        # HBM3e, datasheet
NOMINAL_BF16_TFLOPS = 2250.0    # dense bf16, datasheet


def roofline_fractions(n, d, V, seconds, peaks, fp8=False):
    """The three fractions every record carries, from one duration: HBM, tensor against the burst cuBLAS
    figure, tensor against the sustained one; and the ridge reading max(t_mem, t_mma) / t with t_mma at the
    burst figure (both pipes would be busy for the longer of the two times at best)."""
    by, fl = algorithmic_bytes(n, d, V, fp8), algorithmic_flops(n, d, V)
    t_mem = by / (float(peaks["hbm_gbs"]) * 1e9)
    t_mma = fl / (float(peaks["bf16_tflops"]) * 1e12)
    t_mma_sus = fl / (float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])) * 1e12)
    return {"hbm_frac": t_mem / seconds, "tensor_frac_burst": t_mma / seconds,
            "tensor_frac_sustained": t_mma_sus / seconds, "ridge_frac": max(t_mem, t_mma) / seconds,
            # the same duration against the datasheet figures (context; the measured peaks are the roofline)
            "hbm_frac_of_nominal": by / (NOMINAL_HBM_GBS * 1e9) / seconds,
            "tensor_frac_of_nominal": fl / (NOMINAL_BF16_TFLOPS * 1e12) / seconds}


def time_steps(P, routers, step, steps, sampler, world, kernel_steps):
    """K steps between two CUDA events on the launching stream (clocks sampled meanwhile), then, back to
    back, `kernel_steps` more steps with the projection kernel bracketed by events inside tlr_route.
    Returns (ms per step, ms per projection launch, projection launches timed, seconds of continuous load)."""
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        step(i)
    e1.record(stream)
    while not e1.query():
        sampler.sample()
        time.sleep(0.002)
    sampler.sample()
    for r in routers:
        P.tlr_set_kernel_timing(r.ctx, True)
    for i in range(kernel_steps):
        step(i)
    e2 = torch.cuda.Event(enable_timing=True)
    e2.record(stream)
    while not e2.query():
        sampler.sample()
        time.sleep(0.002)
    torch.cuda.synchronize()
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
    load_s = e0.elapsed_time(e2) * 1e-3
    launches, kms = 0, 0.0
    for r in routers:
        ln, ms = P.tlr_read_kernel_timing(r.ctx)
        launches += ln
        kms += ms
        P.tlr_set_kernel_timing(r.ctx, False)
    return ms_total / steps, kms / max(launches, 1), launches, load_s


def side_record(P, name, routers, h_dev, tau, seconds, gpu_index, peaks, fp8=False):
    """One more workload on heads that are already resident: about `seconds` of back-to-back steps."""
    wl = S.WORKLOADS[name]
    n, d, V = wl.n, wl.d, wl.V
    stream = torch.cuda.current_stream()

    def step(i):
        routers[i % len(routers)].route(h_dev, tau, stream)

    for i in range(5):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(4):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    per = max(e0.elapsed_time(e1) / 4 * 1e-3, 1e-6)
    steps = int(max(20, min(20000, seconds / per)))
    ksteps = int(max(10, min(steps // 2, 4000)))
    sampler = ClockSampler(gpu_index)
    ms, kms, launches, load_s = time_steps(P, routers, step, steps, sampler, 1, ksteps)
    status = max(P.tlr_last_device_status(r.ctx) for r in routers)
    if status & P.TLR_DEV_WAIT_TIMEOUT:
        raise SystemExit("device status flags raised in the %s record: %d" % (name, status))
    rec = {"workload": "%s%s: n=%d rows, d=%d, V=%d, tau=%g" % (name, " with an 8-bit copy of W" if fp8 else "", n, d, V, tau),
           "steps": steps, "ms_per_step": ms, "value": n / (ms * 1e-3), "unit": UNIT,
           "kernel_ms": kms, "kernel_launches_timed": launches, "continuous_load_s": load_s,
           "bound": "hbm" if n <= RIDGE_ROWS_HBM else "tensor", "clocks": sampler.summary(),
           "routed_rows_per_step": int(routers[0].routed_count.item())}
    rec["kernel"] = roofline_fractions(n, d, V, kms * 1e-3, peaks, fp8)
    rec["step"] = roofline_fractions(n, d, V, ms * 1e-3, peaks, fp8)
    rec["frac"] = rec["kernel"]["hbm_frac" if n <= RIDGE_ROWS_HBM else "tensor_frac_burst"]
    return rec


def run_one_rank_of_a_vocab_shard(args):
    """--one-shard-of G on one GPU: the work ONE rank of a G-way vocabulary-sharded step does per call -- the
    projection over V / G rows of W, the per-row summaries stored into the exchange block, the bounded wait on
    the flags and the merge.  All G ranks run one after the other in one stream (every "peer" block is the same
    local block): G pushes, then G merges, and the time per rank is that of the loop divided by G.  No exchange
    latency is in it (there is one GPU); it gives the per-rank time a G-GPU run could approach."""
    import paper_2504_07878_b200 as P
    from paper_2504_07878_b200 import build
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the routing path has no CPU fallback")
    torch.cuda.set_device(0)
    build.build()
    P.load_library()
    G = args.one_shard_of
    wl = S.WORKLOADS[args.workload]
    n, d, V = wl.n, wl.d, wl.V
    tau = 0.5 if wl.tau is None else wl.tau
    h = S.make_h(n, d, seed=0).h.cuda()
    # Two complete sets of ranks (each set: the G shards of its own copy of W, its own exchange block) alternate
    # between steps, so that a step streams its shards from HBM rather than from what the last step left in L2.
    sets = []
    W_host = S.make_W(d, V, seed=0)
    for _ in range(2):
        W = W_host.cuda()
        block = torch.zeros(P.tlr_shard_block_bytes(n, G), dtype=torch.uint8, device="cuda")
        ranks = []
        for g in range(G):
            v0, v1 = P.shard_bounds(V, G, g)
            ranks.append(P.FusedVocabShardedRouter(W[v0:v1], v0, n, g, G, [block] * G, keep=(block, W)))
        sets.append(ranks)
    stream = torch.cuda.current_stream()

    def step(i):
        ranks = sets[i & 1]
        for r in ranks:
            r.push(h)
        for r in ranks:
            r.finish(n, tau)

    for i in range(max(3, args.warmup)):
        step(i)
    steps = min(args.steps, 2000)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    ms_all = e0.elapsed_time(e1) / steps
    ms = ms_all / G
    status = max(P.tlr_last_device_status(r.ctx) for ranks in sets for r in ranks)
    if status & P.TLR_DEV_WAIT_TIMEOUT:
        raise SystemExit("device status flags raised: %d" % status)
    peaks, peak_kind = measured_peaks()
    v0, v1 = P.shard_bounds(V, G, 0)
    shard_bytes = 2 * (v1 - v0) * d + 2 * n * d + 17 * n + 4 + 16 * n * G
    print(json.dumps({"metric": METRIC, "value": n / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": steps,
                      "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "scaling": "strong",
                      "vs_baseline": None, "dtype": "bf16 in, fp32 accumulate and softmax statistics", "data": "synthetic",
                      "config": {"workload": "%s, ONE rank's share of a %d-way vocabulary-sharded step: n=%d rows, d=%d, "
                                             "%d of V=%d rows of W, tau=%g" % (wl.name, G, n, d, v1 - v0, V, tau),
                                 "l2": "two sets of %d ranks (two copies of W) alternate between steps; time = a back-to-back "
                                       "loop in which all %d ranks push and then all merge (%.4f ms), divided by %d"
                                       % (G, G, ms_all, G),
                                 "exchange": "fused: summaries stored into the exchange block, flags, bounded wait in "
                                             "the merge kernel (one GPU: no link latency in this number)"},
                      "gpu_launches": 3 * G * steps,
                      "roofline": {"bound": "hbm", "achieved": shard_bytes / (ms * 1e-3) / 1e9, "peak": float(peaks["hbm_gbs"]),
                                   "unit": "GB/s", "frac": shard_bytes / (ms * 1e-3) / 1e9 / float(peaks["hbm_gbs"]),
                                   "traffic": None, "algorithmic_bytes": shard_bytes, "peak_source": "of " + peak_kind,
                                   "kernel": "tc_projection_kernel + shard_push_kernel + finish_small_kernel (whole call)"}}))


def run_ours(args):
    import paper_2504_07878_b200 as P
    from paper_2504_07878_b200 import build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("--gpus %d needs `python -m torch.distributed.run --nproc-per-node %d`"
                             % (args.gpus, args.gpus))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the routing path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if rank == 0:
        build.build()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    P.load_library()
    gpu_index = physical_gpu_index(local_rank)
    peaks, peak_kind = measured_peaks()

    wl = S.WORKLOADS[args.workload]
    n, d, V = wl.n, wl.d, wl.V
    tau = 0.5 if wl.tau is None else wl.tau
    if args.tau is not None:
        tau = args.tau
    fp8 = bool(args.fp8)
    if fp8 and n > 128:
        raise SystemExit("--fp8 serves decode batches only (n <= 128): pick decode16 or sweep1/8/64, or --rows N")
    # two device copies of W, alternated step by step: together with W > L2 (or, for the 8-bit copy
    # of the 0.5B head, two copies > L2) this makes every step stream W from HBM rather than from
    # whatever the previous step left in L2
    copies = 2
    if fp8:
        codes, wscale = S.make_W8(d, V, seed=0)
        W_host = None
        hid = S.make_h(n, d, seed=rank)
        Ws = [(codes.cuda(), wscale.cuda()) for _ in range(copies)]
        routers = [P.Router(c, max_n=n, wscale=sc) for c, sc in Ws]
    else:
        W_host = S.make_W(d, V, seed=0)
        hid = S.make_h(n, d, seed=rank, W=W_host, planted_fraction=wl.planted_fraction)
        Ws = [W_host.cuda() for _ in range(copies)]
        routers = [P.Router(w, max_n=n) for w in Ws]
    h_dev = hid.h.cuda()
    plan = P.tlr_plan_query(routers[0].ctx, n)
    stream = torch.cuda.current_stream()

    variant_args = {}
    if args.variants:
        seq_len = args.seq_len if args.seq_len > 0 else (512 if n % 512 == 0 else 1)
        variant_args = {"tau_per_row": torch.full((n,), tau, dtype=torch.float32, device="cuda"),
                        "seq_len": seq_len,
                        "first_routed": torch.zeros(n // seq_len, dtype=torch.int32, device="cuda")}

    if args.mlp > 0:
        g = torch.Generator().manual_seed(0)
        W1 = (torch.randn(args.mlp, d, generator=g) / d ** 0.5).to(torch.bfloat16).cuda()
        b1 = (torch.randn(args.mlp, generator=g) * 0.1).cuda()
        w2 = (torch.randn(args.mlp, generator=g) * 0.5).cuda()
        for r in routers:
            r.set_router_mlp(W1, b1, w2, 0.0)
        variant_args["score_source"] = P.TLR_SCORE_MLP

    if variant_args:
        def step(i):
            routers[i % copies].route(h_dev, tau, stream, **variant_args)
    else:
        # arguments marshalled once: each step is one call into the library
        calls = [r.prepared(h_dev, tau, stream) for r in routers]

        def step(i):
            calls[i % copies]()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()

    # ---- timed region: exactly K steps, device time between two events, clocks sampled meanwhile;
    # then, back to back, the dominant kernel alone (bracketed by events inside tlr_route)
    sampler = ClockSampler(gpu_index)
    ms_per_step, kernel_ms, launches, load_s = time_steps(P, routers, step, args.steps, sampler, world,
                                                          min(args.steps, 2000))
    barrier()
    status = max(P.tlr_last_device_status(r.ctx) for r in routers)
    if status & P.TLR_DEV_WAIT_TIMEOUT:
        raise SystemExit("device status flags raised during the timed region: %d" % status)
    routed = int(routers[0].routed_count.item())

    # ---- end to end through the host-buffer entry point (pinned host memory)
    h_pin = hid.h.pin_memory()
    o_tok = torch.empty(n, dtype=torch.int32).pin_memory()
    o_conf = torch.empty(n, dtype=torch.float32).pin_memory()
    o_ent = torch.empty(n, dtype=torch.float32).pin_memory()
    o_mask = torch.empty(n, dtype=torch.uint8).pin_memory()
    o_idx = torch.empty(n, dtype=torch.int32).pin_memory()
    o_cnt = torch.zeros(1, dtype=torch.int32).pin_memory()
    esteps = min(args.steps, 2000)

    def host_step(i):
        P.tlr_route_host(routers[i % copies].ctx, h_pin, n, tau, o_tok, o_conf, o_ent, o_mask, o_idx, o_cnt, stream)

    for i in range(max(3, min(args.warmup, 20))):
        host_step(i)
    barrier()
    t0 = time.perf_counter()
    for i in range(esteps):
        host_step(i)
    torch.cuda.synchronize()
    e2e_sync_s = max_over_ranks(time.perf_counter() - t0, world, "cuda")
    # ... and with two calls in flight per context (submit / collect): every step still brings its h in from the
    # pinned host buffer and hands its six results back to the host, but the transfer, the launches and the
    # host's wake-up overlap the previous step's kernels
    outs = (o_tok, o_conf, o_ent, o_mask, o_idx, o_cnt)

    def pipelined(steps):
        ctx_of = lambda i: routers[i % copies].ctx
        P.tlr_route_host_submit(ctx_of(0), h_pin, n, tau, stream)
        for i in range(1, steps):
            P.tlr_route_host_submit(ctx_of(i), h_pin, n, tau, stream)
            P.tlr_route_host_collect(ctx_of(i - 1), *outs)
        P.tlr_route_host_collect(ctx_of(steps - 1), *outs)

    pipelined(max(3, min(args.warmup, 20)))
    barrier()
    t0 = time.perf_counter()
    pipelined(esteps)
    torch.cuda.synchronize()
    e2e_s = max_over_ranks(time.perf_counter() - t0, world, "cuda")
    h2d = n * d * 2
    d2h = 17 * n + 4 + 4      # the six outputs in one block (routed_idx at full capacity) + the status word

    # ---- the same step under sustained load, and the other regimes of the target on the same head
    sustained = None
    also = []
    if world == 1 and args.extras and args.workload == "decode256" and not fp8 and not variant_args:
        sustained = side_record(P, "decode256", routers, h_dev, tau, 1.5, gpu_index, peaks)
        sustained["note"] = ("the benchmark step back to back for about 1.5 s, then the kernel-timing pass: the "
                             "power-capped regime; compare time x clocks.sm_mhz with the short run above")
        torch.cuda.synchronize()
        time.sleep(0.5)
        wl16 = S.WORKLOADS["decode16"]
        r16 = [P.Router(w, max_n=wl16.n) for w in Ws]
        also.append(side_record(P, "decode16", r16, S.make_h(wl16.n, d, seed=0).h.cuda(), 0.5, 0.3, gpu_index, peaks))
        for r in r16:
            r.close()
        wlp = S.WORKLOADS["prefill8192"]
        rp = [P.Router(w, max_n=wlp.n) for w in Ws]
        hp = S.make_h(wlp.n, d, seed=0, W=W_host, planted_fraction=wlp.planted_fraction).h.cuda()
        also.append(side_record(P, "prefill8192", rp, hp, wlp.tau, 1.2, gpu_index, peaks))
        for r in rp:
            r.close()
        del rp, hp
        codes, wscale = S.make_W8(d, V, seed=0)
        W8 = [(codes.cuda(), wscale.cuda()) for _ in range(copies)]
        r8 = [P.Router(c, max_n=wl16.n, wscale=sc) for c, sc in W8]
        also.append(side_record(P, "decode16", r8, S.make_h(wl16.n, d, seed=0).h.cuda(), 0.5, 0.3, gpu_index, peaks,
                                fp8=True))
        for r in r8:
            r.close()
        del r8, W8
        # the two other heads of the target (1.5B-class head; the d = 2048 sweep at an HBM-bound and a
        # tensor-bound batch size): one device copy each, W alone is three to four times L2
        for names in (("head1p5b",), ("sweep64", "sweep4096")):
            wlx = S.WORKLOADS[names[0]]
            Wx = S.make_W(wlx.d, wlx.V, seed=0).cuda()
            for name in names:
                wly = S.WORKLOADS[name]
                rx = [P.Router(Wx, max_n=wly.n)]
                hx = S.make_h(wly.n, wly.d, seed=0).h.cuda()
                rec = side_record(P, name, rx, hx, 0.5 if wly.tau is None else wly.tau,
                                  0.3 if wly.n <= RIDGE_ROWS_HBM else 1.0, gpu_index, peaks)
                rec["l2"] = "one device copy of W (%.0f MB, larger than L2)" % (2 * wly.V * wly.d / 1e6)
                also.append(rec)
                rx[0].close()
                del rx, hx
            del Wx

    # ---- N > 1: the vocabulary-sharded form of the same decode batch (one exchange step per call)
    vocab_sharded = None
    if world > 1 and n <= 1024 and not fp8 and not variant_args:
        # (a sub-record beside the line's own numbers: an error in it is reported, not allowed to lose the line)
        try:
            vocab_sharded = vocab_sharded_record(P, W_host, S.make_h(n, d, seed=0).h, tau, rank, world, args.steps,
                                                 max(args.warmup, 3))
        except Exception as e:      # noqa: BLE001
            vocab_sharded = {"unavailable": "%s: %s" % (type(e).__name__, e)}

    if rank != 0:
        return
    value = job_throughput(world, n, ms_per_step * 1e-3)
    kfr = roofline_fractions(n, d, V, kernel_ms * 1e-3, peaks, fp8)
    sfr = roofline_fractions(n, d, V, ms_per_step * 1e-3, peaks, fp8)
    hbm_bound = n <= RIDGE_ROWS_HBM
    if hbm_bound:
        achieved = algorithmic_bytes(n, d, V, fp8) / (kernel_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
                "frac": kfr["hbm_frac"]}
    else:
        # always held against the burst cuBLAS figure; the fraction of the sustained figure is beside it
        achieved = algorithmic_flops(n, d, V) / (kernel_ms * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": float(peaks["bf16_tflops"]), "unit": "TFLOP/s",
                "frac": kfr["tensor_frac_burst"], "peak_kind": "burst"}
    roof.update({"traffic": None if (fp8 or args.rows > 0) else ncu_traffic(wl.name), "algorithmic_bytes": algorithmic_bytes(n, d, V, fp8),
                 "algorithmic_flops": algorithmic_flops(n, d, V), "peak_source": "of " + peak_kind,
                 "kernel": ("h_split_kernel + tc8_projection_kernel" if fp8 else
                            "tc_projection_kernel" if plan.path == P.TLR_PATH_TC else "simt_projection_kernel"),
                 "kernel_ms": kernel_ms, "kernel_launches_timed": launches, "continuous_load_s": load_s,
                 # the projection kernel alone (timed by events inside tlr_route, which also switch off the
                 # overlap of its prologue with the previous merge kernel) and the whole step (projection +
                 # merge launches, as timed for tokens/s), each against all three peaks and the ridge bound
                 "kernel_fracs": kfr, "step_fracs": sfr,
                 "step_frac": sfr["hbm_frac"] if hbm_bound else sfr["tensor_frac_burst"],
                 "ridge_frac": kfr["ridge_frac"],
                 "hbm_frac_same_launch": kfr["hbm_frac"], "tensor_frac_same_launch": kfr["tensor_frac_burst"],
                 "tensor_frac_of_sustained": kfr["tensor_frac_sustained"]})

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": ("e4m3 W with one scale per row, bf16 h split into two e4m3 parts, fp32 accumulate and softmax statistics"
                  if fp8 else "bf16 in, fp32 accumulate and softmax statistics"), "data": "synthetic",
        "config": {"workload": "%s%s: n=%d rows, d=%d, V=%d, tau=%g%s" % (wl.name, " with an 8-bit copy of W" if fp8 else "",
                                                                        n, d, V, tau,
                                                                       ", %.0f%% planted rows" % (100 * wl.planted_fraction)
                                                                       if wl.planted_fraction else ""),
                   "l2": "inputs larger than L2: W is %.0f MB and two device copies of it alternate between steps"
                         % ((V * d if fp8 else 2 * V * d) / 1e6),
                   "path": int(plan.path), "grid": int(plan.grid), "block": int(plan.block),
                   "vocab_chunks": int(plan.vocab_chunks), "routed_rows_per_step": routed,
                   "variants": (("per-row tau + first routed per sequence of %d" % variant_args["seq_len"])
                                if "seq_len" in variant_args else "none") +
                               ("; learned router, hidden width %d" % args.mlp if args.mlp > 0 else "")},
        "e2e": {"value": job_throughput(world, n, e2e_s / esteps), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": esteps,
                "api": "tlr_route_host_submit / tlr_route_host_collect, two calls in flight (pinned host buffers)",
                "frac_of_device_rate": (ms_per_step * 1e-3) / (e2e_s / esteps),
                "one_call_at_a_time": {"value": job_throughput(world, n, e2e_sync_s / esteps), "api": "tlr_route_host",
                                       "frac_of_device_rate": (ms_per_step * 1e-3) / (e2e_sync_s / esteps)}},
        # (a learned router runs inside the projection launch wherever the tensor-core kernel does: d % 8 == 0)
        "gpu_launches": (int(plan.launches) + (1 if args.mlp > 0 and (fp8 or d % 8 != 0) else 0)) * args.steps,
        "clocks": sampler.summary(),
        "roofline": roof,
    }
    if sustained is not None:
        out["sustained"] = sustained
    if also:
        out["also"] = also
    if vocab_sharded is not None:
        out["vocab_sharded"] = vocab_sharded
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl, W_host, hid, tau, budget_s=15.0, w8=(codes, wscale) if fp8 else None)
    print(json.dumps(out))


def vocab_sharded_record(P, W_host, h_cpu, tau, rank, world, steps, warmup):
    """The same batch with the vocabulary sharded over the ranks (each holds V / world rows of W): projection
    on the shard, one all-gather of n x 16 bytes per rank over NCCL, merge and decision on every rank.  Total
    work is fixed as N grows (strong scaling of one decode batch); time is the max over ranks."""
    import torch.distributed as dist
    V = W_host.shape[0]
    n = h_cpu.shape[0]
    v0, v1 = P.shard_bounds(V, world, rank)
    copies = 2          # two copies of the shard alternate, as in the main loop (a shard may fit in L2)
    shards = [W_host[v0:v1].cuda() for _ in range(copies)]
    rs = [P.VocabShardedRouter(w, v0, max_n=n, world=world) for w in shards]
    h_dev = h_cpu.cuda()
    stream = torch.cuda.current_stream()
    for i in range(warmup):
        rs[i % copies].route(h_dev, tau)
    dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        rs[i % copies].route(h_dev, tau)
    e1.record(stream)
    torch.cuda.synchronize()
    dist.barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda") / steps
    routed = int(rs[(steps - 1) % copies].routed_count.item())
    for r in rs:
        r.close()
    return {"ms_per_step": ms, "value": n / (ms * 1e-3), "unit": UNIT, "scaling": "strong", "shards": world,
            "rows_of_W_per_rank": v1 - v0, "routed_rows_per_step": routed,
            "exchange": "NCCL all-gather of %d bytes per rank per step" % (16 * n)}


def run_torch_eager(args):
    """--impl torch-eager: what the step costs when written with library calls -- cuBLAS for the logits (written to
    HBM), then torch's softmax, max, entropy, compare and nonzero.  Context beside the fused kernels, not a target
    and not the reference arm; one GPU."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    torch.cuda.set_device(0)
    wl = S.WORKLOADS[args.workload]
    n, d, V = wl.n, wl.d, wl.V
    tau = 0.5 if wl.tau is None else wl.tau
    W_host = S.make_W(d, V, seed=0)
    Ws = [W_host.cuda() for _ in range(2)]
    h = S.make_h(n, d, seed=0, W=W_host, planted_fraction=wl.planted_fraction).h.cuda()

    def step(i):
        z = torch.matmul(h, Ws[i % 2].t()).float()
        p = torch.softmax(z, dim=-1)
        conf, token = p.max(dim=-1)
        entropy = -(p * torch.log(p.clamp_min(1e-38))).sum(dim=-1)
        mask = conf < tau
        idx = torch.nonzero(mask).squeeze(-1)
        return token, conf, entropy, mask, idx

    def gemm_only(i):
        return torch.matmul(h, Ws[i % 2].t())

    def timed(fn, steps):
        for i in range(max(3, args.warmup)):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    steps = min(args.steps, 2000 if n <= 256 else 100)
    ms = timed(step, steps)
    ms_gemm = timed(gemm_only, steps)
    print(json.dumps({"impl": "torch-eager", "metric": METRIC, "value": n / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
                      "steps": steps, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "bf16 GEMM (cuBLAS), fp32 softmax", "data": "synthetic",
                      "config": {"workload": "%s: n=%d rows, d=%d, V=%d, tau=%g" % (wl.name, n, d, V, tau),
                                 "what": "torch.matmul + softmax + max + entropy + compare + nonzero, logits in HBM"},
                      "gemm_only_ms": ms_gemm, "gpu_launches": 0}))


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        ts = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if ts:
            return int(max(ts))
    except Exception:
        pass
    return os.cpu_count() or 1


def cpu_baseline(wl, W_host, hid, tau, budget_s, w8=None):
    """The fp64 oracle, as it stands, on a bounded sample of the workload's rows."""
    from oracle import route_oracle as O
    if w8 is not None:                       # the 8-bit head: the oracle runs on the de-quantised matrix
        Wb = None
        W64 = O.dequantize_e4m3(w8[0].numpy(), w8[1].numpy())
    else:
        Wb = S.bf16_bits(W_host)
        W64 = O.bf16_bits_to_f64(Wb)
    hb = S.bf16_bits(hid.h)
    probe = min(8, wl.n)
    t0 = time.perf_counter()
    O.route_oracle(hb[:probe], Wb, tau, W64=W64)
    per_row = (time.perf_counter() - t0) / probe
    rows = int(max(1, min(wl.n, budget_s / max(per_row, 1e-9))))
    t0 = time.perf_counter()
    O.route_oracle(hb[:rows], Wb, tau, W64=W64)
    dt = time.perf_counter() - t0
    return {"value": rows / dt, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": "first %d of %d rows of the same workload, W already widened to fp64, %.1f s"
                      % (rows, wl.n, dt)}


def run_reference(args):
    """The reference arm: the CPU fp64 oracle on the same workload, a bounded sample of rows per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import route_oracle as O
    wl = S.WORKLOADS[args.workload]
    tau = 0.5 if wl.tau is None else wl.tau
    W_host = S.make_W(wl.d, wl.V, seed=0)
    hid = S.make_h(wl.n, wl.d, seed=0, W=W_host, planted_fraction=wl.planted_fraction)
    Wb = S.bf16_bits(W_host)
    W64 = O.bf16_bits_to_f64(Wb)
    hb = S.bf16_bits(hid.h)
    probe = min(4, wl.n)
    t0 = time.perf_counter()
    O.route_oracle(hb[:probe], Wb, tau, W64=W64)
    per_row = (time.perf_counter() - t0) / probe
    budget = 90.0 / max(1, args.steps + args.warmup)
    rows = int(max(1, min(wl.n, budget / max(per_row, 1e-9))))
    for i in range(args.warmup):
        O.route_oracle(hb[:rows], Wb, tau, W64=W64)
    t0 = time.perf_counter()
    for i in range(args.steps):
        O.route_oracle(hb[:rows], Wb, tau, W64=W64)
    dt = time.perf_counter() - t0
    value = rows * args.steps / dt
    sample = "each step = the first %d of %d rows, W already widened to fp64" % (rows, wl.n)
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": "%s: n=%d rows, d=%d, V=%d, tau=%g" % (wl.name, wl.n, wl.d, wl.V, tau),
                      "sample": sample},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--workload", default="decode256", choices=sorted(S.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "torch-eager"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", dest="extras", action="store_false",
                    help="default workload only: skip the sustained-load record and the decode16 / prefill8192 / "
                         "8-bit records that reuse the resident head")
    ap.add_argument("--tau", type=float, default=None, help="override the workload's threshold")
    ap.add_argument("--variants", action="store_true",
                    help="route with per-row thresholds and report the first routed position per sequence "
                         "(tlr_route_ex; sequences of --seq-len rows)")
    ap.add_argument("--seq-len", type=int, default=0)
    ap.add_argument("--fp8", action="store_true",
                    help="decode workloads (n <= 128) on an 8-bit copy of W (tlr_create_fp8); the roofline then "
                         "counts one byte per weight")
    ap.add_argument("--mlp", type=int, default=0,
                    help="attach a learned router of this hidden width (random weights) and route on its score")
    ap.add_argument("--one-shard-of", type=int, default=0, metavar="G",
                    help="one GPU: time the work of ONE rank of a G-way vocabulary-sharded step (fused exchange), "
                         "a decode workload's batch on V / G rows of W")
    ap.add_argument("--rows", type=int, default=0, metavar="N",
                    help="time the workload's head with a batch of N rows instead of its own (the line's "
                         "config.workload says so)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.rows > 0:
        import dataclasses
        S.WORKLOADS[args.workload] = dataclasses.replace(S.WORKLOADS[args.workload], n=args.rows)
    if args.impl == "torch-eager":
        run_torch_eager(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.one_shard_of > 1:
        run_one_rank_of_a_vocab_shard(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

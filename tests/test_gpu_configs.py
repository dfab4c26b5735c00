"""GPU parity at the full benchmark sizes, in the launch configuration the benchmark times."""
import numpy as np
import pytest
import torch

import tlr_synth as S
from oracle import route_oracle as O
from tests.parity import check_against_oracle, check_self_consistency, run_gpu

pytestmark = pytest.mark.gpu


class Head:
    """W on the host (bits + fp64) and on the device, built once per (d, V)."""
    _cache = {}

    @classmethod
    def get(cls, d, V):
        key = (d, V)
        if key not in cls._cache:
            cls._cache.clear()                      # one head at a time: the fp64 copy is 1-2 GB
            W = S.make_W(d, V, seed=0)
            cls._cache[key] = (W, O.bf16_bits_to_f64(S.bf16_bits(W)), W.cuda())
        return cls._cache[key]


def oracle_rows(hid, W, W64, tau, rows=None):
    hb = S.bf16_bits(hid.h)
    if rows is not None:
        hb = hb[rows]
    return O.route_oracle(hb, S.bf16_bits(W), tau, W64=W64)


def test_config_decode16_percentile_tau(pkg):
    wl = S.WORKLOADS["decode16"]
    W, W64, Wd = Head.get(wl.d, wl.V)
    hid = S.make_h(wl.n, wl.d, seed=0)
    first = oracle_rows(hid, W, W64, 0.5)
    tau = O.percentile_tau(first.conf, 0.07)
    ref = O.with_threshold(first, tau)
    assert ref.routed_count == 1
    gpu = run_gpu(pkg, Wd, hid.h, tau)
    assert gpu["status"] == 0 and gpu["plan"].path == 2
    check_self_consistency(gpu, tau, wl.V)
    rep = check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(hid.h)), W64)
    assert rep["route_exempt_rows"] == 0
    assert gpu["routed_count"] == 1 and gpu["routed_idx"][0] == ref.routed_idx[0]


def test_config_decode256(pkg):
    wl = S.WORKLOADS["decode256"]
    W, W64, Wd = Head.get(wl.d, wl.V)
    hid = S.make_h(wl.n, wl.d, seed=0)
    ref = oracle_rows(hid, W, W64, wl.tau)
    gpu = run_gpu(pkg, Wd, hid.h, wl.tau)
    assert gpu["status"] == 0 and gpu["plan"].path == 2
    check_self_consistency(gpu, wl.tau, wl.V)
    check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(hid.h)), W64)
    assert gpu["routed_count"] == 256 and np.array_equal(gpu["routed_idx"], np.arange(256))


def test_config_prefill8192_planted(pkg):
    wl = S.WORKLOADS["prefill8192"]
    W, W64, Wd = Head.get(wl.d, wl.V)
    hid = S.make_h(wl.n, wl.d, seed=0, W=W, planted_fraction=wl.planted_fraction)
    gpu = run_gpu(pkg, Wd, hid.h, wl.tau)
    assert gpu["status"] == 0 and gpu["plan"].path == 2
    check_self_consistency(gpu, wl.tau, wl.V)
    # every one of the 8192 rows against the oracle (about half a minute of host time)
    others = np.setdiff1d(np.arange(wl.n), hid.planted_rows)
    ref = oracle_rows(hid, W, W64, wl.tau)
    rep = check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(hid.h)), W64)
    assert rep["route_exempt_rows"] == 0              # confidences are ~1e-4 or ~0.997, nowhere near 0.5
    assert gpu["routed_count"] == ref.routed_count
    assert np.array_equal(gpu["routed_idx"][:ref.routed_count], ref.routed_idx)
    # planted rows keep the small model's token; everything else is routed: 8192 - 409 = 7783
    assert np.array_equal(gpu["token"][hid.planted_rows], hid.planted_tokens)
    assert gpu["routed_count"] == wl.n - hid.planted_rows.size == 7783
    assert np.array_equal(gpu["routed_idx"][:7783], others.astype(np.int32))


def test_config_head1p5b_percentile_tau(pkg):
    wl = S.WORKLOADS["head1p5b"]
    W, W64, Wd = Head.get(wl.d, wl.V)
    hid = S.make_h(wl.n, wl.d, seed=0)
    first = oracle_rows(hid, W, W64, 0.5)                    # all 4096 rows: tau needs every confidence
    tau = O.percentile_tau(first.conf, 0.07)
    ref = O.with_threshold(first, tau)
    assert ref.routed_count == 286
    gpu = run_gpu(pkg, Wd, hid.h, tau)
    assert gpu["status"] == 0 and gpu["plan"].path == 2
    check_self_consistency(gpu, tau, wl.V)
    rep = check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(hid.h)), W64)
    if rep["route_exempt_rows"] == 0:
        assert gpu["routed_count"] == 286 and np.array_equal(gpu["routed_idx"][:286], ref.routed_idx)


@pytest.mark.parametrize("n", S.SWEEP_N)
def test_config_sweep(pkg, n):
    wl = S.WORKLOADS["sweep%d" % n]
    W, W64, Wd = Head.get(wl.d, wl.V)
    hid = S.make_h(n, wl.d, seed=0)
    h64 = O.bf16_bits_to_f64(S.bf16_bits(hid.h))
    scores = oracle_rows(hid, W, W64, S.SWEEP_TAU[0])          # all n rows, also at n = 4096 and 16384
    for tau in S.SWEEP_TAU:
        gpu = run_gpu(pkg, Wd, hid.h, tau, max_n=n)
        assert gpu["status"] == 0 and gpu["plan"].path == 2
        check_self_consistency(gpu, tau, wl.V)
        assert gpu["routed_count"] == n and np.array_equal(gpu["routed_idx"], np.arange(n))   # conf ~1e-4 << tau
        check_against_oracle(O.with_threshold(scores, tau), gpu, h64, W64)


@pytest.mark.parametrize("sizes,calls", [([256, 16, 256, 200], 48), ([2400, 1100, 4096, 3000], 10)])
def test_host_calls_in_flight_at_full_size(pkg, sizes, calls):
    """Batches through submit / collect with two calls in flight: the transfer of the next call's h (a copy kernel
    for decode batches, the copy engine on the context's own stream for batches of several MB) overlaps the kernels
    of the call before it, so every collected result must still belong to ITS batch.  Four different batches go
    round; each collected result is compared bit for bit with the device-buffer call on the same batch, and two
    of the batches with the oracle."""
    wl = S.WORKLOADS["decode256"]
    W, W64, Wd = Head.get(wl.d, wl.V)
    hs = [S.make_h(n, wl.d, seed=40 + i).h for i, n in enumerate(sizes)]
    pinned = [h.pin_memory() for h in hs]
    m = max(sizes)
    want = [run_gpu(pkg, Wd, h, wl.tau, max_n=m) for h in hs]
    for i in (0, 1):
        ref = O.route_oracle(S.bf16_bits(hs[i]), S.bf16_bits(W), wl.tau, W64=W64)
        check_against_oracle(ref, want[i], O.bf16_bits_to_f64(S.bf16_bits(hs[i])), W64)
    ctx = pkg.tlr_create(wl.d, wl.V, Wd, m)
    outs = [(torch.empty(m, dtype=torch.int32).pin_memory(), torch.empty(m).pin_memory(), torch.empty(m).pin_memory(),
             torch.empty(m, dtype=torch.uint8).pin_memory(), torch.full((m,), -1, dtype=torch.int32).pin_memory(),
             torch.full((1,), -9, dtype=torch.int32).pin_memory()) for _ in range(2)]

    def check(i, o):
        k, n = i % len(sizes), sizes[i % len(sizes)]
        w = want[k]
        c = int(o[5].item())
        assert c == w["routed_count"]
        assert np.array_equal(o[0].numpy()[:n], w["token"]) and np.array_equal(o[3].numpy()[:n], w["route_mask"])
        assert np.array_equal(o[1].numpy()[:n], w["conf"]) and np.array_equal(o[2].numpy()[:n], w["entropy"])
        assert np.array_equal(o[4].numpy()[:c], w["routed_idx"][:c])

    pkg.tlr_route_host_submit(ctx, pinned[0], sizes[0], wl.tau)
    for i in range(1, calls):
        pkg.tlr_route_host_submit(ctx, pinned[i % len(sizes)], sizes[i % len(sizes)], wl.tau)
        o = outs[i & 1]
        pkg.tlr_route_host_collect(ctx, *o)
        check(i - 1, o)
    o = outs[0]
    pkg.tlr_route_host_collect(ctx, *o)
    check(calls - 1, o)
    assert pkg.tlr_last_device_status(ctx) == 0
    pkg.tlr_destroy(ctx)

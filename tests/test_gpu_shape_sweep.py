"""GPU parity on seeded random shapes: every row against the CPU fp64 oracle, bf16 head and 8-bit head.

The fixed lists of the other parity tests were chosen by hand around the switches of the planner (64 / 128 / 256
rows, 16 / 32 / 64 rows per part on the 8-bit head, one CTA or a pair per worker, tiles of 16..256 vocabulary
rows); this file draws shapes nobody chose: plain calls on both heads, the learned router, the decision variants, the
fused vocabulary-sharded step.  TLR_SWEEP_CASES widens the sweep (default 40 + 16 + 12 + 10 + 10 cases).
"""
import os

import numpy as np
import pytest
import torch

import tlr_synth as S
from oracle import route_oracle as O
from tests.parity import check_against_oracle, check_self_consistency, run_gpu
from tests.test_gpu_fp8 import planted_h, run_fp8

pytestmark = pytest.mark.gpu

CASES = int(os.environ.get("TLR_SWEEP_CASES", "40"))


def draw_shapes(count, seed, n_max, d_step):
    """Log-uniform n, d and V with the oracle's work (n * d * V) bounded."""
    rng = np.random.default_rng(seed)
    shapes = []
    while len(shapes) < count:
        n = int(round(np.exp(rng.uniform(0.0, np.log(n_max)))))
        d = d_step * int(round(np.exp(rng.uniform(np.log(1), np.log(2048 // d_step)))))
        V = int(round(np.exp(rng.uniform(np.log(2), np.log(120000)))))
        if n * d * V > 1.2e9:
            continue
        shapes.append((n, d, V))
    return shapes


@pytest.mark.parametrize("n,d,V", draw_shapes(CASES, seed=2025, n_max=900, d_step=8))
def test_bf16_head_on_a_drawn_shape(pkg, n, d, V):
    W = S.make_W(d, V, seed=n + d + V, std=0.1)
    hid = S.make_h(n, d, seed=n + d + V, W=W, planted_fraction=0.1 if n >= 16 else 0.0)
    first = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    tau = O.percentile_tau(first.conf, 0.5) if n > 1 else 0.5
    ref = O.with_threshold(first, tau)
    gpu = run_gpu(pkg, W.cuda(), hid.h, tau)
    assert gpu["status"] == 0 and gpu["plan"].path == 2
    check_self_consistency(gpu, tau, V)
    rep = check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(hid.h)), O.bf16_bits_to_f64(S.bf16_bits(W)))
    if rep["route_exempt_rows"] == 0:
        assert gpu["routed_count"] == ref.routed_count
        assert np.array_equal(gpu["routed_idx"][:ref.routed_count], ref.routed_idx)


@pytest.mark.parametrize("n,d,V", draw_shapes(max(1, (CASES * 2) // 5), seed=77, n_max=128, d_step=16))
def test_8bit_head_on_a_drawn_shape(pkg, n, d, V):
    codes, scale = S.make_W8(d, V, seed=n + d + V, std=0.1)
    W64 = O.dequantize_e4m3(codes.numpy(), scale.numpy())
    h = planted_h(n, d, W64, seed=n + d + V)
    first = O.route_oracle(S.bf16_bits(h), None, 0.5, W64=W64)
    tau = O.percentile_tau(first.conf, 0.5) if n > 1 else 0.5
    ref = O.with_threshold(first, tau)
    gpu = run_fp8(pkg, codes, scale, h, tau)
    assert gpu["status"] == 0
    check_self_consistency(gpu, tau, V)
    rep = check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(h)), W64)
    if rep["route_exempt_rows"] == 0:
        assert gpu["routed_count"] == ref.routed_count
        assert np.array_equal(gpu["routed_idx"][:ref.routed_count], ref.routed_idx)


def draw_router_shapes(count, seed):
    rng = np.random.default_rng(seed)
    shapes = []
    while len(shapes) < count:
        n = int(round(np.exp(rng.uniform(np.log(2), np.log(900)))))
        d = 8 * int(round(np.exp(rng.uniform(np.log(1), np.log(160)))))
        dh = int(round(np.exp(rng.uniform(np.log(1), np.log(700)))))
        V = int(round(np.exp(rng.uniform(np.log(2), np.log(60000)))))
        if n * d * (V + dh) > 1.0e9:
            continue
        shapes.append((n, d, dh, V))
    return shapes


@pytest.mark.parametrize("n,d,dh,V", draw_router_shapes(max(1, (CASES * 3) // 10), seed=11))
def test_learned_router_inside_the_launch_on_a_drawn_shape(pkg, n, d, dh, V):
    W = S.make_W(d, V, seed=n + V, std=0.1)
    hid = S.make_h(n, d, seed=n + dh)
    g = torch.Generator().manual_seed(dh + d)
    W1 = (torch.randn(dh, d, generator=g) / d ** 0.5).to(torch.bfloat16)
    b1 = torch.randn(dh, generator=g) * 0.1
    w2 = torch.randn(dh, generator=g) * 0.5
    b2 = -0.1
    ref_score = O.mlp_router_score(S.bf16_bits(hid.h), S.bf16_bits(W1), b1.numpy(), w2.numpy(), b2)
    base = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    tau = float(np.median(ref_score))
    want = O.route_decision(ref_score, tau)
    r = pkg.Router(W.cuda(), max_n=n)
    r.set_router_mlp(W1.cuda(), b1.cuda(), w2.cuda(), b2)
    scores = torch.full((n,), float("nan"), device="cuda")
    r.route(hid.h.cuda(), tau, score_source=pkg.TLR_SCORE_MLP, mlp_score=scores)
    torch.cuda.synchronize()
    assert pkg.tlr_last_device_status(r.ctx) == 0
    got = scores.cpu().numpy()
    assert np.max(np.abs(got - ref_score)) <= 1e-3
    mask = r.route_mask[:n].cpu().numpy()
    near = np.abs(ref_score - tau) <= 1e-3
    assert np.array_equal(mask[~near], want[0][~near])
    assert np.array_equal(mask == 1, got < np.float32(tau))
    c = int(r.routed_count.item())
    assert c == int(mask.sum()) and np.array_equal(r.routed_idx[:c].cpu().numpy(), np.flatnonzero(mask))
    sure = base.top2_gap >= 1e-3
    assert np.array_equal(r.token[:n].cpu().numpy()[sure], base.token[sure])
    assert np.max(np.abs(r.conf[:n].cpu().numpy() - base.conf) / base.conf) <= 1e-3
    assert np.max(np.abs(r.entropy[:n].cpu().numpy() - base.entropy)) <= 1e-3
    r.close()


def draw_variant_shapes(count, seed):
    rng = np.random.default_rng(seed)
    shapes = []
    while len(shapes) < count:
        seq_len = int(round(np.exp(rng.uniform(0.0, np.log(300)))))
        seqs = int(round(np.exp(rng.uniform(0.0, np.log(40)))))
        d = 8 * int(round(np.exp(rng.uniform(np.log(2), np.log(64)))))
        V = int(round(np.exp(rng.uniform(np.log(50), np.log(30000)))))
        if seq_len * seqs > 5000 or seq_len * seqs * d * V > 1.0e9:
            continue
        shapes.append((seqs, seq_len, d, V))
    return shapes


@pytest.mark.parametrize("seqs,seq_len,d,V", draw_variant_shapes(max(1, CASES // 4), seed=5))
def test_decision_variants_on_a_drawn_shape(pkg, seqs, seq_len, d, V):
    """Per-row thresholds, both polarities and the first routed position of every sequence."""
    from tests.test_gpu_variants import run_ex
    n = seqs * seq_len
    W = S.make_W(d, V, seed=n + V, std=0.12)
    hid = S.make_h(n, d, seed=n + d, W=W, planted_fraction=0.3 if n >= 4 else 0.0)
    base = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    Wd = W.cuda()
    rng = np.random.default_rng(n + V)
    tau_rows = rng.choice(np.array([0.0, 0.01, 0.3, 0.999, 1.0], dtype=np.float32), size=n)
    for above in (False, True):
        ref = O.with_threshold(base, tau_rows, route_above=above)
        clear = np.abs(base.conf - tau_rows) > 1e-3 * tau_rows          # rows whose decision no rounding can flip
        g = run_ex(pkg, Wd, hid.h, 0.77, tau_rows=tau_rows, route_above=above, seq_len=seq_len)
        assert np.array_equal(g["route_mask"][clear], ref.route_mask[clear])
        own = (g["conf"] > tau_rows) if above else (g["conf"] < tau_rows)
        assert np.array_equal(g["route_mask"] == 1, own)
        c = g["routed_count"]
        assert c == int(g["route_mask"].sum())
        assert np.array_equal(g["routed_idx"][:c], np.flatnonzero(g["route_mask"]).astype(np.int32))
        assert np.array_equal(g["first"], O.first_routed(g["route_mask"], seq_len))
        if clear.all():
            assert c == ref.routed_count and np.array_equal(g["routed_idx"][:c], ref.routed_idx)


def draw_shard_shapes(count, seed):
    rng = np.random.default_rng(seed)
    shapes = []
    while len(shapes) < count:
        n = int(round(np.exp(rng.uniform(0.0, np.log(300)))))
        d = 8 * int(round(np.exp(rng.uniform(np.log(2), np.log(128)))))
        shards = int(rng.integers(2, 9))
        V = int(round(np.exp(rng.uniform(np.log(32 * shards + 1), np.log(60000)))))
        if n * d * V > 8.0e8:
            continue
        shapes.append((n, d, V, shards))
    return shapes


@pytest.mark.parametrize("n,d,V,shards", draw_shard_shapes(max(1, CASES // 4), seed=9))
def test_fused_sharded_step_on_a_drawn_shape(pkg, n, d, V, shards):
    """The vocabulary cut into 2..8 shards, exchange fused into the kernels (ranks one after the other on one GPU)."""
    from tests.test_gpu_sharded_fused import make_ranks, outputs, poison
    W = S.make_W(d, V, seed=n + V, std=0.1)
    Wd = W.cuda()
    W64 = O.bf16_bits_to_f64(S.bf16_bits(W))
    ranks, block = make_ranks(pkg, Wd, n, shards)
    reader = ranks[(n + V) % shards]
    hid = S.make_h(n, d, seed=n + d, W=W, planted_fraction=0.1 if n >= 16 else 0.0)
    first = O.route_oracle(S.bf16_bits(hid.h), None, 0.5, W64=W64)
    tau = O.percentile_tau(first.conf, 0.5) if n > 1 else 0.5
    ref = O.with_threshold(first, tau)
    h = hid.h.cuda()
    for r in ranks:
        r.push(h)
    poison(reader)
    reader.finish(n, tau)
    torch.cuda.synchronize()
    for r in ranks:
        assert pkg.tlr_last_device_status(r.ctx) == 0
    gpu = outputs(reader, n)
    check_self_consistency(gpu, tau, V)
    rep = check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(hid.h)), W64)
    if rep["route_exempt_rows"] == 0:
        assert gpu["routed_count"] == ref.routed_count
        assert np.array_equal(gpu["routed_idx"][:ref.routed_count], ref.routed_idx)
    for r in ranks:
        r.close()

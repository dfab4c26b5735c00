"""GPU parity on seeded random shapes: every row against the CPU fp64 oracle, bf16 head and 8-bit head.

The fixed lists of the other parity tests were chosen by hand around the switches of the planner (64 / 128 / 256
rows, 16 / 32 / 64 rows per part on the 8-bit head, one CTA or a pair per worker, tiles of 16..256 vocabulary
rows); this file draws shapes nobody chose.  TLR_SWEEP_CASES widens the sweep (default 40 + 16 cases).
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


@pytest.mark.parametrize("n,d,V", draw_shapes(max(1, (CASES * 2) // 5), seed=77, n_max=64, d_step=16))
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

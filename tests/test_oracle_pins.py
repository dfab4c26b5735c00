"""Pins for the CPU oracle: everything here is fixed by the paper or by mathematics,
never by the oracle's own output and never by the CUDA path."""
import math
import os

import numpy as np
import pytest
import torch

import tlr_synth as S
from oracle import route_oracle as O


def bits_of(values):
    return S.bf16_bits(S.bf16_from_values(values))


# ---------------------------------------------------------------- widening
def test_bf16_widening_known_patterns():
    bits = np.array([0x3F80, 0xC000, 0x0000, 0x8000, 0x3DCD, 0x4049, 0x7F80], dtype=np.uint16)
    got = O.bf16_bits_to_f64(bits)
    assert got[0] == 1.0 and got[1] == -2.0 and got[2] == 0.0
    assert got[3] == 0.0 and math.copysign(1.0, got[3]) == -1.0
    assert got[4] == 0.10009765625          # 0x3DCD = 1.6015625 * 2^-4
    assert got[5] == 3.140625               # 0x4049 = 1.5703125 * 2
    assert math.isinf(got[6])


# ---------------------------------------------------------------- logits, hand-worked
def test_logits_hand_worked_nonsquare():
    # n=2, d=3, V=4: small integers, exact in bf16 and in fp64; numbers worked by hand.
    h = [[1, 2, -1], [0, 3, 2]]
    W = [[1, 0, 0], [0, 1, 0], [1, 1, 1], [2, -1, 0]]
    z = O.logits_fp64(O.bf16_bits_to_f64(bits_of(h)), O.bf16_bits_to_f64(bits_of(W)))
    assert z.shape == (2, 4)
    assert z.tolist() == [[1.0, 2.0, 2.0, 0.0], [0.0, 3.0, 5.0, -3.0]]
    r = O.route_oracle(bits_of(h), bits_of(W), 0.5)
    # row 0 has an exact tie between tokens 1 and 2: the lower index wins, gap 0
    assert r.token.tolist() == [1, 2]
    assert r.top2_gap.tolist() == [0.0, 2.0]
    # row 0: p = (e^-1, 1, 1, e^-2)/(2 + e^-1 + e^-2)
    s0 = 2 + math.exp(-1) + math.exp(-2)
    assert r.conf[0] == pytest.approx(1 / s0, rel=1e-14)
    s1 = 1 + math.exp(-2) + math.exp(-5) + math.exp(-8)
    assert r.conf[1] == pytest.approx(1 / s1, rel=1e-14)
    assert r.route_mask.tolist() == [1, 0]          # 0.399 < 0.5 <= 0.876
    assert r.routed_idx.tolist() == [0] and r.routed_count == 1


def test_textbook_softmax_1_2_3(golden_dir):
    with open(os.path.join(golden_dir, "softmax_1_2_3.txt")) as f:
        row = [l for l in f if not l.startswith("#")][0].split()
    p0, p1, p2, H = map(float, row)
    # logits (1,2,3) from d=1: h = [1], W = [[1],[2],[3]]
    r = O.route_oracle(bits_of([[1]]), bits_of([[1], [2], [3]]), 0.7)
    assert r.token[0] == 2
    assert r.conf[0] == pytest.approx(p2, abs=2e-10)
    assert r.entropy[0] == pytest.approx(H, abs=2e-9)
    assert r.route_mask[0] == 1                        # 0.665 < 0.7
    # reversed vocabulary order: same numbers, token index 0
    r = O.route_oracle(bits_of([[1]]), bits_of([[3], [2], [1]]), 0.6)
    assert r.token[0] == 0 and r.route_mask[0] == 0
    assert r.conf[0] == pytest.approx(p2, abs=2e-10)


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("V", [2, 7, 1000])
def test_all_equal_logits(V):
    # h = 0 gives z = 0 for every token: uniform distribution
    r = O.route_oracle(bits_of([[0, 0]]), bits_of([[1, -1]] * V), 0.5)
    assert r.token[0] == 0
    assert r.conf[0] == pytest.approx(1.0 / V, rel=1e-14)
    assert r.entropy[0] == pytest.approx(math.log(V), rel=1e-13)
    assert r.top2_gap[0] == 0.0


@pytest.mark.parametrize("a,V,pos", [(4.0, 5, 0), (2.0, 64, 63), (16.0, 300, 17), (0.5, 3, 1)])
def test_one_high_logit_closed_form(a, V, pos):
    # one token has logit a, the other V-1 have 0:
    #   conf = e^a / (e^a + V - 1),  H = ln(e^a + V - 1) - a e^a / (e^a + V - 1)
    W = [[0.0]] * V
    W = [list(w) for w in W]
    W[pos] = [a]
    r = O.route_oracle(bits_of([[1]]), bits_of(W), 0.5)
    ea = math.exp(a)
    assert r.token[0] == pos
    assert r.conf[0] == pytest.approx(ea / (ea + V - 1), rel=1e-13)
    assert r.entropy[0] == pytest.approx(math.log(ea + V - 1) - a * ea / (ea + V - 1), rel=1e-11, abs=1e-14)
    assert r.top2_gap[0] == a


def test_saturated_row_zero_times_log_zero():
    # logit gap of 2000: every other probability underflows to exactly 0; H must be 0, not NaN
    r = O.route_oracle(bits_of([[1]]), bits_of([[0], [2000], [0]]), 1.0)
    assert r.token[0] == 1 and r.conf[0] == 1.0 and r.entropy[0] == 0.0
    assert r.route_mask[0] == 0      # conf == 1 is not strictly below tau = 1


# ---------------------------------------------------------------- library and brute force
def test_against_library_softmax_and_entropy():
    g = torch.Generator().manual_seed(5)
    h = (torch.randn(9, 24, generator=g) * 1.5).to(torch.bfloat16)
    W = (torch.randn(301, 24, generator=g)).to(torch.bfloat16)
    r = O.route_oracle(S.bf16_bits(h), S.bf16_bits(W), 0.3)
    z = h.double() @ W.double().t()
    p = torch.softmax(z, dim=1)
    np.testing.assert_array_equal(r.token, torch.argmax(z, dim=1).numpy())
    np.testing.assert_allclose(r.conf, p.max(dim=1).values.numpy(), rtol=1e-12)
    np.testing.assert_allclose(r.entropy, torch.distributions.Categorical(probs=p).entropy().numpy(), rtol=1e-10)
    top2 = torch.topk(z, 2, dim=1).values
    np.testing.assert_allclose(r.top2_gap, (top2[:, 0] - top2[:, 1]).numpy(), rtol=1e-12, atol=1e-14)


def test_against_pure_python_bruteforce():
    g = torch.Generator().manual_seed(11)
    h = torch.randn(5, 4, generator=g).to(torch.bfloat16)
    W = torch.randn(8, 4, generator=g).to(torch.bfloat16)
    tau = 0.5
    r = O.route_oracle(S.bf16_bits(h), S.bf16_bits(W), tau)
    rows, routed = O.route_bruteforce(h.double().tolist(), W.double().tolist(), tau)
    for i, (tok, conf, H, flag) in enumerate(rows):
        assert r.token[i] == tok
        assert r.conf[i] == pytest.approx(conf, rel=1e-13)
        assert r.entropy[i] == pytest.approx(H, rel=1e-12)
        assert r.route_mask[i] == flag
    assert r.routed_idx.tolist() == routed
    assert 0 < len(routed) < 5       # the case exercises both outcomes


def test_bruteforce_itself_on_hand_case():
    rows, routed = O.route_bruteforce([[1.0]], [[1.0], [2.0], [3.0]], 0.7)
    assert rows[0][0] == 2 and rows[0][1] == pytest.approx(0.6652409558, abs=1e-9) and routed == [0]


# ---------------------------------------------------------------- invariants
def _random_case(n=40, d=16, V=257, seed=3, scale=2.0):
    g = torch.Generator().manual_seed(seed)
    h = (torch.randn(n, d, generator=g) * scale).to(torch.bfloat16)
    W = torch.randn(V, d, generator=g).to(torch.bfloat16)
    return S.bf16_bits(h), S.bf16_bits(W)


def test_invariants_and_threshold_extremes():
    hb, Wb = _random_case()
    V = Wb.shape[0]
    r0 = O.route_oracle(hb, Wb, 0.0)
    r1 = O.route_oracle(hb, Wb, 1.0)
    assert r0.routed_count == 0 and r0.route_mask.sum() == 0 and r0.routed_idx.size == 0   # "small_only": nothing routed
    assert r1.routed_count == hb.shape[0] and r1.routed_idx.tolist() == list(range(hb.shape[0]))
    assert np.all(r0.conf >= 1.0 / V - 1e-15) and np.all(r0.conf <= 1.0)
    assert np.all(r0.entropy >= 0.0) and np.all(r0.entropy <= math.log(V) + 1e-12)
    # confidence is the largest probability, so H >= -ln(conf) ... and H <= ln V
    assert np.all(r0.entropy >= -np.log(r0.conf) * r0.conf - 1e-12)
    for tau in (0.05, 0.2, 0.5, 0.8):
        r = O.route_oracle(hb, Wb, tau)
        assert r.routed_count == int(r.route_mask.sum()) == r.routed_idx.size
        assert np.all(np.diff(r.routed_idx) > 0)
        assert np.all(r.route_mask[r.routed_idx] == 1)
        assert np.array_equal(r.route_mask == 1, r.conf < float(np.float32(tau)))


def test_count_monotone_in_threshold_like_table1(golden_dir):
    taus, counts = [], []
    with open(os.path.join(golden_dir, "table1_routing_number.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            t, c = line.split()
            taus.append(float(t)); counts.append(int(c))
    assert counts == sorted(counts)                  # what the paper's table shows
    hb, Wb = _random_case(n=64, scale=3.0, seed=8)
    ours = [O.route_oracle(hb, Wb, t).routed_count for t in taus]
    assert ours == sorted(ours) and ours[0] < ours[-1]
    # and the routed sets are nested
    prev = set()
    for t in taus:
        cur = set(O.route_oracle(hb, Wb, t).routed_idx.tolist())
        assert prev <= cur
        prev = cur


def test_row_permutation_equivariance_and_block_size_irrelevance():
    hb, Wb = _random_case(n=37)
    perm = np.random.default_rng(0).permutation(37)
    a = O.route_oracle(hb, Wb, 0.3, row_block=128)
    b = O.route_oracle(hb[perm], Wb, 0.3, row_block=5)
    np.testing.assert_array_equal(a.token[perm], b.token)
    np.testing.assert_array_equal(a.conf[perm], b.conf)
    np.testing.assert_array_equal(a.entropy[perm], b.entropy)
    np.testing.assert_array_equal(a.route_mask[perm], b.route_mask)


def test_vocab_permutation_moves_the_token_only():
    hb, Wb = _random_case(n=12, V=100)
    perm = np.random.default_rng(1).permutation(100)
    a = O.route_oracle(hb, Wb, 0.3)
    b = O.route_oracle(hb, Wb[perm], 0.3)
    np.testing.assert_array_equal(perm[b.token], a.token)
    np.testing.assert_allclose(a.conf, b.conf, rtol=1e-13)
    np.testing.assert_allclose(a.entropy, b.entropy, rtol=1e-12)


def test_duplicate_embedding_rows_tie_to_lower_index():
    hb, Wb = _random_case(n=6, V=50)
    a = O.route_oracle(hb, Wb, 0.3)
    W2 = np.concatenate([Wb, Wb], axis=0)            # every logit appears twice
    b = O.route_oracle(hb, W2, 0.3)
    np.testing.assert_array_equal(a.token, b.token)  # the copy at index v+50 must lose
    np.testing.assert_allclose(b.conf, a.conf / 2, rtol=1e-13)
    np.testing.assert_allclose(b.entropy, a.entropy + math.log(2), rtol=1e-12)
    assert np.all(b.top2_gap == 0.0)


def test_non_finite_row_is_routed():
    h = S.bf16_from_values([[1.0, 0.0], [1.0, 1.0]]).clone()
    h[0, 0] = float("nan")
    W = S.bf16_from_values([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])
    with np.errstate(invalid="ignore"):
        r = O.route_oracle(S.bf16_bits(h), S.bf16_bits(W), 0.0)
    assert r.route_mask.tolist() == [1, 0] and r.routed_idx.tolist() == [0]


def test_percentile_tau_routes_exactly_k():
    conf = np.random.default_rng(2).uniform(1e-5, 2e-4, size=4096)
    tau = O.percentile_tau(conf)
    assert int((conf < tau).sum()) == 286            # floor(0.07 * 4096)
    assert O.percentile_tau(np.array([0.3, 0.1, 0.2]) ) == pytest.approx(0.15, rel=1e-6)   # k = max(1, 0)


# ---------------------------------------------------------------- the synthetic workload's closed forms
@pytest.fixture(scope="module")
def head():
    d, V = 896, 151936
    W = S.make_W(d, V, seed=0)
    return d, V, W, O.bf16_bits_to_f64(S.bf16_bits(W))


def test_workload_distribution_closed_forms(head):
    d, V, W, W64 = head
    H = S.make_h(24, d, seed=0)
    hb = S.bf16_bits(H.h)
    # unit RMS after rounding
    rms = np.sqrt((O.bf16_bits_to_f64(hb) ** 2).mean(axis=1))
    assert np.all(np.abs(rms - 1.0) < 2e-3)
    z = O.logits_fp64(O.bf16_bits_to_f64(hb), W64)
    sigma = 0.02 * math.sqrt(d)                          # logits are N(0, 0.02^2 d) for unit-RMS h
    assert abs(z.std() - sigma) < 0.01 * sigma           # a transposed or unnormalised operand fails this
    r = O.route_oracle(hb, S.bf16_bits(W), 0.5, W64=W64)
    # log-normal sum: E[H] = ln V - sigma^2/2 up to O(1/sqrt(V)) fluctuations
    assert abs(r.entropy.mean() - (math.log(V) - sigma * sigma / 2)) < 5e-3
    assert r.routed_count == 24                          # base confidences are ~1e-4, far below 0.5
    assert np.all(r.conf < 1e-3) and np.all(r.conf > 1.0 / V)


def test_workload_planted_rows(head):
    d, V, W, W64 = head
    n = 60
    H = S.make_h(n, d, seed=0, W=W, planted_fraction=0.05)
    assert H.planted_rows.size == 3 and len(set(H.planted_rows.tolist())) == 3
    r = O.route_oracle(S.bf16_bits(H.h), S.bf16_bits(W), 0.5, W64=W64)
    np.testing.assert_array_equal(r.token[H.planted_rows], H.planted_tokens)
    assert np.all(r.conf[H.planted_rows] > 0.9) and np.all(r.entropy[H.planted_rows] < 0.5)
    assert r.routed_count == n - 3
    assert set(r.routed_idx.tolist()) == set(range(n)) - set(H.planted_rows.tolist())


def test_generators_are_seeded_and_independent_of_n():
    a = S.make_W(8, 100, seed=0); b = S.make_W(8, 100, seed=0); c = S.make_W(8, 100, seed=1)
    assert torch.equal(a, b) and not torch.equal(a, c)
    h1 = S.make_h(4, 8, seed=0).h; h2 = S.make_h(4, 8, seed=0).h
    assert torch.equal(h1, h2)
    assert S.make_h(0, 8).h.shape == (0, 8)


# ---------------------------------------------------------------- variants of the decision
def test_polarity_and_per_row_threshold():
    conf = np.array([0.1, 0.5, 0.5000001, 0.9, np.nan])
    below = O.route_decision(conf, 0.5)[0]
    above = O.route_decision(conf, 0.5, route_above=True)[0]
    assert below.tolist() == [1, 0, 0, 0, 1]         # strict: 0.5 is not below 0.5; NaN is routed
    assert above.tolist() == [0, 0, 1, 1, 1]         # strict: 0.5 is not above 0.5; NaN is routed
    # away from equality and NaN the two polarities are complements
    hb, Wb = _random_case(n=50, seed=4)
    r = O.route_oracle(hb, Wb, 0.2)
    up = O.with_threshold(r, 0.2, route_above=True)
    assert np.array_equal(up.route_mask, 1 - r.route_mask)
    # a constant vector is the scalar; a vector applies row by row
    vec = O.route_decision(conf[:4], np.array([0.05, 0.6, 0.4, 0.95]))[0]
    assert vec.tolist() == [0, 1, 0, 1]
    assert np.array_equal(O.route_decision(r.conf, np.full(50, 0.2))[0], r.route_mask)


def test_first_routed_position_per_sequence():
    mask = np.array([0, 0, 1, 1,   0, 0, 0, 0,   1, 0, 0, 1,   0, 0, 0, 1], dtype=np.uint8)
    assert O.first_routed(mask, 4).tolist() == [2, 4, 0, 3]         # worked by hand; 4 = none routed
    assert O.first_routed(mask, 16).tolist() == [2]
    assert O.first_routed(mask, 1).tolist() == (1 - mask).tolist()  # length-1 sequences: 0 if routed else 1
    # equals the minimum of the segment's entries of the compacted index list
    rng = np.random.default_rng(3)
    m = (rng.random(60) < 0.1).astype(np.uint8)
    idx = np.flatnonzero(m)
    for b, f in enumerate(O.first_routed(m, 12)):
        seg = idx[(idx >= 12 * b) & (idx < 12 * (b + 1))]
        assert f == (seg.min() - 12 * b if seg.size else 12)
    with pytest.raises(ValueError):
        O.first_routed(mask, 5)


# ---------------------------------------------------------------- learned router score (shape assumed, not the paper's)
def test_mlp_router_score_closed_forms_and_library():
    h = bits_of([[1, 2], [-1, 0], [0, 0]])
    W1 = bits_of([[1, 0], [0, 1], [-1, -1]])            # hidden = relu([h0, h1, -h0-h1] + b1)
    b1 = np.array([0.0, 0.5, 0.0], np.float32)
    w2 = np.array([1.0, -2.0, 3.0], np.float32)
    s = O.mlp_router_score(h, W1, b1, w2, 0.25)
    # row 0: hidden (1, 2.5, 0) -> 1 - 5 + 0 + .25 = -3.75; row 1: hidden (0, .5, 1) -> -1 + 3 + .25 = 2.25;
    # row 2: hidden (0, .5, 0) -> -1 + .25 = -0.75                                  (worked by hand)
    expect = [1 / (1 + math.exp(3.75)), 1 / (1 + math.exp(-2.25)), 1 / (1 + math.exp(0.75))]
    np.testing.assert_allclose(s, expect, rtol=1e-14)
    # zero output weights: sigmoid(b2) for every row
    np.testing.assert_allclose(O.mlp_router_score(h, W1, b1, np.zeros(3, np.float32), 0.0), 0.5)
    # independent library evaluation
    g = torch.Generator().manual_seed(2)
    hh = torch.randn(7, 24, generator=g).to(torch.bfloat16)
    WW = torch.randn(40, 24, generator=g).to(torch.bfloat16)
    bb = torch.randn(40, generator=g); ww = torch.randn(40, generator=g)
    lib = torch.sigmoid(torch.relu(hh.double() @ WW.double().t() + bb.double()) @ ww.double() - 0.3)
    got = O.mlp_router_score(S.bf16_bits(hh), S.bf16_bits(WW), bb.numpy(), ww.numpy(), -0.3)
    np.testing.assert_allclose(got, lib.numpy(), rtol=1e-7)    # -0.3 is rounded to fp32 inside the oracle


# ---------------------------------------------------------------- vocabulary-sharded form

def test_shard_summaries_merge_to_the_plain_definition():
    """Any contiguous partition of the vocabulary, summarised and merged, gives steps 2-4 of the
    plain definition: token exactly (also when the maximum is tied across two ranges), conf and
    entropy to rounding."""
    rng = np.random.default_rng(5)
    n, d, V = 9, 16, 211
    h = S.bf16_bits(torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32)).to(torch.bfloat16))
    Wt = torch.from_numpy((0.3 * rng.standard_normal((V, d))).astype(np.float32)).to(torch.bfloat16)
    Wt[20] = Wt[20] * 4.0                             # a long row, so that a hidden state along it peaks there
    Wt[150] = Wt[20]                                  # ... and an exact copy of it in another range: a tie
    hb = S.bf16_bits(Wt[20:21])                       # a row whose maximum is that tied pair
    h = np.concatenate([h, hb], axis=0)
    W = S.bf16_bits(Wt)
    ref = O.route_oracle(h, W, 0.5)
    for cuts in ([0, 211], [0, 100, 211], [0, 32, 64, 160, 211], [0, 1, 210, 211]):
        parts = [O.shard_summary(h, W[a:b], a) for a, b in zip(cuts[:-1], cuts[1:])]
        token, conf, ent = O.merge_summaries(parts)
        assert np.array_equal(token, ref.token)
        assert np.allclose(conf, ref.conf, rtol=1e-12, atol=0)
        assert np.allclose(ent, ref.entropy, rtol=0, atol=1e-12)
    assert ref.token[-1] == 20                        # the tie went to the lower index


def test_shard_summary_hand_worked():
    """Two ranges of a four-token vocabulary with integer logits: range A = {0, 2}, range B = {2, 1}."""
    h = S.bf16_bits(torch.tensor([[1.0, 0.0]], dtype=torch.bfloat16))
    W = S.bf16_bits(torch.tensor([[0.0, 5.0], [2.0, 1.0], [2.0, 7.0], [1.0, 3.0]], dtype=torch.bfloat16))
    mA, iA, sA, tA = O.shard_summary(h, W[0:2], 0)
    mB, iB, sB, tB = O.shard_summary(h, W[2:4], 2)
    assert mA[0] == 2.0 and iA[0] == 1 and sA[0] == pytest.approx(1 + math.exp(-2)) and tA[0] == pytest.approx(-2 * math.exp(-2))
    assert mB[0] == 2.0 and iB[0] == 2 and sB[0] == pytest.approx(1 + math.exp(-1)) and tB[0] == pytest.approx(-math.exp(-1))
    token, conf, ent = O.merge_summaries([(mA, iA, sA, tA), (mB, iB, sB, tB)])
    Ssum = 2 + math.exp(-2) + math.exp(-1)
    assert token[0] == 1 and conf[0] == pytest.approx(1 / Ssum)
    p = np.array([math.exp(-2), 1.0, 1.0, math.exp(-1)]) / Ssum
    assert ent[0] == pytest.approx(float(-(p * np.log(p)).sum()))


# ---------------------------------------------------------------- 8-bit copy of W

def test_e4m3_values_against_the_format_definition():
    """Hand-picked codes of the OCP e4m3 format, its extremes, its symmetry and its ordering."""
    v = O.e4m3_value(np.arange(256, dtype=np.uint8))
    assert v[0x00] == 0.0 and v[0x80] == 0.0
    assert v[0x01] == 2.0 ** -9 and v[0x07] == 7 * 2.0 ** -9          # subnormals
    assert v[0x08] == 2.0 ** -6                                        # smallest normal
    assert v[0x38] == 1.0 and v[0x3c] == 1.5 and v[0x40] == 2.0 and v[0xc0] == -2.0
    assert v[0x7e] == 448.0 and v[0xfe] == -448.0                      # largest finite
    assert np.isnan(v[0x7f]) and np.isnan(v[0xff])
    assert np.all(np.diff(v[:0x7f]) > 0)                               # magnitudes grow with the code
    assert np.array_equal(v[0x80:0xff], -v[0x00:0x7f])
    import torch as _t                                                  # a library's decoder of the same format
    lib = _t.arange(256, dtype=_t.uint8).view(_t.float8_e4m3fn).double().numpy()
    assert np.array_equal(np.nan_to_num(v, nan=-1.0), np.nan_to_num(lib, nan=-1.0))


def test_dequantized_head_and_generator_recipe():
    codes, scale = S.make_W8(32, 50, seed=3, std=0.02)
    W = O.dequantize_e4m3(codes.numpy(), scale.numpy())
    assert W.shape == (50, 32) and np.all(np.isfinite(W))
    assert np.allclose(np.abs(W).max(axis=1), 448.0 * scale.numpy().astype(np.float64), rtol=1e-6)   # row maximum maps to 448
    assert 0.015 < W.std() < 0.025                                     # still the N(0, 0.02^2) head
    # a hand-made head: codes 0x38 (1.0) and 0xc0 (-2.0) with scales 0.5 and 3
    hand = O.dequantize_e4m3(np.array([[0x38, 0xc0], [0x40, 0x01]], np.uint8), np.array([0.5, 3.0], np.float32))
    assert np.array_equal(hand, np.array([[0.5, -1.0], [6.0, 3.0 * 2.0 ** -9]]))

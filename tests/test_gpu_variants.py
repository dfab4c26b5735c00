"""GPU parity of tlr_route_ex: per-row thresholds, the opposite polarity, first routed position."""
import numpy as np
import pytest
import torch

import tlr_synth as S
from oracle import route_oracle as O
from tests.parity import check_against_oracle, to_np

pytestmark = pytest.mark.gpu


def run_ex(P, Wd, h_cpu, tau, tau_rows=None, route_above=False, seq_len=0):
    n = h_cpu.shape[0]
    r = P.Router(Wd, max_n=n)
    first = torch.full((max(1, n // seq_len if seq_len else 1),), -9, dtype=torch.int32, device="cuda")
    tr = None if tau_rows is None else torch.from_numpy(np.asarray(tau_rows, dtype=np.float32)).cuda()
    r.route(h_cpu.cuda(), tau, tau_per_row=tr, route_above=route_above, seq_len=seq_len,
            first_routed=first if seq_len else None)
    torch.cuda.synchronize()
    assert P.tlr_last_device_status(r.ctx) == 0
    out = {"token": to_np(r.token[:n]), "conf": to_np(r.conf[:n]), "entropy": to_np(r.entropy[:n]),
           "route_mask": to_np(r.route_mask[:n]), "routed_idx": to_np(r.routed_idx),
           "routed_count": int(r.routed_count.item()), "first": to_np(first)}
    r.close()
    return out


@pytest.mark.parametrize("n,seq_len", [(96, 8), (640, 64), (2048, 256)])   # small kernel, cluster, multi-block
def test_variants_against_oracle(pkg, n, seq_len):
    d, V = 128, 9000
    W = S.make_W(d, V, seed=7, std=0.12)
    hid = S.make_h(n, d, seed=n, W=W, planted_fraction=0.3)
    base = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    Wd = W.cuda()
    rng = np.random.default_rng(n)
    tau_rows = rng.choice(np.array([0.0, 0.01, 0.3, 0.999, 1.0], dtype=np.float32), size=n)

    # scalar tau, below (the plain rule) + first routed position
    g = run_ex(pkg, Wd, hid.h, 0.5, seq_len=seq_len)
    check_against_oracle(base, g)
    assert np.array_equal(g["route_mask"], base.route_mask)
    assert np.array_equal(g["first"], O.first_routed(base.route_mask, seq_len))
    # nothing routed anywhere: every sequence reports seq_len
    g0 = run_ex(pkg, Wd, hid.h, 0.0, seq_len=seq_len)
    assert g0["routed_count"] == 0 and np.all(g0["first"] == seq_len)

    # opposite polarity
    ref = O.with_threshold(base, 0.5, route_above=True)
    g = run_ex(pkg, Wd, hid.h, 0.5, route_above=True, seq_len=seq_len)
    assert np.array_equal(g["route_mask"], ref.route_mask)
    assert g["routed_count"] == ref.routed_count and np.array_equal(g["routed_idx"][:ref.routed_count], ref.routed_idx)
    assert np.array_equal(g["first"], O.first_routed(ref.route_mask, seq_len))
    assert np.array_equal(g["route_mask"], 1 - base.route_mask)   # complements away from equality

    # one threshold per row, both polarities
    for above in (False, True):
        ref = O.with_threshold(base, tau_rows, route_above=above)
        g = run_ex(pkg, Wd, hid.h, 0.123, tau_rows=tau_rows, route_above=above, seq_len=seq_len)
        assert np.array_equal(g["route_mask"], ref.route_mask)
        assert g["routed_count"] == ref.routed_count
        assert np.array_equal(g["routed_idx"][:ref.routed_count], ref.routed_idx)
        assert np.array_equal(g["first"], O.first_routed(ref.route_mask, seq_len))
        # the GPU decision agrees with its own confidence
        own = (g["conf"] > tau_rows) if above else (g["conf"] < tau_rows)
        assert np.array_equal(g["route_mask"] == 1, own)


def test_variant_argument_errors(pkg):
    W = S.make_W(64, 500, seed=1)
    hid = S.make_h(10, 64, seed=1)
    r = pkg.Router(W.cuda(), max_n=10)
    first = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(pkg.TlrError) as e:     # 10 rows are not a multiple of 4
        r.route(hid.h.cuda(), 0.5, seq_len=4, first_routed=first)
    assert e.value.code == 1
    with pytest.raises(pkg.TlrError) as e:     # seq_len without an output buffer
        r.route(hid.h.cuda(), 0.5, seq_len=5, first_routed=None)
    assert e.value.code == 1
    r.close()


def test_prefill_config_first_routed(pkg):
    # the prefill workload's shape: 16 sequences x 512 positions, 5% planted rows keep the small model
    wl = S.WORKLOADS["prefill8192"]
    W = S.make_W(wl.d, wl.V, seed=0)
    hid = S.make_h(wl.n, wl.d, seed=0, W=W, planted_fraction=wl.planted_fraction)
    g = run_ex(pkg, W.cuda(), hid.h, wl.tau, seq_len=512)
    planted = np.zeros(wl.n, dtype=bool)
    planted[hid.planted_rows] = True
    expect_mask = (~planted).astype(np.uint8)             # every base row is routed (conf ~1e-4), planted rows are not
    assert np.array_equal(g["route_mask"], expect_mask)
    assert np.array_equal(g["first"], O.first_routed(expect_mask, 512))
    # under the opposite polarity only the planted rows are routed
    g2 = run_ex(pkg, W.cuda(), hid.h, wl.tau, route_above=True, seq_len=512)
    assert np.array_equal(g2["route_mask"], planted.astype(np.uint8))
    assert np.array_equal(g2["first"], O.first_routed(planted.astype(np.uint8), 512))


@pytest.mark.parametrize("n,d,dh", [(50, 128, 96), (700, 896, 256), (33, 36, 300)])
def test_learned_router_score(pkg, n, d, dh):
    V = 3000
    W = S.make_W(d, V, seed=3, std=0.1)
    hid = S.make_h(n, d, seed=5)
    g = torch.Generator().manual_seed(dh)
    W1 = (torch.randn(dh, d, generator=g) / d ** 0.5).to(torch.bfloat16)
    b1 = torch.randn(dh, generator=g) * 0.1
    w2 = torch.randn(dh, generator=g) * 0.5
    b2 = 0.2
    ref_score = O.mlp_router_score(S.bf16_bits(hid.h), S.bf16_bits(W1), b1.numpy(), w2.numpy(), b2)
    base = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    tau = float(np.median(ref_score))
    want = O.route_decision(ref_score, tau)

    r = pkg.Router(W.cuda(), max_n=n)
    with pytest.raises(pkg.TlrError):                      # no router attached yet
        r.route(hid.h.cuda(), tau, score_source=pkg.TLR_SCORE_MLP)
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
    assert np.array_equal(mask == 1, got < np.float32(tau))          # decided on the learned score
    c = int(r.routed_count.item())
    assert c == int(mask.sum()) and np.array_equal(r.routed_idx[:c].cpu().numpy(), np.flatnonzero(mask))
    assert 0 < c < n
    # token / conf / entropy are still the LM head's
    assert np.array_equal(r.token[:n].cpu().numpy()[base.top2_gap >= 1e-3], base.token[base.top2_gap >= 1e-3])
    assert np.max(np.abs(r.conf[:n].cpu().numpy() - base.conf)) <= 1e-3
    # the score alone, decision still on the confidence
    r.route(hid.h.cuda(), 0.5, mlp_score=scores)
    torch.cuda.synchronize()
    assert np.array_equal(r.route_mask[:n].cpu().numpy(), base.route_mask)
    r.close()


def test_learned_router_on_the_8bit_head_and_in_a_graph(pkg):
    """Two more places the learned score must be right: on the 8-bit head (where the first layer runs in its own
    kernel, the projection kernel multiplying e4m3 operands only) and inside a captured CUDA graph (where it is part
    of the projection launch)."""
    n, d, dh, V = 40, 128, 64, 3000
    hid = S.make_h(n, d, seed=9)
    g = torch.Generator().manual_seed(7)
    W1 = (torch.randn(dh, d, generator=g) / d ** 0.5).to(torch.bfloat16)
    b1 = torch.randn(dh, generator=g) * 0.1
    w2 = torch.randn(dh, generator=g) * 0.5
    ref_score = O.mlp_router_score(S.bf16_bits(hid.h), S.bf16_bits(W1), b1.numpy(), w2.numpy(), -0.1)
    tau = float(np.median(ref_score))
    near = np.abs(ref_score - tau) <= 1e-3
    want = O.route_decision(ref_score, tau)[0]

    codes, scale = S.make_W8(d, V, seed=3, std=0.1)
    r8 = pkg.Router(codes.cuda(), max_n=n, wscale=scale.cuda())
    r8.set_router_mlp(W1.cuda(), b1.cuda(), w2.cuda(), -0.1)
    scores = torch.full((n,), float("nan"), device="cuda")
    r8.route(hid.h.cuda(), tau, score_source=pkg.TLR_SCORE_MLP, mlp_score=scores)
    torch.cuda.synchronize()
    assert pkg.tlr_last_device_status(r8.ctx) == 0
    assert np.max(np.abs(scores.cpu().numpy() - ref_score)) <= 1e-3
    assert np.array_equal(r8.route_mask[:n].cpu().numpy()[~near], want[~near])
    r8.close()

    r = pkg.Router(S.make_W(d, V, seed=3, std=0.1).cuda(), max_n=n)
    r.set_router_mlp(W1.cuda(), b1.cuda(), w2.cuda(), -0.1)
    assert pkg.tlr_plan_query(r.ctx, n).launches == 2
    buf = hid.h.cuda().clone()
    scores.fill_(float("nan"))
    r.route(buf, tau, score_source=pkg.TLR_SCORE_MLP, mlp_score=scores)          # eager first (one-time set-up)
    torch.cuda.synchronize()
    eager = (scores.cpu().numpy().copy(), r.route_mask[:n].cpu().numpy().copy(), int(r.routed_count.item()))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        r.route(buf, tau, score_source=pkg.TLR_SCORE_MLP, mlp_score=scores)
    scores.fill_(float("nan")); r.route_mask.fill_(9)
    graph.replay()
    torch.cuda.synchronize()
    assert np.array_equal(scores.cpu().numpy(), eager[0]) and np.array_equal(r.route_mask[:n].cpu().numpy(), eager[1])
    assert int(r.routed_count.item()) == eager[2]
    assert np.max(np.abs(eager[0] - ref_score)) <= 1e-3 and np.array_equal(eager[1][~near], want[~near])
    del graph
    r.close()

"""Vocabulary-sharded step on the GPU: the shards of one machine's W are processed one after the
other on the same device (sequential calls, nothing waits on anything), their summaries stacked as an
all-gather would deliver them, and the merged decision compared with the oracle and with the
unsharded call."""
import numpy as np
import pytest
import torch

import tlr_synth as S
from oracle import route_oracle as O
from tests.parity import check_against_oracle, check_self_consistency, run_gpu, to_np

pytestmark = pytest.mark.gpu


def run_sharded(P, W, h_cpu, tau, shards):
    n, V = h_cpu.shape[0], W.shape[0]
    h = h_cpu.cuda()
    Wd = W.cuda()
    routers, parts = [], []
    for g in range(shards):
        v0, v1 = P.shard_bounds(V, shards, g)
        r = P.VocabShardedRouter(Wd[v0:v1], v0, max_n=n, world=shards)
        parts.append(r.summarize(h).clone())
        routers.append(r)
    gathered = torch.stack(parts).contiguous()            # [shards, n, 4], rank-major like the all-gather
    last = routers[-1]
    last.token.fill_(-7); last.conf.fill_(float("nan")); last.entropy.fill_(float("nan"))
    last.route_mask.fill_(9); last.routed_idx.fill_(-3); last.routed_count.fill_(-5)
    last.finish(gathered, n, tau)
    torch.cuda.synchronize()
    status = 0
    for r in routers:
        status |= P.tlr_last_device_status(r.ctx)
    out = {"token": to_np(last.token[:n]), "conf": to_np(last.conf[:n]), "entropy": to_np(last.entropy[:n]),
           "route_mask": to_np(last.route_mask[:n]), "routed_idx": to_np(last.routed_idx),
           "routed_count": int(last.routed_count.item()), "status": status, "summaries": to_np(gathered)}
    for r in routers:
        r.close()
    return out


@pytest.mark.parametrize("n,d,V,shards", [(16, 64, 3000, 2), (37, 128, 4099, 3), (200, 256, 20011, 4),
                                          (300, 896, 9001, 8), (1, 64, 640, 2),
                                          # the benchmark's decode batch on the 0.5B-class head, eight shards
                                          (256, 896, 151936, 8)])
def test_sharded_matches_oracle_and_unsharded(pkg, n, d, V, shards):
    W = S.make_W(d, V, seed=n + V, std=0.1)
    hid = S.make_h(n, d, seed=n + V, W=W, planted_fraction=0.1 if n >= 16 else 0.0)
    first = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    tau = O.percentile_tau(first.conf, 0.5) if n > 1 else 0.5
    ref = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), tau)
    gpu = run_sharded(pkg, W, hid.h, tau, shards)
    assert gpu["status"] == 0
    check_self_consistency(gpu, tau, V)
    h64 = O.bf16_bits_to_f64(S.bf16_bits(hid.h)); W64 = O.bf16_bits_to_f64(S.bf16_bits(W))
    rep = check_against_oracle(ref, gpu, h64, W64)
    if rep["route_exempt_rows"] == 0:
        assert gpu["routed_count"] == ref.routed_count
        assert np.array_equal(gpu["routed_idx"][:ref.routed_count], ref.routed_idx)

    # each shard's summary against the oracle's definition of it
    for g in range(shards):
        v0, v1 = pkg.shard_bounds(V, shards, g)
        m, idx, s, t = O.shard_summary(S.bf16_bits(hid.h), S.bf16_bits(W)[v0:v1], v0)
        got = gpu["summaries"][g]
        got_idx = got[:, 1].copy().view(np.int32)
        assert np.allclose(got[:, 0], m, rtol=1e-5, atol=1e-4)     # fp32 accumulation over d products
        clear = np.ones(n, bool)
        if v1 - v0 > 1:                                   # rows whose top two logits inside the shard are near-tied
            z = h64 @ W64[v0:v1].T
            top2 = np.sort(z, axis=1)[:, -2:]
            clear = (top2[:, 1] - top2[:, 0]) >= 1e-3
        assert np.array_equal(got_idx[clear], idx[clear].astype(np.int32))
        assert np.allclose(got[:, 2], s, rtol=1e-4, atol=0)
        assert np.allclose(got[:, 3], t, rtol=1e-3, atol=1e-3)

    # the unsharded call on the same device: same decisions, scores equal to fp32 rounding
    one = run_gpu(pkg, W.cuda(), hid.h, tau)
    stable = ref.top2_gap >= 1e-3
    assert np.array_equal(one["token"][stable], gpu["token"][stable])
    assert np.allclose(one["conf"], gpu["conf"], rtol=1e-5, atol=0)
    assert np.allclose(one["entropy"], gpu["entropy"], rtol=0, atol=1e-4)


def test_tie_across_shards_goes_to_the_lower_index(pkg):
    d, V = 64, 2048
    W = S.make_W(d, V, seed=3, std=0.05)
    W[100] = W[100] * 6.0
    W[1500] = W[100]                                      # identical rows in different shards
    h = W[100:101].clone().repeat(5, 1)
    gpu = run_sharded(pkg, W, h, 0.5, 4)
    assert np.all(gpu["token"] == 100)


def test_shard_argument_errors(pkg):
    W = S.make_W(64, 1000, seed=1).cuda()
    r = pkg.VocabShardedRouter(W, 0, max_n=8, world=1)
    h = torch.zeros((9, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pkg.TlrError) as e:
        r.summarize(h)
    assert e.value.code == 6                              # more rows than max_n
    with pytest.raises(pkg.TlrError):
        pkg.tlr_shard_finish(r.ctx, r.summary, 0, 4, 0.5, r.token, r.conf, r.entropy, r.route_mask, r.routed_idx,
                             r.routed_count)                 # zero shards
    r.close()


def test_sharded_8bit_head(pkg):
    """Shards of an e4m3 head (codes and scales cut at the same rows), merged, against the oracle on the
    de-quantised matrix."""
    n, d, V, shards = 24, 128, 5000, 3
    codes, scale = S.make_W8(d, V, seed=8, std=0.1)
    W64 = O.dequantize_e4m3(codes.numpy(), scale.numpy())
    h = S.make_h(n, d, seed=8).h
    ref = O.route_oracle(S.bf16_bits(h), None, 0.5, W64=W64)
    cd, sd, hd = codes.cuda(), scale.cuda(), h.cuda()
    routers, parts = [], []
    for g in range(shards):
        v0, v1 = pkg.shard_bounds(V, shards, g)
        r = pkg.VocabShardedRouter(cd[v0:v1], v0, max_n=n, world=shards, wscale=sd[v0:v1])
        parts.append(r.summarize(hd).clone())
        routers.append(r)
    last = routers[-1]
    last.finish(torch.stack(parts).contiguous(), n, 0.5)
    torch.cuda.synchronize()
    gpu = {"token": to_np(last.token[:n]), "conf": to_np(last.conf[:n]), "entropy": to_np(last.entropy[:n]),
           "route_mask": to_np(last.route_mask[:n]), "routed_idx": to_np(last.routed_idx),
           "routed_count": int(last.routed_count.item())}
    check_self_consistency(gpu, 0.5, V)
    check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(h)), W64)
    for r in routers:
        assert pkg.tlr_last_device_status(r.ctx) == 0
        r.close()

"""Vocabulary-sharded step with the exchange fused into the kernels, on ONE GPU: the "peers" of every rank are
all the same local exchange block, and the ranks run one after the other in one stream (nothing waits on a
kernel that runs at the same time: by the time a merge kernel looks at the flags, the kernels that set them
have finished -- or, in the time-out test, nobody ever sets one and the bounded wait runs out).  Results are
compared with the oracle and with the all-gather form, for two calls in a row (the two halves of the block
alternate).  Also here: the merge of row-sharded index lists."""
import ctypes

import numpy as np
import pytest
import torch

import tlr_synth as S
from oracle import route_oracle as O
from tests.parity import check_against_oracle, check_self_consistency, to_np

pytestmark = pytest.mark.gpu


def make_ranks(P, Wd, max_n, shards):
    V = Wd.shape[0]
    block = torch.zeros(P.tlr_shard_block_bytes(max_n, shards), dtype=torch.uint8, device="cuda")
    assert block.data_ptr() % 256 == 0
    ranks = []
    for g in range(shards):
        v0, v1 = P.shard_bounds(V, shards, g)
        ranks.append(P.FusedVocabShardedRouter(Wd[v0:v1], v0, max_n, g, shards, [block] * shards, keep=block))
    return ranks, block


def outputs(r, n):
    return {"token": to_np(r.token[:n]), "conf": to_np(r.conf[:n]), "entropy": to_np(r.entropy[:n]),
            "route_mask": to_np(r.route_mask[:n]), "routed_idx": to_np(r.routed_idx),
            "routed_count": int(r.routed_count.item())}


def poison(r):
    r.token.fill_(-7); r.conf.fill_(float("nan")); r.entropy.fill_(float("nan"))
    r.route_mask.fill_(9); r.routed_idx.fill_(-3); r.routed_count.fill_(-5)


@pytest.mark.parametrize("n,d,V,shards", [(16, 64, 3000, 2), (37, 128, 4099, 3), (200, 256, 20011, 8),
                                          (256, 896, 151936, 8)])
def test_fused_exchange_matches_oracle_for_two_calls_in_a_row(pkg, n, d, V, shards):
    W = S.make_W(d, V, seed=n + V, std=0.1)
    Wd = W.cuda()
    W64 = O.bf16_bits_to_f64(S.bf16_bits(W))
    ranks, block = make_ranks(pkg, Wd, n, shards)
    reader = ranks[1 % shards]                      # any rank can finish: every block holds every summary
    for call, rows in enumerate((n, max(1, n // 2))):
        hid = S.make_h(rows, d, seed=call + n, W=W, planted_fraction=0.1 if rows >= 16 else 0.0)
        first = O.route_oracle(S.bf16_bits(hid.h), None, 0.5, W64=W64)
        tau = O.percentile_tau(first.conf, 0.5) if rows > 1 else 0.5
        ref = O.with_threshold(first, tau)
        h = hid.h.cuda()
        for r in ranks:
            r.push(h)
        poison(reader)
        reader.finish(rows, tau)
        torch.cuda.synchronize()
        for r in ranks:
            assert pkg.tlr_last_device_status(r.ctx) == 0
        gpu = outputs(reader, rows)
        check_self_consistency(gpu, tau, V)
        rep = check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(hid.h)), W64)
        if rep["route_exempt_rows"] == 0:
            assert gpu["routed_count"] == ref.routed_count
            assert np.array_equal(gpu["routed_idx"][:ref.routed_count], ref.routed_idx)
        # the all-gather form on the same shards: the same summaries through the same merge, bit for bit
        gatherers = []
        for g in range(shards):
            v0, v1 = pkg.shard_bounds(V, shards, g)
            gatherers.append(pkg.VocabShardedRouter(Wd[v0:v1], v0, max_n=rows, world=shards))
        parts = [ag.summarize(h).clone() for ag in gatherers]
        gatherers[-1].finish(torch.stack(parts).contiguous(), rows, tau)
        torch.cuda.synchronize()
        want = outputs(gatherers[-1], rows)
        for ag in gatherers:
            ag.close()
        for key in ("token", "conf", "entropy", "route_mask"):
            assert np.array_equal(gpu[key], want[key]), key
        assert gpu["routed_count"] == want["routed_count"]
        assert np.array_equal(gpu["routed_idx"][:gpu["routed_count"]], want["routed_idx"][:gpu["routed_count"]])
    for r in ranks:
        r.close()


def test_a_flag_that_is_never_set_runs_the_wait_out_and_the_context_survives(pkg):
    n, d, V, shards = 20, 64, 3000, 3
    W = S.make_W(d, V, seed=5, std=0.1)
    hid = S.make_h(n, d, seed=5)
    ref = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    ranks, block = make_ranks(pkg, W.cuda(), n, shards)
    h = hid.h.cuda()
    ranks[0].push(h)
    ranks[1].push(h)                                 # rank 2 "never joins"
    pkg.tlr_debug_inject(ranks[0].ctx, 0, 200)        # every wait of this context gives up after 0.2 s
    ranks[0].finish(n, 0.5)
    torch.cuda.synchronize()
    assert pkg.tlr_last_device_status(ranks[0].ctx) & pkg.TLR_DEV_WAIT_TIMEOUT
    # the missing rank arrives: the same call number is now complete, and the context works as before
    ranks[2].push(h)
    poison(ranks[0])
    ranks[0].finish(n, 0.5)
    torch.cuda.synchronize()
    assert pkg.tlr_last_device_status(ranks[0].ctx) == 0
    gpu = outputs(ranks[0], n)
    check_against_oracle(ref, gpu)
    for r in ranks:
        r.close()


def test_fused_exchange_argument_errors(pkg):
    W = S.make_W(64, 1000, seed=1).cuda()
    ctx = pkg.tlr_create(64, 1000, W, 8)
    h = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    out = [torch.zeros(8, dtype=t, device="cuda") for t in (torch.int32, torch.float32, torch.float32, torch.uint8,
                                                             torch.int32)] + [torch.zeros(1, dtype=torch.int32, device="cuda")]
    with pytest.raises(pkg.TlrError) as e:
        pkg.tlr_shard_push(ctx, h, 4, 0)             # not attached
    assert e.value.code == 1
    block = torch.zeros(pkg.tlr_shard_block_bytes(8, 2) + 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(pkg.TlrError) as e:
        pkg.tlr_shard_attach(ctx, 0, 2, [block.data_ptr() + 16, block.data_ptr()])
    assert e.value.code == 2                         # a block that is not 256-byte aligned
    with pytest.raises(pkg.TlrError):
        pkg.tlr_shard_attach(ctx, 2, 2, [block, block])   # rank out of range
    pkg.tlr_shard_attach(ctx, 0, 2, [block, block])
    with pytest.raises(pkg.TlrError) as e:
        pkg.tlr_shard_finish_fused(ctx, 4, 0.5, *out)     # nothing pushed yet
    assert e.value.code == 1
    pkg.tlr_destroy(ctx)


@pytest.mark.parametrize("rows_per_rank,d,V", [((40, 40, 40), 64, 3000), ((300, 1, 129, 77), 128, 5003), ((5, 0, 9), 64, 700)])
def test_row_sharded_lists_merge_into_the_global_list(pkg, rows_per_rank, d, V):
    """Every "rank" routes its own rows (here one after the other on one GPU); its index list lands in its slot as
    an all-gather would deliver it, and one kernel makes the global ascending list -- which must be the oracle's
    list for the concatenated batch."""
    W = S.make_W(d, V, seed=V, std=0.1)
    Wd = W.cuda()
    total = sum(rows_per_rank)
    hid = S.make_h(total, d, seed=V, W=W, planted_fraction=0.2)
    first = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    tau = O.percentile_tau(first.conf, 0.5)
    ref = O.with_threshold(first, tau)
    cap = max(max(rows_per_rank), 1)
    world = len(rows_per_rank)
    gathered = torch.full((world, cap), -1, dtype=torch.int32, device="cuda")
    counts = torch.zeros(world, dtype=torch.int32, device="cuda")
    offs = pkg.row_offsets(rows_per_rank)
    router = pkg.Router(Wd, max_n=cap)
    for g, rows in enumerate(rows_per_rank):
        h = hid.h[offs[g]:offs[g] + rows].cuda() if rows else torch.empty((0, d), dtype=torch.bfloat16, device="cuda")
        _, _, _, _, idx, cnt = router.route(h, tau)
        gathered[g].copy_(idx[:cap])
        counts[g:g + 1].copy_(cnt)
    out, n_out = pkg.merge_routed(gathered, counts, torch.tensor(offs, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    near = np.abs(ref.conf - ref.tau) <= 1e-3 * ref.tau
    if not near.any():
        assert int(n_out.item()) == ref.routed_count
        assert np.array_equal(to_np(out[:ref.routed_count]), ref.routed_idx)
    got = to_np(out[:int(n_out.item())])
    assert np.all(np.diff(got) > 0) and int(n_out.item()) == int(to_np(counts).sum())
    router.close()
    with pytest.raises(pkg.TlrError):
        pkg.tlr_rows_merge(gathered, counts, None, world, cap, out, n_out)


@pytest.mark.parametrize("n", [24, 100])        # one MMA per K step / one per part of h
def test_fused_exchange_on_the_8bit_head(pkg, n):
    """Shards of an e4m3 head (codes and scales cut at the same rows) with the exchange fused into the kernels,
    against the oracle on the de-quantised matrix."""
    d, V, shards = 128, 9000, 4
    codes, scale = S.make_W8(d, V, seed=8, std=0.1)
    W64 = O.dequantize_e4m3(codes.numpy(), scale.numpy())
    h = S.make_h(n, d, seed=n).h
    first = O.route_oracle(S.bf16_bits(h), None, 0.5, W64=W64)
    tau = O.percentile_tau(first.conf, 0.5)
    ref = O.with_threshold(first, tau)
    cd, sd, hd = codes.cuda(), scale.cuda(), h.cuda()
    block = torch.zeros(pkg.tlr_shard_block_bytes(n, shards), dtype=torch.uint8, device="cuda")
    ranks = []
    for g in range(shards):
        v0, v1 = pkg.shard_bounds(V, shards, g)
        ranks.append(pkg.FusedVocabShardedRouter(cd[v0:v1], v0, n, g, shards, [block] * shards, wscale=sd[v0:v1],
                                                 keep=block))
    for r in ranks:
        r.push(hd)
    poison(ranks[2])
    ranks[2].finish(n, tau)
    torch.cuda.synchronize()
    for r in ranks:
        assert pkg.tlr_last_device_status(r.ctx) == 0
    gpu = outputs(ranks[2], n)
    check_self_consistency(gpu, tau, V)
    rep = check_against_oracle(ref, gpu, O.bf16_bits_to_f64(S.bf16_bits(h)), W64)
    if rep["route_exempt_rows"] == 0:
        assert gpu["routed_count"] == ref.routed_count
        assert np.array_equal(gpu["routed_idx"][:ref.routed_count], ref.routed_idx)
    for r in ranks:
        r.close()

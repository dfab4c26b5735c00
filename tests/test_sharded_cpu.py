"""Host-side logic of the vocabulary-sharded step: the shard bounds, and -- as two gloo ranks on CPU --
that the all-gather delivers the per-row summaries rank-major, so that merging what every rank receives
reproduces the unsharded result.  The per-shard summaries here come from the oracle (there is no GPU);
the GPU kernels that produce and merge them are tested in tests/test_gpu_sharded.py."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


@pytest.mark.parametrize("V,world", [(151936, 8), (128256, 4), (1000, 3), (64, 2), (33, 2)])
def test_shard_bounds_tile_the_vocabulary(V, world):
    from paper_2504_07878_b200.sharded import GRANULE, shard_bounds
    edges = [shard_bounds(V, world, r) for r in range(world)]
    assert edges[0][0] == 0 and edges[-1][1] == V
    for (a0, a1), (b0, b1) in zip(edges[:-1], edges[1:]):
        assert a1 == b0 and a0 < a1
    assert all(v0 % GRANULE == 0 for v0, _ in edges)          # 16-byte aligned row blocks for any d % 8 == 0
    sizes = [v1 - v0 for v0, v1 in edges]
    assert max(sizes) - min(sizes) <= 2 * GRANULE


def test_shard_bounds_rejects_bad_requests():
    from paper_2504_07878_b200.sharded import shard_bounds
    with pytest.raises(ValueError):
        shard_bounds(1000, 4, 4)
    with pytest.raises(ValueError):
        shard_bounds(40, 3, 0)                                # fewer granules than shards


def _rank_main(rank, world, port, out_dir):
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    import torch.distributed as dist
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import tlr_synth as S
    from oracle import route_oracle as O
    from paper_2504_07878_b200.sharded import gather_summaries, shard_bounds
    n, d, V = 12, 32, 1000
    W = S.make_W(d, V, seed=7, std=0.2)                       # every rank builds the same W and h ...
    h = S.make_h(n, d, seed=7).h
    v0, v1 = shard_bounds(V, world, rank)                     # ... and summarises only its own rows
    m, idx, s, t = O.shard_summary(S.bf16_bits(h), S.bf16_bits(W)[v0:v1], v0)
    local = torch.from_numpy(np.stack([m, idx.astype(np.float64), s, t], axis=1))      # [n, 4]
    got = gather_summaries(local).numpy()                     # [world, n, 4]
    np.save(os.path.join(out_dir, "rank%d.npy" % rank), got)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_gather_rank_major_and_merge_to_the_unsharded_result(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    import tlr_synth as S
    from oracle import route_oracle as O
    from paper_2504_07878_b200.sharded import shard_bounds
    n, d, V = 12, 32, 1000
    W = S.make_W(d, V, seed=7, std=0.2)
    h = S.make_h(n, d, seed=7).h
    ref = O.route_oracle(S.bf16_bits(h), S.bf16_bits(W), 0.5)
    got = [np.load(tmp_path / ("rank%d.npy" % r)) for r in range(world)]
    assert np.array_equal(got[0], got[1])                     # every rank holds the same gathered block
    for g in range(world):                                    # slot g is rank g's shard
        v0, v1 = shard_bounds(V, world, g)
        idx = got[0][g, :, 1].astype(np.int64)
        assert np.all((idx >= v0) & (idx < v1))
    parts = [(got[0][g, :, 0], got[0][g, :, 1].astype(np.int64), got[0][g, :, 2], got[0][g, :, 3])
             for g in range(world)]
    token, conf, ent = O.merge_summaries(parts)
    assert np.array_equal(token, ref.token)
    assert np.allclose(conf, ref.conf, rtol=1e-12) and np.allclose(ent, ref.entropy, atol=1e-12)

"""Host-side logic of the two multi-GPU exchanges that need more than a barrier, run as two gloo ranks on CPU.

Row sharding: every rank routes its own rows; the ranks all-gather their routed-index lists, counts and row
numbers, and the global list is each rank's list shifted by the number of rows before it.  Here the per-rank
results come from the oracle (there is no GPU); the exchange is the package's own (exchange_routed), and the
merged list -- rebuilt from what the exchange delivered by the documented rule -- must be the oracle's list for
the concatenated batch.  The kernel that does this merge on the GPU is tested in tests/test_gpu_sharded_fused.py.

Fused vocabulary-shard exchange: the address tables every rank derives from the ranks' block addresses (the
library's own host function) must be consistent -- no two ranks write the same bytes of a peer's block, the two
halves that alternate between calls are disjoint, every flag lies in the header."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

ROWS = (23, 9)          # rows of rank 0 and rank 1
D, V, CAP = 32, 1000, 32


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _batch():
    import tlr_synth as S
    W = S.make_W(D, V, seed=9, std=0.2)
    hid = S.make_h(sum(ROWS), D, seed=9, W=W, planted_fraction=0.3)
    return W, hid


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
    import paper_2504_07878_b200 as P
    W, hid = _batch()
    start = sum(ROWS[:rank])
    mine = O.route_oracle(S.bf16_bits(hid.h)[start:start + ROWS[rank]], S.bf16_bits(W), 0.5)
    idx = torch.full((CAP,), -1, dtype=torch.int32)
    idx[:mine.routed_count] = torch.from_numpy(mine.routed_idx)
    gathered, counts, offsets = P.exchange_routed(idx, torch.tensor([mine.routed_count], dtype=torch.int32), ROWS[rank])
    np.savez(os.path.join(out_dir, "rows%d.npz" % rank), gathered=gathered.numpy(), counts=counts.numpy(),
             offsets=offsets.numpy())

    # fused vocabulary-shard exchange: everybody learns everybody's block address, then derives its own tables
    base = torch.tensor([(rank + 1) << 32], dtype=torch.int64)             # a made-up, 256-byte aligned address
    bases = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(bases, base)
    blocks = [int(b.item()) for b in bases]
    tables = [P.tlr_debug_shard_table(64, rank, world, blocks, parity) for parity in (0, 1)]
    np.save(os.path.join(out_dir, "table%d.npy" % rank), np.array(tables, dtype=np.int64))   # [parity][slot|flag][peer]
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_exchange_lists_and_tables(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    import tlr_synth as S
    from oracle import route_oracle as O
    import paper_2504_07878_b200 as P
    W, hid = _batch()
    ref = O.route_oracle(S.bf16_bits(hid.h), S.bf16_bits(W), 0.5)
    assert 0 < ref.routed_count < sum(ROWS)
    got = [np.load(tmp_path / ("rows%d.npz" % r)) for r in range(world)]
    for key in ("gathered", "counts", "offsets"):
        assert np.array_equal(got[0][key], got[1][key])                    # every rank holds the same exchange result
    assert got[0]["offsets"].tolist() == P.row_offsets(ROWS) == [0, ROWS[0]]
    merged = np.concatenate([got[0]["gathered"][g, :got[0]["counts"][g]] + got[0]["offsets"][g] for g in range(world)])
    assert np.array_equal(merged, ref.routed_idx) and int(got[0]["counts"].sum()) == ref.routed_count

    max_n = 64
    size = P.tlr_shard_block_bytes(max_n, world)
    header = 256
    assert size == header + 2 * world * max_n * 16
    tables = [np.load(tmp_path / ("table%d.npy" % r)) for r in range(world)]     # [rank][parity][slot|flag][peer]
    blocks = [(r + 1) << 32 for r in range(world)]
    for peer in range(world):
        spans, flags = [], []
        for rank in range(world):
            for parity in (0, 1):
                slot, flag = tables[rank][parity][0][peer], tables[rank][parity][1][peer]
                assert blocks[peer] + header <= slot and slot + max_n * 16 <= blocks[peer] + size and slot % 16 == 0
                assert blocks[peer] <= flag < blocks[peer] + header and flag % 4 == 0
                spans.append((slot, slot + max_n * 16))
                flags.append(flag)
        spans.sort()
        assert all(a[1] <= b[0] for a, b in zip(spans[:-1], spans[1:]))         # nobody writes anybody else's slot
        assert len(set(flags)) == 2 * world
    # a rank's own view of peer g is the same address as peer g's view of itself with that rank's number
    assert tables[0][0][0][1] - blocks[1] == tables[0][0][0][0] - blocks[0]

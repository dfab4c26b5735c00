"""Host-side logic of the multi-GPU benchmark path, run as two gloo ranks on CPU.

The routing path shards by rows with no data-path collective, so what N > 1 adds on the host is
the rendezvous, the per-rank workload (each rank its own seeded batch) and the max-over-ranks
time that turns into the whole-job throughput."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out_dir):
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    import torch.distributed as dist
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import tlr_synth as S
    # each rank draws its own batch (seed = rank), as the benchmark does
    h = S.make_h(8, 16, seed=rank).h
    slow = bench.max_over_ranks(10.0 * (rank + 1), world, "cpu")     # rank 1 is the slow one
    dist.barrier()
    with open(os.path.join(out_dir, "rank%d.txt" % rank), "w") as f:
        f.write("%r %r\n" % (slow, float(h.double().sum())))
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    rows = [open(tmp_path / ("rank%d.txt" % r)).read().split() for r in range(world)]
    assert float(rows[0][0]) == float(rows[1][0]) == 20.0
    assert rows[0][1] != rows[1][1]                    # different batches on different ranks


def test_job_throughput_is_the_sum_over_ranks():
    import bench
    assert bench.job_throughput(1, 256, 1e-4) == pytest.approx(2.56e6)
    assert bench.job_throughput(8, 256, 1e-4) == pytest.approx(8 * 2.56e6)
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5

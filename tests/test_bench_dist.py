"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, max-over-ranks timing and whole-job aggregation."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
    out[rank] = (ms, bench.aggregate(3.0e12, world, ms), bench.rank_seed_offset(rank))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_max_time_and_summed_work():
    world, port = 2, _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0][0] == out[1][0] == 15.0                          # max over ranks, on every rank
    assert abs(out[0][1] - 2 * 3.0e12 / 15.0e-3 / 1e12) < 1e-9     # both ranks' work over the slowest time
    assert out[0][2] != out[1][2]                                  # each rank draws its own batch


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, 1) == 7.5
    assert abs(bench.aggregate(2.0e12, 1, 1000.0) - 2.0) < 1e-12       # 2e12 ops in 1000 ms = 2 TOPS

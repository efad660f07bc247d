"""The N > 1 benchmark path on CPU: two gloo ranks, each an independent replica, agree on the
slowest rank's time and on the aggregate (no GPU; the data path has no collective)."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 0.010 * (rank + 1)                     # rank 1 is the slow one
    slowest = bench.max_over_ranks(mine, dist)
    units = bench.sum_over_ranks(1000.0 * (rank + 1), dist)
    dist.barrier()
    out[rank] = (slowest, units)
    dist.destroy_process_group()


def test_two_ranks_agree_on_slowest_time_and_total_units():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    assert abs(res[0][0] - 0.020) < 1e-12 and res[0][1] == 3000.0


def test_single_process_helpers_are_identity():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(0.5, None) == 0.5
    assert bench.sum_over_ranks(7.0, None) == 7.0
    ab = bench.algorithmic_bytes(335_141_888, 16, 32768)
    # ~12.13 n + 20.1 bytes per parameter per step, dominated by the worker kernel
    per_param = ab["step"] / 335_141_888
    assert 12.1 * 16 + 20 < per_param < 12.4 * 16 + 20.5
    assert ab["worker"] / ab["step"] > 0.85

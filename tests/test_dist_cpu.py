"""The N > 1 path of the benchmark on CPU: two gloo ranks shard independent sequences with no data-path
collective; the whole-job rate divides the units of all ranks by the slowest rank's time."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_24133_b200 import dist as rd


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, lr, w = rd.init("gloo")
    assert (r, w) == (rank, world)
    lo, hi = rd.shard_range(7, r, w)
    units = float(hi - lo) * 100.0                 # 100 tokens per sequence
    ms = 2.0 if r == 0 else 5.0                    # rank 1 is slower
    rd.barrier()
    rate, slow = rd.whole_job_rate(units, ms, "cpu")
    out[rank] = (lo, hi, rate, slow)
    dist.destroy_process_group()


def test_two_rank_sharding_and_whole_job_rate():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][:2] == (0, 4) and res[1][:2] == (4, 7)          # disjoint, covering, near-equal
    for r in (0, 1):
        assert abs(res[r][3] - 5.0) < 1e-12                        # max over ranks
        assert abs(res[r][2] - 700.0 / 5e-3) < 1e-6                # all units / slowest time


def test_shard_range_covers_everything_once():
    for total in (1, 7, 32, 33):
        for world in (1, 2, 3, 8):
            spans = [rd.shard_range(total, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def test_single_process_paths_need_no_process_group():
    assert rd.env_world()[2] >= 1
    assert rd.max_over_ranks(3.5, "cpu") == 3.5
    assert rd.whole_job_rate(10.0, 2.0, "cpu") == (5000.0, 2.0)

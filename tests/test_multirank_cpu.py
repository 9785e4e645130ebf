"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The method shards by client stream and
exchanges nothing on the data path; what the ranks share is the timing (max over ranks) from which
the whole-job rate is formed."""
import os
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank                        # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, dist)
    streams = bench.rank_streams(3, world, rank)
    gathered = [None] * world
    dist.all_gather_object(gathered, streams)
    dist.barrier()
    out[rank] = (ms, bench.whole_job_rate(80.0, world, ms), gathered)
    dist.destroy_process_group()


def test_two_ranks_share_only_the_timing():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        ms, rate, gathered = res[rank]
        assert ms == 15.0                                # the slowest rank sets the time on every rank
        assert rate == pytest.approx(2 * 80.0 / 0.015)   # units of all ranks / that time
        flat = sorted(s for part in gathered for s in part)
        assert flat == list(range(6))                    # streams are partitioned: disjoint and complete


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None) == 3.5
    assert bench.rank_streams(16, 1, 0) == list(range(16))
    assert bench.whole_job_rate(8.0, 1, 1.0) == 8000.0

"""Host logic of the multi-GPU benchmark (replicas, no data-path collective) on two CPU ranks over gloo:
every rank gets its own reproducible batch, the job's time is the slowest rank's, throughput is the sum."""

import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    perm = bench.rank_batch_permutation(1024, rank)
    my_ms = 10.0 + 5.0 * rank  # rank 1 is the slow one
    job_ms = bench.max_over_ranks(my_ms, world, "cpu")
    gathered = [None] * world
    dist.all_gather_object(gathered, perm.tolist())
    out[rank] = (job_ms, bench.whole_job_qps(1024, world, 4, job_ms), gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_share_the_slowest_time_and_search_distinct_batches():
    world = 2
    port = 29000 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert set(out.keys()) == {0, 1}
    for rank in range(world):
        job_ms, qps, perms = out[rank]
        assert job_ms == 15.0                                   # max over ranks, seen by every rank
        assert abs(qps - 1024 * 2 * 4 / 0.015) < 1e-6           # whole-job aggregate
        assert sorted(perms[0]) == list(range(1024)) and sorted(perms[1]) == list(range(1024))
        assert perms[0] != perms[1]                             # each replica has its own batch


def test_batches_are_reproducible_and_single_rank_is_a_noop():
    import bench
    assert torch.equal(bench.rank_batch_permutation(64, 3), bench.rank_batch_permutation(64, 3))
    assert bench.max_over_ranks(7.5, 1, "cpu") == 7.5

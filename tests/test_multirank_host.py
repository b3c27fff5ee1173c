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


def _shard_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import numpy as np
    import oracle
    from paper_2503_14649_b200 import sharded, synth
    from tests.helpers import host_index
    shards = synth.make_ivfpq_shards(world, 900, 16, 8, 4, 5, metric="l2", seed=5)
    # this rank answers for its own shard only (the oracle stands in for the GPU search on a CPU rank)
    ids, dists = oracle.ivfpq_search(host_index(oracle, shards[rank]), shards[rank].queries.numpy(), 3, 7)
    all_ids, all_dists = sharded.gather_parts(torch.from_numpy(ids), torch.from_numpy(dists))
    merged = oracle.merge_results(all_ids.numpy(), all_dists.numpy(), 7, "l2")
    out[rank] = (all_ids.numpy().copy(), merged[0], merged[1], ids)
    dist.barrier()
    dist.destroy_process_group()


def test_two_shard_ranks_exchange_their_answers_in_rank_order():
    """The exchange step of the sharded search over gloo: after the all-gather every rank holds every
    shard's answer at that shard's index, so aggregating gives the answer over the whole database."""
    import numpy as np
    import oracle
    from paper_2503_14649_b200 import synth
    from tests.helpers import host_index
    world = 2
    port = 31000 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_shard_worker, args=(world, port, out), nprocs=world, join=True)
    shards = synth.make_ivfpq_shards(world, 900, 16, 8, 4, 5, metric="l2", seed=5)
    want = oracle.sharded_search([host_index(oracle, s) for s in shards], shards[0].queries.numpy(), 3, 7)
    for rank in range(world):
        all_ids, m_ids, m_d, own = out[rank]
        assert all_ids.shape == (2, 5, 7) and np.array_equal(all_ids[rank], own)
        assert np.array_equal(m_ids, want[0]) and np.array_equal(m_d, want[1])
    assert np.array_equal(out[0][0], out[1][0])
    # both shards contribute
    assert (want[0] < 900).any() and (want[0] >= 900).any()

"""GPU parity of the sharded search (paper, Sec. 4: independent index per shard, results aggregated):
the aggregation kernel against the oracle's definition entry by entry, and the whole path with the
shards searched one after the other on one GPU."""

import numpy as np
import pytest
import torch

import oracle
from paper_2503_14649_b200 import binding, sharded, synth
from tests.helpers import IvfPqRescorer, host_index, match_results

pytestmark = pytest.mark.gpu


def _random_parts(rng, nparts, nq, k_in, metric, pad_frac=0.2, distinct=True):
    """Shard answers in rago_search's layout: rows best first, padding (-1, +-inf) at the end."""
    total = nparts * nq * k_in
    if distinct:
        vals = rng.permutation(total).astype(np.float32) * 0.25 - 1000.0   # exact in fp32, all different
    else:
        vals = rng.integers(0, 12, total).astype(np.float32)               # many ties
    d = vals.reshape(nparts, nq, k_in)
    d = np.sort(d, axis=2) if metric == "l2" else -np.sort(-d, axis=2)
    ids = rng.permutation(total).astype(np.int64).reshape(nparts, nq, k_in) + 5
    n_real = rng.integers(0, k_in + 1, (nparts, nq))
    n_real[rng.random((nparts, nq)) > pad_frac] = k_in
    pad = np.arange(k_in)[None, None, :] >= n_real[:, :, None]
    ids[pad] = -1
    d[pad] = np.inf if metric == "l2" else -np.inf
    return ids, np.ascontiguousarray(d)


@pytest.mark.parametrize("nparts,nq,k_in,k_out,metric", [
    (1, 7, 10, 10, "l2"), (3, 33, 100, 100, "ip"), (8, 9, 1000, 1000, "l2"), (8, 5, 1024, 1024, "ip"),
    (4, 11, 37, 5, "l2"), (2, 6, 3, 40, "ip"), (16, 4, 300, 1, "l2"), (5, 3, 1, 4, "l2")])
def test_merge_kernel_matches_definition(nparts, nq, k_in, k_out, metric):
    rng = np.random.default_rng(nparts * 1000 + k_in)
    ids, d = _random_parts(rng, nparts, nq, k_in, metric)
    gi, gd = binding.rago_merge_results(torch.from_numpy(ids).cuda(), torch.from_numpy(d).cuda(), k_out, metric)
    torch.cuda.synchronize()
    oi, od = oracle.merge_results(ids, d, k_out, metric)
    assert np.array_equal(gi.cpu().numpy(), oi)            # scores are all different: one right answer
    assert np.array_equal(gd.cpu().numpy(), od)            # distances are copied, bit for bit


@pytest.mark.parametrize("metric", ["l2", "ip"])
def test_merge_kernel_with_ties_and_all_padding(metric):
    rng = np.random.default_rng(3)
    ids, d = _random_parts(rng, 6, 20, 50, metric, pad_frac=0.5, distinct=False)
    ids[:, 4, :] = -1                                       # a query no shard has an answer for
    d[:, 4, :] = np.inf if metric == "l2" else -np.inf
    gi, gd = binding.rago_merge_results(torch.from_numpy(ids).cuda(), torch.from_numpy(d).cuda(), 64, metric)
    gi, gd = gi.cpu().numpy(), gd.cpu().numpy()
    oi, od = oracle.merge_results(ids, d, 64, metric)
    assert np.array_equal(gd, od)                           # the score sequence is unique
    assert (gi[4] == -1).all()
    for q in range(20):
        # inside a group of equal scores any order is right; the group cut by k_out may differ in members
        real = od[q][oi[q] >= 0]
        last = real[-1] if real.size else None
        pool = {(int(i), float(s)) for i, s in zip(ids[:, q].ravel(), d[:, q].ravel()) if i >= 0}
        got = [(int(i), float(s)) for i, s in zip(gi[q], gd[q]) if i >= 0]
        assert len(got) == real.size and len(set(got)) == len(got) and set(got) <= pool
        inner = {e for e in got if e[1] != last}
        assert inner == {(int(i), float(s)) for i, s in zip(oi[q], od[q]) if i >= 0 and s != last}


def test_merge_argument_errors():
    ids = torch.zeros((2, 3, 4), dtype=torch.int64, device="cuda")
    d = torch.zeros((2, 3, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.RagoError) as e:
        binding.rago_merge_results(ids, d, 2000, "l2")
    assert e.value.status == 3   # RAGO_EUNSUPPORTED
    with pytest.raises(binding.RagoError) as e:
        binding.rago_merge_results(ids, d, 0, "l2")
    assert e.value.status == 1   # RAGO_EINVAL
    with pytest.raises(binding.RagoError):
        binding.rago_merge_results(ids, d, 4, 7)
    with pytest.raises(ValueError):
        binding.rago_merge_results(ids, d[:, :, :2], 4, "l2")


@pytest.mark.parametrize("metric,S,nprobe,k", [("l2", 4, 8, 100), ("ip", 3, 5, 33), ("l2", 2, 64, 1000)])
def test_sharded_search_on_one_gpu_matches_oracle(metric, S, nprobe, k):
    """Each shard has its own index; the shards are searched in turn on this GPU (one GPU stands in for S),
    their answers are laid out as the all-gather leaves them and aggregated by the kernel."""
    shards = synth.make_ivfpq_shards(S, 30_000, 64, 64, 16, 40, metric=metric, seed=31 + S)
    q = shards[0].queries.cuda().contiguous()
    parts_i, parts_d = [], []
    for sh in shards:
        ix = binding.load_index_from(sh, "cuda")
        i, d = ix.rago_search(q, nprobe, k)
        torch.cuda.synchronize()
        ix.rago_check()
        parts_i.append(i.clone())
        parts_d.append(d.clone())
        ix.close()
    gi, gd = binding.rago_merge_results(torch.stack(parts_i), torch.stack(parts_d), k, metric)
    gi, gd = gi.cpu().numpy(), gd.cpu().numpy()
    hixs = [host_index(oracle, sh) for sh in shards]
    oi, od = oracle.sharded_search(hixs, shards[0].queries.numpy(), nprobe, k, nthreads=oracle.default_threads())
    sgn = 1.0 if metric == "l2" else -1.0
    rss = [IvfPqRescorer(oracle, h) for h in hixs]
    qh = shards[0].queries.numpy()
    for i in range(q.shape[0]):
        def rescore(ident, i=i):  # ids are s * 30 000 + a permutation: the owning shard scores its vector
            if ident < 0 or ident >= S * 30_000:
                raise KeyError(ident)
            return rss[ident // 30_000].for_query(qh[i], sgn)(ident)
        assert not match_results(gi[i], sgn * gd[i], oi[i], sgn * od[i], rel=1e-4, rescore=rescore), i
    owners = np.unique(oi[oi >= 0] // 30_000)
    assert owners.size == S                                  # every shard contributes to the answers


def test_single_rank_sharded_call_equals_plain_search():
    data = synth.make_ivfpq(50_000, 64, 32, 16, 25, metric="l2", seed=4)
    ix = binding.load_index_from(data, "cuda")
    q = data.queries.cuda()
    a = ix.rago_search(q, 6, 20)
    a = (a[0].clone(), a[1].clone())
    b = sharded.rago_search_sharded(ix, q, 6, 20)
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    ix.close()

"""GPU parity of the two-level coarse quantiser (paper, Methodology: a multi-level tree index scanned top-down)
against the oracle's step-by-step definition: probe lists equal except inside coarse-score ties, search results
equal except inside distance ties, distances within 1e-4 relative."""

import numpy as np
import pytest
import torch

import oracle
from paper_2503_14649_b200 import binding, synth
from tests.helpers import IvfPqRescorer, coarse_rescorer, host_index, match_results

pytestmark = pytest.mark.gpu

REL = 1e-4


def _tree_host(data):
    top, off = data.extra["level1"], data.extra["child_offsets"]
    top_h = top.cpu().view(torch.uint16).numpy() if top.dtype == torch.bfloat16 else top.cpu().numpy()
    return top_h, off.cpu().numpy()


def _load_with_tree(data, b1):
    ix = binding.load_index_from(data, "cuda")
    ix.rago_index_set_coarse_tree(data.extra["level1"].cuda().contiguous(), data.extra["child_offsets"].cuda().contiguous(), b1)
    return ix


def _check_probes(data, b1, nprobe, queries=None):
    q_t = data.queries if queries is None else queries
    hix = host_index(oracle, data)
    top_h, off_h = _tree_host(data)
    q = q_t.cpu().numpy()
    ol, oc = oracle.coarse_tree(hix.centroids, top_h, off_h, b1, q, nprobe, data.metric, coarse_bf16=data.coarse_bf16,
                                nthreads=oracle.default_threads())
    ix = _load_with_tree(data, b1)
    gl, gc = ix.rago_search_probes(q_t.cuda().contiguous(), nprobe)
    torch.cuda.synchronize()
    ix.rago_check()
    gl, gc = gl.cpu().numpy(), gc.cpu().numpy()
    ix.close()
    sgn = 1.0 if data.metric == "l2" else -1.0
    for i in range(q.shape[0]):
        if not np.array_equal(gl[i], ol[i]):
            problems = match_results(gl[i].astype(np.int64), sgn * gc[i], ol[i].astype(np.int64), sgn * oc[i], rel=REL,
                                     rescore=coarse_rescorer(oracle, hix.centroids, q[i], data.metric, data.coarse_bf16, sgn))
            assert not problems, ("probe lists", i, problems[:4])
        assert np.allclose(gc[i], oc[i], rtol=REL, atol=REL * max(1.0, np.abs(oc[i]).max())), ("coarse", i)


# N, d, nlist, M, nq, n1, b1, nprobe, metric, bf16
CASES = [
    (3000, 64, 60, 16, 5, 10, 1, 4, "l2", False),        # uneven nodes? 60 / 10 = 6 children each, one node kept
    (3000, 64, 61, 16, 7, 9, 3, 12, "ip", False),        # nodes of 6 and 7 children
    (4000, 96, 256, 16, 40, 16, 4, 33, "l2", True),      # bf16 quantiser, a batch above the small-batch threshold
    (4000, 128, 512, 32, 1, 32, 8, 16, "l2", False),     # one query: many CTAs share its candidates
    (4000, 768, 1024, 64, 130, 32, 5, 64, "ip", True),   # the Hyperscale shape in miniature
    (2000, 32, 40, 16, 6, 40, 40, 40, "l2", False),      # every node kept, every list probed
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "nl%d_n1%d_b%d_np%d_nq%d_%s%s" % (c[2], c[5], c[6], c[7], c[4], c[8],
                                                                                         "_bf16" if c[9] else ""))
def test_tree_probes_match_oracle(case):
    N, d, nlist, M, nq, n1, b1, nprobe, metric, bf16 = case
    data = synth.make_ivfpq_hashed(N, d, nlist, M, nq, metric=metric, seed=500 + nlist, coarse_bf16=bf16, tree_n1=n1)
    _check_probes(data, b1, nprobe)


@pytest.mark.parametrize("metric,bf16,nq", [("l2", False, 16), ("ip", True, 48), ("l2", False, 1)])
def test_tree_search_matches_oracle(metric, bf16, nq):
    """The latency shape in miniature (d = 512, M = 32, 16 probes of 128 x 32 lists) and its bf16 / inner-product twin."""
    data = synth.make_ivfpq_hashed(300_000, 512, 1024, 32, nq, metric=metric, seed=77, coarse_bf16=bf16, tree_n1=32)
    hix = host_index(oracle, data)
    top_h, off_h = _tree_host(data)
    q = data.queries.numpy()
    oi, od, op = oracle.ivfpq_search_tree(hix, top_h, off_h, 4, q, 16, 20, nthreads=oracle.default_threads(), want_probes=True)
    ix = _load_with_tree(data, 4)
    gi, gd = ix.rago_search(data.queries.cuda().contiguous(), 16, 20)
    gl, _ = ix.rago_search_probes(data.queries.cuda().contiguous(), 16)
    torch.cuda.synchronize()
    ix.rago_check()
    gi, gd, gl = gi.cpu().numpy(), gd.cpu().numpy(), gl.cpu().numpy()
    ix.close()
    rs = IvfPqRescorer(oracle, hix)
    sgn = 1.0 if metric == "l2" else -1.0
    for i in range(nq):
        assert set(gl[i].tolist()) == set(op[i].tolist()), ("probe lists", i)
        problems = match_results(gi[i], sgn * gd[i], oi[i], sgn * od[i], rel=REL, rescore=rs.for_query(q[i], sgn))
        assert not problems, (i, problems[:4])


def test_keeping_every_node_gives_the_one_level_answer_and_the_level_can_be_removed():
    data = synth.make_ivfpq_hashed(60_000, 128, 256, 16, 24, metric="l2", seed=78, tree_n1=16)
    ix = binding.load_index_from(data, "cuda")
    q = data.queries.cuda().contiguous()
    flat = ix.rago_search(q, 8, 30)
    flat = (flat[0].clone(), flat[1].clone())
    top, off = data.extra["level1"].cuda(), data.extra["child_offsets"].cuda()
    ix.rago_index_set_coarse_tree(top, off, 16)
    full = ix.rago_search(q, 8, 30)
    torch.cuda.synchronize()
    assert torch.equal(flat[0], full[0]) and torch.allclose(flat[1], full[1], rtol=1e-6, atol=0)
    ix.rago_index_set_coarse_tree(top, off, 1)
    narrow = ix.rago_search_probes(q, 8)[0].clone()
    ix.rago_index_set_coarse_tree(None, None)
    again = ix.rago_search(q, 8, 30)
    torch.cuda.synchronize()
    assert torch.equal(flat[0], again[0]) and torch.equal(flat[1], again[1])
    offs = off.cpu().numpy()
    for i in range(24):   # with one node kept all probes are siblings
        nodes = np.searchsorted(offs, narrow[i].cpu().numpy(), side="right") - 1
        assert len(set(nodes.tolist())) == 1
    ix.close()


def test_tree_argument_errors():
    data = synth.make_ivfpq_hashed(3000, 64, 64, 16, 4, metric="l2", seed=79, tree_n1=8)
    ix = binding.load_index_from(data, "cuda")
    top, off = data.extra["level1"].cuda(), data.extra["child_offsets"].cuda()
    for b1 in (0, 9, 65):
        with pytest.raises(binding.RagoError):
            ix.rago_index_set_coarse_tree(top, off, b1)
    bad = off.clone()
    bad[3] = bad[2] - 1
    with pytest.raises(binding.RagoError) as e:
        ix.rago_index_set_coarse_tree(top, bad, 2)
    assert "decrease" in str(e.value)
    ix.rago_index_set_coarse_tree(top, off, 2)           # two nodes of eight lists each
    q = data.queries.cuda().contiguous()
    with pytest.raises(binding.RagoError) as e:
        ix.rago_search(q, 17, 5)                          # more probes than two nodes can offer
    assert e.value.status == 1
    ix.rago_search(q, 16, 5)
    with pytest.raises(binding.RagoError):                # the no-workspace coarse step scores every list
        ix.rago_search_probes_noalloc(q, 4, torch.empty((4, 4), dtype=torch.int32, device="cuda"),
                                      torch.empty((4, 4), dtype=torch.float32, device="cuda"))
    torch.cuda.synchronize()
    ix.close()

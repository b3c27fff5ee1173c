"""Tensor-core coarse step (tcgen05 GEMM with the nprobe selection fused into its epilogue) against the
CPU oracle: probe lists equal except inside coarse-score ties, coarse values within 1e-4 relative, and
the whole search unchanged by the choice of coarse kernel."""

import numpy as np
import pytest
import torch

import oracle
from paper_2503_14649_b200 import binding, synth
from tests.helpers import IvfPqRescorer, coarse_rescorer, host_index, match_results

pytestmark = pytest.mark.gpu

REL = 1e-4


def _probe_parity(data, nprobe, mode):
    hix = host_index(oracle, data)
    q = data.queries.cpu().numpy()
    ol, oc = oracle.coarse(hix.centroids, q, nprobe, data.metric, coarse_bf16=data.coarse_bf16,
                           nthreads=oracle.default_threads())
    ix = binding.load_index_from(data, "cuda")
    ix.rago_set_coarse_mode(mode)
    gl, gc = ix.rago_search_probes(data.queries.cuda().contiguous(), nprobe)
    torch.cuda.synchronize()
    ix.rago_check()
    gl, gc = gl.cpu().numpy(), gc.cpu().numpy()
    ix.close()
    sgn = 1.0 if data.metric == "l2" else -1.0
    for i in range(q.shape[0]):
        if not np.array_equal(gl[i], ol[i]):
            problems = match_results(gl[i].astype(np.int64), sgn * gc[i], ol[i].astype(np.int64), sgn * oc[i], rel=REL,
                                     rescore=coarse_rescorer(oracle, hix.centroids, q[i], data.metric, data.coarse_bf16, sgn))
            assert not problems, ("probe order", i, problems[:4])
        assert np.allclose(gc[i], oc[i], rtol=REL, atol=REL * max(1.0, np.abs(oc[i]).max())), ("coarse", i)


# N, d, nlist, M, nq, nprobe, metric, bf16
TC_CASES = [
    (2000, 64, 300, 16, 40, 8, "l2", False),      # one ragged column tile, one ragged row tile
    (2000, 64, 300, 16, 40, 8, "ip", True),
    (2000, 96, 1000, 16, 130, 16, "l2", True),    # d not a multiple of 64, two row tiles
    (2000, 128, 513, 16, 257, 33, "ip", False),   # three row tiles, column tail of one list
    (500, 32, 40, 16, 5, 40, "l2", False),        # nprobe = nlist, tiny batch forced onto tensor cores
]


@pytest.fixture(params=[1, 2, 3], ids=["one_row_tile", "paired_row_tiles", "cta_pair"])
def pairing(request):
    """Both main loops of the tensor-core kernel: batches of more than 128 queries take the forced one."""
    binding.rago_debug_set_gemm_pairing(request.param)
    yield request.param
    binding.rago_debug_set_gemm_pairing(0)


# every case under the one-row-tile loop, and those with more than 128 queries under the paired loop as well
TC_RUNS = [(c, 1) for c in TC_CASES] + [(c, 2) for c in TC_CASES if c[4] > 128] + [(c, 3) for c in TC_CASES if c[4] > 128]


@pytest.mark.parametrize("case,pair", TC_RUNS, ids=lambda v: ("d%d_nl%d_nq%d_np%d_%s%s" % (v[1], v[2], v[4], v[5], v[6],
                         "_bf16" if v[7] else "")) if isinstance(v, tuple) else {1: "single", 2: "paired", 3: "cta_pair"}[v])
def test_tensor_core_probes_match_oracle(case, pair):
    N, d, nlist, M, nq, nprobe, metric, bf16 = case
    binding.rago_debug_set_gemm_pairing(pair)
    try:
        data = synth.make_ivfpq(N, d, nlist, M, nq, metric=metric, seed=300 + nlist + nq, coarse_bf16=bf16)
        _probe_parity(data, nprobe, mode=2)
    finally:
        binding.rago_debug_set_gemm_pairing(0)


@pytest.mark.parametrize("metric,bf16", [("l2", False), ("ip", True)])
def test_long_rows_exercise_list_compaction(metric, bf16, pairing):
    """16 384 lists, 600 queries: a CTA sees several column tiles of a row, so candidate lists fill up and
    are compacted while the GEMM runs."""
    data = synth.make_ivfpq(4000, 64, 16384, 16, 600, metric=metric, seed=77, coarse_bf16=bf16)
    _probe_parity(data, 32, mode=2)


def test_large_nprobe_uses_the_wide_lists_and_the_score_matrix(pairing):
    data = synth.make_ivfpq(3000, 64, 8192, 16, 150, metric="l2", seed=78)
    _probe_parity(data, 300, mode=2)    # nsel = 308: 1024-key lists
    _probe_parity(data, 1000, mode=2)   # nsel = 1008: score-matrix epilogue


def test_search_results_do_not_depend_on_the_coarse_kernel():
    data = synth.make_ivfpq(60_000, 128, 256, 32, 96, metric="l2", seed=79, zipf=1.1)
    ix = binding.load_index_from(data, "cuda")
    q = data.queries.cuda().contiguous()
    out = {}
    for mode in (1, 2):
        ix.rago_set_coarse_mode(mode)
        ids, dists = ix.rago_search(q, 16, 50)
        torch.cuda.synchronize()
        ix.rago_check()
        out[mode] = (ids.cpu().numpy().copy(), dists.cpu().numpy().copy())
    ix.close()
    rs = IvfPqRescorer(oracle, host_index(oracle, data))
    qh = data.queries.numpy()
    for i in range(96):  # the fp32-pipe run stands where the oracle's list would; an id only one run lists is oracle-scored
        assert not match_results(out[2][0][i], out[2][1][i], out[1][0][i], out[1][1][i], rel=REL,
                                 rescore=rs.for_query(qh[i])), i

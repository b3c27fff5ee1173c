"""The no-allocation coarse step (rago_search_probes_noalloc) against rago_search_probes.

Some users of the library cannot allocate device memory when they search: the GPU's free memory
belongs to an LLM server's pool, or an allocation would synchronise a device that is busy serving.
For them the library keeps the coarse step's score matrix in a fixed array of its own.  This test
calls that entry point through the C ABI twice in a row (the second call finds the first call's
data in the shared array and must not be disturbed by it) and expects the same probe lists and
coarse values as the workspace-based entry point and as the CPU oracle's coarse step, then checks that an
oversized batch is refused.  The file name sorts last so that every other GPU test has run before this one.
"""

import numpy as np
import pytest
import torch

import oracle
from paper_2503_14649_b200 import binding, synth
from tests.helpers import coarse_rescorer, host_index, match_results

pytestmark = pytest.mark.gpu

REL = 1e-4  # the tolerance of the other GPU parity tests


@pytest.mark.parametrize("metric,bf16", [("l2", False), ("ip", True)])
def test_noalloc_probes_match_workspace_probes_twice(metric, bf16):
    data = synth.make_ivfpq(6000, 128, 96, 16, 48, metric=metric, seed=901, coarse_bf16=bf16)
    ix = binding.load_index_from(data, "cuda")
    q_all = data.queries.cuda().contiguous()
    hix = host_index(oracle, data)
    sgn = 1.0 if metric == "l2" else -1.0
    nprobe = 12
    # outputs are the caller's and exist before the calls; the calls themselves allocate nothing
    for lo, hi in ((0, 48), (5, 29)):  # second call: fewer, different queries over the same array
        q = q_all[lo:hi].contiguous()
        want_lists, want_coarse = ix.rago_search_probes(q, nprobe)
        got_lists = torch.full((hi - lo, nprobe), -7, dtype=torch.int32, device="cuda")
        got_coarse = torch.full((hi - lo, nprobe), float("nan"), dtype=torch.float32, device="cuda")
        ix.rago_search_probes_noalloc(q, nprobe, got_lists, got_coarse)
        torch.cuda.synchronize()
        assert torch.equal(got_lists.cpu(), want_lists.cpu())
        g, w = got_coarse.cpu().numpy(), want_coarse.cpu().numpy()
        assert np.allclose(g, w, rtol=REL, atol=REL * max(1.0, float(np.abs(w).max())))
        # and against the oracle's coarse step directly, so that this file stands on its own
        qh = data.queries[lo:hi].numpy()
        ol, oc = oracle.coarse(hix.centroids, qh, nprobe, metric, coarse_bf16=bf16)
        gl = got_lists.cpu().numpy().astype(np.int64)
        for i in range(hi - lo):
            assert not match_results(gl[i], sgn * g[i], ol[i].astype(np.int64), sgn * oc[i], rel=REL,
                                     rescore=coarse_rescorer(oracle, hix.centroids, qh[i], metric, bf16, sgn)), i
    ix.close()


def test_noalloc_refuses_batches_beyond_the_builtin_scratch():
    data = synth.make_ivfpq(3000, 64, 2048, 16, 4, metric="l2", seed=902)
    ix = binding.load_index_from(data, "cuda")
    nq = 4 * 1024 * 1024 // (2048 * 4) + 1  # one query more than the score matrix can hold
    q = torch.zeros((nq, 64), device="cuda")
    lists = torch.empty((nq, 4), dtype=torch.int32, device="cuda")
    coarse = torch.empty((nq, 4), dtype=torch.float32, device="cuda")
    before = binding.rago_kernel_launches()
    with pytest.raises(binding.RagoError) as e:
        ix.rago_search_probes_noalloc(q, 4, lists, coarse)
    assert e.value.status == 4 and "limit" in str(e.value)
    assert binding.rago_kernel_launches() == before
    ix.rago_search_probes_noalloc(q[:16].contiguous(), 4, lists[:16], coarse[:16])  # a batch that fits still works
    torch.cuda.synchronize()
    ix.close()

"""The failure path of the bounded device-side waits, driven without anything being wrong.

Every wait of the library's kernels (on a bulk copy, on the tensor pipe, between the roles of a CTA) gives up
after a fixed number of polls, raises the CTA's abort flag, records RAGO_ETIMEOUT in the workspace's error word
and lets the kernel end normally.  rago_selftest_wait_timeout runs that very wait on a barrier nobody signals,
with a small poll limit: the wait runs out by itself within a millisecond, nothing faults or hangs.  Checked
here: rago_check reports the time-out, the second waiting warp is released through the abort flag, the device
and the workspace stay usable (the next search on the same workspace is correct and reports no error), and the
variant that holds tensor memory during the wait gives it back (a tensor-core coarse step runs right after).
"""

import numpy as np
import pytest
import torch

import oracle
from paper_2503_14649_b200 import binding, synth
from tests.helpers import IvfPqRescorer, host_index, match_results

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("with_tmem", [False, True])
def test_an_expired_wait_is_reported_and_leaves_the_device_usable(with_tmem):
    data = synth.make_ivfpq(30_000, 128, 300, 16, 40, metric="l2", seed=611)
    ix = binding.load_index_from(data, "cuda")
    ix.rago_set_coarse_mode(2)  # tensor cores: the next search allocates tensor memory itself
    q = data.queries.cuda().contiguous()
    ws = torch.zeros(ix.search_workspace_bytes(40, 8, 10), dtype=torch.uint8, device="cuda")
    ix.rago_search(q, 8, 10, workspace=ws)
    binding.rago_check(ws)                                         # a healthy workspace reports nothing

    binding.rago_selftest_wait_timeout(ws, 64, with_tmem)          # 64 polls of at most 4 us each
    with pytest.raises(binding.RagoError) as e:
        binding.rago_check(ws)
    assert e.value.status == 6 and "wait" in str(e.value)          # RAGO_ETIMEOUT
    words = ws[:64].view(torch.int32).cpu().numpy()
    assert words[0] == 1                                           # the error word itself
    assert words[8] == 1 and words[9] == 1                         # first wait expired; second released by the abort flag

    # the same workspace, the same device, right away: a correct search and a clean error word
    ids, dists = ix.rago_search(q, 8, 10, workspace=ws)
    torch.cuda.synchronize()
    binding.rago_check(ws)
    hix = host_index(oracle, data)
    oi, od = oracle.ivfpq_search(hix, data.queries.numpy(), 8, 10, nthreads=oracle.default_threads())
    rs = IvfPqRescorer(oracle, hix)
    gi, gd = ids.cpu().numpy(), dists.cpu().numpy()
    for i in range(40):
        assert not match_results(gi[i], gd[i], oi[i], od[i], rel=1e-4, rescore=rs.for_query(data.queries[i].numpy())), i
    ix.close()


def test_selftest_arguments_are_checked_on_the_host():
    ws = torch.zeros(512, dtype=torch.uint8, device="cuda")
    before = binding.rago_kernel_launches()
    for polls in (0, 5000):
        with pytest.raises(binding.RagoError) as e:
            binding.rago_selftest_wait_timeout(ws, polls, False)
        assert e.value.status == 1
    assert binding.rago_kernel_launches() == before

"""GPU parity of the 4-bit product-quantised index (the paper's low-precision PQ variant, Sec. 2) against the
numpy definition in the oracle: ids equal except inside ties, distances within 1e-4 relative."""

import numpy as np
import pytest
import torch

import oracle
from paper_2503_14649_b200 import binding, synth
from tests.helpers import match_results

pytestmark = pytest.mark.gpu


def _compare(data, nprobe, k):
    bf16 = data.centroids.dtype == torch.bfloat16
    cen = data.centroids.view(torch.uint16).numpy() if bf16 else data.centroids.numpy()
    oi, od = oracle.ivfpq4_search(cen, data.codebooks.numpy(), data.codes.numpy(), data.list_offsets.numpy(),
                                  data.ids.numpy(), data.metric, data.queries.numpy(), nprobe, k, coarse_bf16=bf16)
    ix = binding.rago_index_load_pq4(data.centroids.cuda(), data.codebooks.cuda(), data.codes.cuda(),
                                     data.list_offsets.cuda(), data.ids.cuda(), data.metric)
    gi, gd = ix.rago_search(data.queries.cuda().contiguous(), nprobe, k)
    torch.cuda.synchronize()
    ix.rago_check()
    gi, gd = gi.cpu().numpy(), gd.cpu().numpy()
    ix.close()
    sgn = 1.0 if data.metric == "l2" else -1.0
    ids_h, off_h, qh = data.ids.numpy(), data.list_offsets.numpy(), data.queries.numpy()
    order = np.argsort(ids_h, kind="stable")
    for i in range(gi.shape[0]):
        def rescore(ident, i=i):
            # the oracle's score of that one vector: a search of its own list alone, restricted to the vector
            j = int(np.searchsorted(ids_h[order], ident))
            if j >= ids_h.size or int(ids_h[order][j]) != ident:
                raise KeyError(ident)
            pos = int(order[j])
            lst = int(np.searchsorted(off_h, pos, side="right") - 1)
            one_off = np.zeros_like(off_h)
            one_off[lst + 1:] = 1
            si, sd = oracle.ivfpq4_search(cen, data.codebooks.numpy(), data.codes.numpy()[pos:pos + 1], one_off,
                                          ids_h[pos:pos + 1], data.metric, qh[i:i + 1], cen.shape[0], 1, coarse_bf16=bf16)
            assert int(si[0, 0]) == ident
            return sgn * float(sd[0, 0])
        assert not match_results(gi[i], sgn * gd[i], oi[i], sgn * od[i], rel=1e-4, rescore=rescore), i


@pytest.mark.parametrize("N,d,nlist,M4,nq,nprobe,k,metric,bf16", [
    (20_000, 64, 32, 32, 20, 6, 25, "l2", False),       # 16 code bytes, dsub 2
    (60_000, 128, 64, 64, 40, 8, 100, "ip", False),     # 32 code bytes
    (50_000, 192, 48, 96, 33, 5, 10, "l2", True),       # 48 code bytes, bf16 coarse quantiser
    (40_000, 256, 40, 128, 17, 40, 300, "ip", True),    # 64 code bytes, every list probed
    (30_000, 768, 32, 192, 12, 4, 50, "l2", False),     # the Mid shape's d with 96 code bytes, dsub 4
    (25_000, 256, 16, 256, 9, 3, 7, "l2", False),       # 128 code bytes, dsub 1
    (3_000, 160, 8, 160, 5, 2, 1000, "ip", False),      # 80 code bytes, k beyond the candidates
])
def test_pq4_search_matches_definition(N, d, nlist, M4, nq, nprobe, k, metric, bf16):
    data = synth.make_ivfpq4(N, d, nlist, M4, nq, metric=metric, seed=N % 97, coarse_bf16=bf16,
                             zipf=1.0 if N > 40_000 else None)
    _compare(data, nprobe, k)


def test_pq4_argument_errors():
    data = synth.make_ivfpq4(1000, 64, 8, 32, 2, seed=3)
    cb = data.codebooks.cuda()
    with pytest.raises(binding.RagoError) as e:       # odd number of sub-spaces
        binding.Index(data.centroids.cuda(), cb[:31].contiguous(), data.codes.cuda(), data.list_offsets.cuda(),
                      data.ids.cuda(), "l2")
    assert e.value.status == 1
    with pytest.raises(binding.RagoError) as e:       # 8 code bytes: no scan kernel of that width
        binding.Index(data.centroids.cuda(), cb[:16].contiguous(), data.codes.cuda()[:, :8].contiguous(),
                      data.list_offsets.cuda(), data.ids.cuda(), "l2")
    assert e.value.status == 3

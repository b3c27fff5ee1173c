"""Host checks of the seeded input generators (no method arithmetic is tested here)."""

import numpy as np
import torch

from paper_2503_14649_b200 import synth


def test_hash_codes_are_position_addressable():
    a = synth.hash_codes(7, 0, 1000, 32)
    b = synth.hash_codes(7, 400, 100, 32)
    assert a.dtype == torch.uint8 and a.shape == (1000, 32)
    assert torch.equal(a[400:500], b)
    assert not torch.equal(a, synth.hash_codes(8, 0, 1000, 32))
    hist = torch.bincount(a.flatten().long(), minlength=256)
    assert hist.min() > 60 and hist.max() < 200  # roughly uniform bytes


def test_hash_ids_unique_nonnegative():
    i = synth.hash_ids(123, 50000)
    assert i.min() >= 0 and torch.unique(i).numel() == 50000
    assert torch.equal(i[10:20], synth.hash_ids(133, 10))


def test_jitter_lengths_sum_and_range():
    L = synth.jitter_lengths(1, 1_000_003, 4096)
    assert int(L.sum()) == 1_000_003
    mean = 1_000_003 / 4096
    assert L.min() >= 0.45 * mean and L.max() <= 1.6 * mean
    off = synth.offsets_from_lengths(L)
    assert off[0] == 0 and off[-1] == 1_000_003 and (off[1:] >= off[:-1]).all()


def test_make_ivfpq_structure_and_determinism():
    a = synth.make_ivfpq(5000, 32, 16, 8, 10, seed=3, zipf=1.1, keep_vectors=True)
    b = synth.make_ivfpq(5000, 32, 16, 8, 10, seed=3, zipf=1.1)
    assert torch.equal(a.codes, b.codes) and torch.equal(a.ids, b.ids) and torch.equal(a.queries, b.queries)
    assert a.codes.shape == (5000, 8) and a.list_offsets[-1] == 5000
    assert torch.equal(torch.sort(a.ids).values, torch.arange(5000))
    L = a.list_offsets[1:] - a.list_offsets[:-1]
    assert L[0] > 3 * L[8:].float().mean()  # rank-1 component dominates under Zipf weights
    # codes really are nearest codewords of the residuals (checked on a few vectors by a plain loop)
    off = a.list_offsets.numpy()
    cb = a.codebooks.numpy()
    for pos in (0, 17, 4999):
        lst = int(np.searchsorted(off, pos, side="right") - 1)
        r = (a.vectors[pos] - a.centroids[lst]).numpy().reshape(8, 4)
        for m in range(8):
            dist = ((cb[m] - r[m][None]) ** 2).sum(1)
            assert int(a.codes[pos, m]) == int(dist.argmin())


def test_nearest_assignment_lists_are_voronoi_cells():
    a = synth.make_ivfpq(2000, 16, 8, 4, 4, seed=5, assign="nearest", keep_vectors=True)
    off = a.list_offsets.numpy()
    lab = np.repeat(np.arange(8), np.diff(off))
    d2 = ((a.vectors[:, None, :] - a.centroids[None]) ** 2).sum(-1).numpy()
    assert (d2.argmin(1) == lab).mean() > 0.999


def test_flat_rows_are_unit_norm_bf16():
    db, q = synth.make_flat(1000, 64, 4, seed=2)
    assert db.dtype == torch.bfloat16 and q.shape == (4, 64)
    assert torch.allclose(db.float().norm(dim=1), torch.ones(1000), atol=2e-2)


def test_paper_size_arithmetic():
    # 64e9 vectors x 96-byte codes = 5.6 TiB (RAGO, methodology: database description)
    assert abs(64e9 * 96 / 2 ** 40 - 5.6) < 0.05
    c = synth.CONFIGS[2]
    assert c["d"] // c["M"] == 8 and c["M"] == 96  # 1 byte per 8 dims, 768-d -> 96 bytes


def test_batch_stream():
    s = synth.batch_size_stream(1)
    assert len(s) == 256 and set(s) == {1, 4, 16}

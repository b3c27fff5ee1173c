"""Pins for the CPU oracle: things fixed by the paper's definitions and by arithmetic,
none of which call the oracle to produce their expected values.

* hand-worked 2-D / 4-D examples (tests/golden/*.json, computed by hand);
* numpy brute force written from the plain definitions (K most similar vectors under
  squared L2 / inner product) -- coarse step, flat search, and full IVF-PQ search
  checked as exact kNN over the *decoded* database restricted to the probed lists;
* lossless PQ + nprobe = nlist reproduces exact kNN on the raw vectors;
* bf16 rounding against torch's conversion;
* structural invariants (monotone in nprobe, storage-order invariance, padding).
"""

import json
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2503_14649_b200 import synth
from tests.helpers import host_index

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _inf(v):
    return float(v) if not isinstance(v, str) else float(v)


def _load_example(name):
    g = json.load(open(os.path.join(GOLD, name)))
    d, M = g["d"], g["M"]
    dsub = d // M
    cb = np.full((M, 256, dsub), g["unused_codeword_value"], np.float32)
    cw = np.asarray(g["codewords_0_to_3"], np.float32).reshape(4, dsub)
    cb[:, :4, :] = cw[None]
    return g, cb


@pytest.mark.parametrize("name", ["handworked_2d.json", "handworked_4d.json"])
@pytest.mark.parametrize("metric", ["l2", "ip"])
def test_handworked_examples(name, metric):
    g, cb = _load_example(name)
    ix = oracle.Index(np.asarray(g["centroids"], np.float32), cb, np.asarray(g["codes"], np.uint8),
                      np.asarray(g["list_offsets"], np.int64), np.asarray(g["ids"], np.int64), metric)
    q = np.asarray([g["query"]], np.float32)
    lists, scores = oracle.coarse(ix.centroids, q, g["nlist"], metric)
    want = np.asarray(g[metric]["coarse"])
    order = np.argsort(want if metric == "l2" else -want, kind="stable")
    assert lists[0].tolist() == order.tolist()
    assert np.allclose(scores[0], want[order], rtol=0, atol=0)
    for case in g[metric]["cases"]:
        ids, dists = oracle.ivfpq_search(ix, q, case["nprobe"], case["k"])
        assert ids[0].tolist() == case["ids"], case
        assert dists[0].tolist() == [_inf(v) for v in case["dists"]], case
    # the printed tables: one vector per codeword combination reproduces table sums
    if metric == "l2" and "table_probe0" in g["l2"]:
        t0 = np.asarray(g["l2"]["table_probe0"])
        for pos in range(g["list_offsets"][1]):
            c = g["codes"][pos]
            want_sum = sum(t0[m][c[m]] for m in range(g["M"]))
            assert oracle.adc_score(ix, q[0], 0, pos) == want_sum
    # decoded vectors as printed
    for pos, dec in enumerate(g["decoded"]):
        lst = int(np.searchsorted(ix.offsets, pos, side="right") - 1)
        _, got = oracle.decode_score(ix, q[0], lst, pos, want_decoded=True)
        assert got.tolist() == dec


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 10.0 ** rng.integers(-20, 20, 20000),
                        np.asarray([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, -65504.0, 1e-40],
                                   np.float32)]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.uint16).numpy()
    assert np.array_equal(oracle.f32_to_bf16_bits(x), want)


def _brute_coarse(cen, q, metric):
    cen = cen.astype(np.float64)
    q = q.astype(np.float64)
    if metric == "l2":  # expanded form, unlike the oracle's (q-c)^2 loop
        return (q * q).sum(1)[:, None] - 2.0 * q @ cen.T + (cen * cen).sum(1)[None, :]
    return q @ cen.T


@pytest.mark.parametrize("metric", ["l2", "ip"])
def test_coarse_against_numpy_bruteforce(metric):
    rng = np.random.default_rng(2)
    cen = rng.standard_normal((300, 24)).astype(np.float32)
    q = rng.standard_normal((17, 24)).astype(np.float32)
    lists, scores = oracle.coarse(cen, q, 11, metric, nthreads=3)
    s = _brute_coarse(cen, q, metric)
    order = np.argsort(s if metric == "l2" else -s, axis=1, kind="stable")[:, :11]
    assert np.array_equal(lists, order)
    assert np.allclose(scores, np.take_along_axis(s, order, 1), rtol=1e-12, atol=1e-12)


def test_coarse_bf16_reading():
    """bf16 coarse quantiser: the query is rounded to bf16 for the coarse step."""
    rng = np.random.default_rng(3)
    cen = torch.from_numpy(rng.standard_normal((200, 32)).astype(np.float32)).to(torch.bfloat16)
    q = rng.standard_normal((9, 32)).astype(np.float32)
    lists, scores = oracle.coarse(cen.view(torch.uint16).numpy(), q, 7, "ip", coarse_bf16=True)
    qb = torch.from_numpy(q).to(torch.bfloat16).double().numpy()
    s = qb @ cen.double().numpy().T
    order = np.argsort(-s, axis=1, kind="stable")[:, :7]
    assert np.array_equal(lists, order)
    assert np.allclose(scores, np.take_along_axis(s, order, 1), rtol=1e-13)
    # and it is not the unrounded product
    s_raw = q.astype(np.float64) @ cen.double().numpy().T
    assert not np.allclose(scores, np.take_along_axis(s_raw, order, 1), rtol=1e-9)


def test_flat_against_numpy_bruteforce():
    db, q = synth.make_flat(700, 48, 5, seed=11)
    ids, sc = oracle.flat_search(db.view(torch.uint16).numpy(), q.view(torch.uint16).numpy(), 13, nthreads=2)
    s = q.double().numpy() @ db.double().numpy().T
    order = np.argsort(-s, axis=1, kind="stable")[:, :13]
    assert np.array_equal(ids, order)
    assert np.allclose(sc, np.take_along_axis(s, order, 1), rtol=1e-6)
    # k beyond N pads with (-1, -inf)
    ids2, sc2 = oracle.flat_search(db[:3].view(torch.uint16).numpy(), q.view(torch.uint16).numpy(), 5)
    assert (ids2[:, 3:] == -1).all() and np.isneginf(sc2[:, 3:]).all()
    rows = np.asarray([5, 0, 699], np.int64)
    assert np.allclose(oracle.flat_scores(db.view(torch.uint16).numpy(), q[1].view(torch.uint16).numpy(), rows),
                       s[1, rows], rtol=1e-13)


def _decode_all(data):
    """Reconstruction y^ = centroid + concatenated codewords, in float64 numpy."""
    cen = data.centroids.double().numpy()
    cb = data.codebooks.double().numpy()
    codes = data.codes.numpy().astype(np.int64)
    off = data.list_offsets.numpy()
    lab = np.repeat(np.arange(data.nlist), np.diff(off))
    M = data.M
    parts = [cb[m][codes[:, m]] for m in range(M)]
    return lab, np.concatenate(parts, axis=1), cen


def _bruteforce_ivfpq(data, nprobe, k):
    """Exact kNN over the decoded vectors of the probed lists (definition, not the table algorithm)."""
    lab, resid, cen = _decode_all(data)
    q = data.queries.double().numpy()
    qc = data.queries.to(torch.bfloat16).float() if data.coarse_bf16 else data.queries
    cs = _brute_coarse(data.centroids.float().numpy(), qc.numpy(), data.metric)
    order = np.argsort(cs if data.metric == "l2" else -cs, axis=1, kind="stable")[:, :nprobe]
    ids = data.ids.numpy()
    out_i = np.full((q.shape[0], k), -1, np.int64)
    out_d = np.full((q.shape[0], k), np.inf if data.metric == "l2" else -np.inf)
    for i in range(q.shape[0]):
        sel = np.nonzero(np.isin(lab, order[i]))[0]
        if data.metric == "l2":
            y = cen[lab[sel]] + resid[sel]
            s = ((q[i][None] - y) ** 2).sum(1)
            key = np.lexsort((ids[sel], s))
        else:
            s = cs[i, lab[sel]] + resid[sel] @ q[i]
            key = np.lexsort((ids[sel], -s))
        key = key[:k]
        out_i[i, :key.size] = ids[sel][key]
        out_d[i, :key.size] = s[key]
    return out_i, out_d, order


@pytest.mark.parametrize("metric,bf16", [("l2", False), ("ip", False), ("ip", True), ("l2", True)])
@pytest.mark.parametrize("nprobe", [1, 5, 16])
def test_search_is_exact_knn_over_decoded_probed_lists(metric, bf16, nprobe):
    data = synth.make_ivfpq(3000, 32, 16, 8, 12, metric=metric, seed=21 + nprobe, coarse_bf16=bf16)
    ix = host_index(oracle, data)
    k = 9
    ids, dists, probes = oracle.ivfpq_search(ix, data.queries.numpy(), nprobe, k, nthreads=2, want_probes=True)
    bi, bd, border = _bruteforce_ivfpq(data, nprobe, k)
    assert np.array_equal(probes, border)
    assert np.allclose(dists, bd, rtol=2e-6, atol=1e-6)
    same = ids == bi
    # an id may differ only where two scores tie to rounding
    for r, c in zip(*np.nonzero(~same)):
        assert abs(bd[r, c] - bd[r, max(c - 1, 0)]) < 1e-6 * abs(bd[r, c]) or \
            abs(bd[r, c] - bd[r, min(c + 1, k - 1)]) < 1e-6 * abs(bd[r, c])
    assert same.mean() > 0.99


@pytest.mark.parametrize("metric", ["l2", "ip"])
def test_table_sum_equals_decode_then_score(metric):
    data = synth.make_ivfpq(500, 24, 6, 6, 3, metric=metric, seed=5)
    ix = host_index(oracle, data)
    lab, resid, cen = _decode_all(data)
    q = data.queries.numpy()
    for pos in range(0, 500, 37):
        lst = int(lab[pos])
        a = oracle.adc_score(ix, q[1], lst, pos)
        b, dec = oracle.decode_score(ix, q[1], lst, pos, want_decoded=True)
        y = cen[lst] + resid[pos]
        assert np.allclose(dec, y, rtol=0, atol=1e-12)
        direct = ((q[1].astype(np.float64) - y) ** 2).sum() if metric == "l2" else float(q[1].astype(np.float64) @ y)
        assert abs(a - b) <= 1e-6 * max(1.0, abs(b))
        assert abs(b - direct) <= 1e-12 * max(1.0, abs(direct))


def test_lossless_pq_full_probe_equals_exact_knn():
    """dsub = 1, every residual coordinate is a codeword => IVF-PQ with nprobe = nlist is exact kNN."""
    rng = np.random.default_rng(7)
    d, nlist, N, nq, k = 6, 5, 400, 8, 10
    grid = (np.arange(256, dtype=np.float32) - 128.0) / 32.0  # exactly representable
    cb = np.repeat(grid[None, :, None], d, axis=0).astype(np.float32)  # [M=d][256][1]
    cen = rng.integers(-8, 9, (nlist, d)).astype(np.float32)
    lab = np.sort(rng.integers(0, nlist, N))
    codes = rng.integers(0, 256, (N, d)).astype(np.uint8)
    vectors = cen[lab] + grid[codes]  # exact in float
    off = np.concatenate([[0], np.cumsum(np.bincount(lab, minlength=nlist))]).astype(np.int64)
    ids = rng.permutation(N).astype(np.int64)
    q = (rng.integers(-64, 65, (nq, d)) / 8.0).astype(np.float32)
    for metric in ("l2", "ip"):
        ix = oracle.Index(cen, cb, codes, off, ids, metric)
        got_i, got_d = oracle.ivfpq_search(ix, q, nlist, k)
        v = vectors.astype(np.float64)
        qq = q.astype(np.float64)
        s = ((qq[:, None, :] - v[None]) ** 2).sum(-1) if metric == "l2" else qq @ v.T
        for i in range(nq):
            key = np.lexsort((ids, s[i] if metric == "l2" else -s[i]))[:k]
            assert got_i[i].tolist() == ids[key].tolist()
            assert np.array_equal(got_d[i], s[i][key].astype(np.float32))


def test_invariants_nprobe_monotone_permutation_padding_empty_lists():
    data = synth.make_ivfpq(2000, 16, 32, 4, 6, metric="l2", seed=9)
    ix = host_index(oracle, data)
    q = data.queries.numpy()
    prev = None
    for nprobe in (1, 2, 4, 8, 32):
        _, dd = oracle.ivfpq_search(ix, q, nprobe, 7)
        if prev is not None:
            assert (dd <= prev).all()  # more lists can only improve every rank
        prev = dd
    # storage order of the lists does not matter: rebuild with lists laid out in reverse
    off = data.list_offsets.numpy()
    codes, ids = data.codes.numpy(), data.ids.numpy()
    pieces = [(codes[off[l]:off[l + 1]], ids[off[l]:off[l + 1]]) for l in range(data.nlist)]
    rev_lengths = [p[0].shape[0] for p in pieces]
    # same list numbering, but within-list order reversed
    codes2 = np.concatenate([p[0][::-1] for p in pieces])
    ids2 = np.concatenate([p[1][::-1] for p in pieces])
    ix2 = oracle.Index(ix.centroids, ix.codebooks, codes2, off, ids2, "l2")
    a = oracle.ivfpq_search(ix, q, 8, 7)
    b = oracle.ivfpq_search(ix2, q, 8, 7)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert sum(rev_lengths) == data.N
    # empty lists and k beyond the candidates
    off3 = off.copy()
    keep = off[3]
    off3[4:] = keep  # lists 3.. are empty, only the first three keep their vectors
    ix3 = oracle.Index(ix.centroids, ix.codebooks, codes[:keep], off3, ids[:keep], "l2")
    i3, d3 = oracle.ivfpq_search(ix3, q, 32, int(keep) + 5)
    assert (i3[:, keep:] == -1).all() and np.isposinf(d3[:, keep:]).all()
    assert (np.sort(i3[:, :keep], axis=1) == np.sort(ids[:keep])[None]).all()


def test_bad_arguments_are_refused():
    data = synth.make_ivfpq(50, 8, 4, 2, 2, seed=1)
    ix = host_index(oracle, data)
    with pytest.raises(ValueError):
        oracle.ivfpq_search(ix, data.queries.numpy(), 5, 3)  # nprobe > nlist
    with pytest.raises(ValueError):
        oracle.ivfpq_search(ix, data.queries.numpy(), 1, 0)


def _decoded_vectors(data):
    lab, resid, cen = _decode_all(data)
    return cen[lab] + resid


@pytest.mark.parametrize("metric", ["l2", "ip"])
def test_sharded_full_probe_equals_bruteforce_over_the_union_of_shards(metric):
    """Independent indexes per shard, results aggregated (paper, Sec. 4, retrieval model): with every
    list of every shard probed, the aggregate is the exact kNN over all decoded vectors of all
    shards, whichever shard holds them."""
    S, k = 3, 17
    shards = synth.make_ivfpq_shards(S, 700, 16, 8, 4, 6, metric=metric, seed=77)
    q = shards[0].queries.double().numpy()
    got_i, got_d = oracle.sharded_search([host_index(oracle, sh) for sh in shards], shards[0].queries.numpy(), 8, k)
    y = np.concatenate([_decoded_vectors(sh) for sh in shards])
    ids = np.concatenate([sh.ids.numpy() for sh in shards])
    assert np.unique(ids).size == ids.size
    if metric == "l2":
        s = ((q[:, None, :] - y[None]) ** 2).sum(2)
        order = np.argsort(s, axis=1, kind="stable")[:, :k]
    else:
        s = q @ y.T
        order = np.argsort(-s, axis=1, kind="stable")[:, :k]
    assert np.array_equal(got_i, ids[order])
    assert np.allclose(got_d, np.take_along_axis(s, order, 1), rtol=2e-6, atol=1e-6)
    # every shard contributes to some query's answer, so no part is dropped silently
    assert set(np.unique(got_i // 700)) == set(range(S))


def test_merge_results_by_hand():
    """Two shards, two queries, worked by hand: padding is skipped, ties go to the smaller id, short
    unions are padded."""
    inf = np.inf
    ids = np.array([[[5, 9, -1], [4, -1, -1]],
                    [[7, 2, 8], [-1, -1, -1]]], np.int64)
    l2 = np.array([[[0.5, 2.0, inf], [1.0, inf, inf]],
                   [[0.25, 2.0, 3.0], [inf, inf, inf]]], np.float32)
    oi, od = oracle.merge_results(ids, l2, 4, "l2")
    assert oi.tolist() == [[7, 5, 2, 9], [4, -1, -1, -1]]
    assert od[0].tolist() == [0.25, 0.5, 2.0, 2.0] and od[1, 0] == 1.0 and np.isposinf(od[1, 1:]).all()
    ip = np.where(np.isinf(l2), -inf, -l2).astype(np.float32)   # same order under inner product
    oi2, od2 = oracle.merge_results(ids, ip, 2, "ip")
    assert oi2.tolist() == [[7, 5], [4, -1]] and od2[0].tolist() == [-0.25, -0.5] and np.isneginf(od2[1, 1])


@pytest.mark.parametrize("metric", ["l2", "ip"])
def test_pq4_handworked_example(metric):
    g = json.load(open(os.path.join(GOLD, "handworked_pq4.json")))
    cb = np.zeros((2, 16, 1), np.float32)
    cb[0, :, 0] = np.arange(16)
    cb[1, :, 0] = -np.arange(16)
    for case in g[metric]["cases"]:
        ids, dists = oracle.ivfpq4_search(np.asarray(g["centroids"], np.float32), cb,
                                          np.asarray(g["packed_codes"], np.uint8), g["list_offsets"], g["ids"], metric,
                                          np.asarray([g["query"]], np.float32), case["nprobe"], case["k"])
        assert ids[0].tolist() == case["ids"], case
        assert dists[0].tolist() == [_inf(v) for v in case["dists"]], case


def _pair_codebooks(cb4):
    """[M4, 16, ds] -> [M4/2, 256, 2 ds]: codeword `byte` of pair j = codeword byte & 15 of sub-space 2j followed
    by codeword byte >> 4 of sub-space 2j + 1."""
    M4, _, ds = cb4.shape
    byte = np.arange(256)
    return np.concatenate([cb4[0::2][:, byte & 15, :], cb4[1::2][:, byte >> 4, :]], axis=2).astype(np.float32)


@pytest.mark.parametrize("metric,bf16", [("l2", False), ("ip", False), ("l2", True), ("ip", True)])
def test_pq4_equals_8bit_search_over_paired_subspaces(metric, bf16):
    """A 4-bit index is an 8-bit index in disguise: pairs of sub-spaces with all 256 concatenated codewords, the
    packed byte as the code.  The numpy 4-bit definition and the 8-bit oracle (different code) must agree on it."""
    data = synth.make_ivfpq4(4000, 32, 16, 16, 9, metric=metric, seed=61, coarse_bf16=bf16)
    cen = data.centroids.view(torch.uint16).numpy() if bf16 else data.centroids.numpy()
    cb4 = data.codebooks.numpy()
    a_i, a_d = oracle.ivfpq4_search(cen, cb4, data.codes.numpy(), data.list_offsets.numpy(), data.ids.numpy(), metric,
                                    data.queries.numpy(), 5, 12, coarse_bf16=bf16)
    ix8 = oracle.Index(cen, _pair_codebooks(cb4), data.codes.numpy(), data.list_offsets.numpy(), data.ids.numpy(),
                       metric, coarse_bf16=bf16)
    b_i, b_d = oracle.ivfpq_search(ix8, data.queries.numpy(), 5, 12)
    assert np.array_equal(a_i, b_i)
    assert np.allclose(a_d, b_d, rtol=2e-6, atol=1e-6)
    # and the codes really are nibbles of the nearest codewords: unpack(pack(x)) == x
    codes = torch.randint(0, 16, (50, 8), dtype=torch.uint8)
    assert np.array_equal(oracle.unpack_pq4(synth.pack_pq4(codes).numpy()), codes.numpy())


def test_merge_results_invariants():
    """Aggregation does not depend on the order of the shards, a single shard is returned as it is (cut to k), and
    merging in two steps equals merging at once."""
    rng = np.random.default_rng(11)
    nparts, nq, k = 5, 7, 12
    d = np.sort(rng.permutation(nparts * nq * k).astype(np.float32).reshape(nparts, nq, k) * 0.5, axis=2)
    ids = rng.permutation(nparts * nq * k).astype(np.int64).reshape(nparts, nq, k)
    ids[3, :, 8:] = -1
    d[3, :, 8:] = np.inf
    a = oracle.merge_results(ids, d, k, "l2")
    perm = [4, 0, 3, 1, 2]
    b = oracle.merge_results(ids[perm], d[perm], k, "l2")
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    one = oracle.merge_results(ids[:1], d[:1], 5, "l2")
    assert np.array_equal(one[0], ids[0][:, :5]) and np.array_equal(one[1], d[0][:, :5])
    left = oracle.merge_results(ids[:2], d[:2], k, "l2")
    right = oracle.merge_results(ids[2:], d[2:], k, "l2")
    two = oracle.merge_results(np.stack([left[0], right[0]]), np.stack([left[1], right[1]]), k, "l2")
    assert np.array_equal(two[0], a[0]) and np.array_equal(two[1], a[1])
    # inner product: the same lists with the sign flipped rank the same way
    c = oracle.merge_results(ids, np.where(np.isinf(d), -np.inf, -d).astype(np.float32), k, "ip")
    assert np.array_equal(c[0], a[0])


# ---- two-level coarse quantiser ------------------------------------------------------------------------------

def _numpy_tree_probes(cen, top, off, b1, q, nprobe, metric):
    """The definition again, in numpy: best b1 nodes, then the best nprobe of their children (ties: smaller index)."""
    def score(rows):
        rows = np.asarray(rows, np.float64)
        return ((q[None, :] - rows) ** 2).sum(1) if metric == "l2" else rows @ q
    s1 = score(top)
    key1 = s1 if metric == "l2" else -s1
    nodes = np.lexsort((np.arange(len(top)), key1))[:b1]
    cand = np.concatenate([np.arange(off[n], off[n + 1]) for n in nodes])
    s2 = score(cen[cand])
    key2 = s2 if metric == "l2" else -s2
    order = np.lexsort((cand, key2))[:nprobe]
    out = np.full(nprobe, -1, np.int64)
    out[:order.size] = cand[order]
    return out


def test_tree_coarse_matches_the_hand_worked_example():
    g = json.load(open(os.path.join(GOLD, "handworked_tree.json")))
    cen = np.array(g["centroids"], np.float32)
    top = np.array(g["level1"], np.float32)
    off = np.array(g["child_offsets"], np.int32)
    for metric in ("l2", "ip"):
        q = np.array([g[metric]["query"]], np.float32)
        _, flat = oracle.coarse(cen, q, 4, metric)
        assert sorted(flat[0].tolist()) == sorted(g[metric]["list_scores"])       # the per-list values themselves
        for case in g[metric]["cases"]:
            lists, scores = oracle.coarse_tree(cen, top, off, case["b1"], q, case["nprobe"], metric)
            assert lists[0].tolist() == case["lists"], (metric, case)
            for l, s in zip(lists[0], scores[0]):
                if l >= 0:
                    assert s == g[metric]["list_scores"][l]
    lists, _ = oracle.coarse(cen, np.array([g["l2"]["query"]], np.float32), 2, "l2")
    assert lists[0].tolist() == g["l2"]["flat_nprobe2"]                         # the tree with b1 = 1 differs from it


@pytest.mark.parametrize("metric,bf16", [("l2", False), ("ip", False), ("l2", True), ("ip", True)])
def test_tree_with_every_node_kept_is_the_one_level_search(metric, bf16):
    data = synth.make_ivfpq(3000, 32, 48, 16, 9, metric=metric, seed=71, coarse_bf16=bf16)
    top, off = synth.make_coarse_tree(data.centroids, 6)
    hix = host_index(oracle, data)
    top_h = top.view(torch.uint16).numpy() if bf16 else top.numpy()
    q = data.queries.numpy()
    want_l, want_s = oracle.coarse(hix.centroids, q, 7, metric, coarse_bf16=bf16)
    got_l, got_s = oracle.coarse_tree(hix.centroids, top_h, off.numpy(), 6, q, 7, metric, coarse_bf16=bf16)
    assert np.array_equal(want_l, got_l) and np.array_equal(want_s, got_s)
    a = oracle.ivfpq_search(hix, q, 7, 12)
    b = oracle.ivfpq_search_tree(hix, top_h, off.numpy(), 6, q, 7, 12)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


@pytest.mark.parametrize("metric", ["l2", "ip"])
def test_tree_coarse_equals_its_numpy_restatement(metric):
    data = synth.make_ivfpq_hashed(2000, 24, 60, 8, 11, metric=metric, seed=72, tree_n1=10)
    cen = data.centroids.numpy()
    top, off = data.extra["level1"].numpy(), data.extra["child_offsets"].numpy()
    q = data.queries.numpy()
    for b1, nprobe in ((1, 4), (3, 9), (10, 60), (2, 20)):
        lists, _ = oracle.coarse_tree(cen, top, off, b1, q, nprobe, metric)
        for i in range(q.shape[0]):
            want = _numpy_tree_probes(cen.astype(np.float64), top, off, b1, q[i].astype(np.float64), nprobe, metric)
            assert lists[i].tolist() == want.tolist(), (metric, b1, nprobe, i)
    # narrowing the first level can only lose lists the one-level search would have probed, never invent new scores
    flat_l, flat_s = oracle.coarse(cen, q, 9, metric)
    tree_l, tree_s = oracle.coarse_tree(cen, top, off, 3, q, 9, metric)
    sgn = 1.0 if metric == "l2" else -1.0
    assert np.all(sgn * tree_s >= sgn * flat_s - 1e-12)


def test_tree_search_scans_only_the_lists_the_tree_picks():
    data = synth.make_ivfpq_hashed(4000, 32, 40, 16, 6, metric="l2", seed=73, tree_n1=8)
    hix = host_index(oracle, data)
    top, off = data.extra["level1"].numpy(), data.extra["child_offsets"].numpy()
    q = data.queries.numpy()
    ids, dists, probes = oracle.ivfpq_search_tree(hix, top, off, 2, q, 5, 10, want_probes=True)
    want_probes, _ = oracle.coarse_tree(hix.centroids, top, off, 2, q, 5, "l2")
    assert np.array_equal(probes, want_probes)
    # the same answer as a one-level search over an index in which every other list is empty
    for i in range(q.shape[0]):
        keep = set(probes[i].tolist())
        lens = np.diff(hix.offsets)
        sel = np.concatenate([np.arange(hix.offsets[l], hix.offsets[l + 1]) for l in sorted(keep)])
        new_off = np.zeros(hix.nlist + 1, np.int64)
        new_off[1:] = np.cumsum([lens[l] if l in keep else 0 for l in range(hix.nlist)])
        sub = oracle.Index(hix.centroids, hix.codebooks, hix.codes[sel], new_off, hix.ids[sel], "l2")
        a = oracle.ivfpq_search(sub, q[i:i + 1], hix.nlist, 10)
        assert np.array_equal(a[0][0], ids[i]) and np.array_equal(a[1][0], dists[i])

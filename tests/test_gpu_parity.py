"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  ids must be equal except inside distance ties; distances within
1e-4 relative (flat search: 1e-3)."""

import numpy as np
import pytest
import torch

import oracle
from paper_2503_14649_b200 import binding, synth
from tests.helpers import IvfPqRescorer, coarse_rescorer, host_index, match_results

pytestmark = pytest.mark.gpu

REL = 1e-4  # fp32 distances vs the double-precision oracle


def _gpu_search(data, nprobe, k, queries=None):
    ix = binding.load_index_from(data, "cuda")
    q = (data.queries if queries is None else queries).cuda().contiguous()
    ids, dists = ix.rago_search(q, nprobe, k)
    lists, coarse = ix.rago_search_probes(q, nprobe)
    torch.cuda.synchronize()
    ix.rago_check()
    out = ids.cpu().numpy(), dists.cpu().numpy(), lists.cpu().numpy(), coarse.cpu().numpy()
    ix.close()
    return out


def _compare(data, nprobe, k, rel=REL, max_probe_mismatch=0):
    hix = host_index(oracle, data)
    q = data.queries.cpu().numpy()
    oi, od, op = oracle.ivfpq_search(hix, q, nprobe, k, nthreads=oracle.default_threads(), want_probes=True)
    _, oc = oracle.coarse(hix.centroids, q, nprobe, data.metric, coarse_bf16=data.coarse_bf16,
                          nthreads=oracle.default_threads())
    gi, gd, gl, gc = _gpu_search(data, nprobe, k)
    bad_probe_queries = 0
    rs = IvfPqRescorer(oracle, hix)
    for i in range(q.shape[0]):
        # probe lists: same lists in the same order, except where coarse scores tie within tolerance
        if not np.array_equal(gl[i], op[i]):
            sgn = 1.0 if data.metric == "l2" else -1.0
            assert not match_results(gl[i].astype(np.int64), sgn * gc[i], op[i].astype(np.int64), sgn * oc[i], rel=rel,
                                     rescore=coarse_rescorer(oracle, hix.centroids, q[i], data.metric, data.coarse_bf16, sgn)
                                     ), ("probe order", i, gl[i], op[i])
            if set(gl[i].tolist()) != set(op[i].tolist()):
                bad_probe_queries += 1
                continue  # a different list was probed at a coarse tie: final results legitimately differ
        assert np.allclose(gc[i], oc[i], rtol=rel, atol=rel * max(1.0, np.abs(oc[i]).max())), ("coarse", i)
        sgn = 1.0 if data.metric == "l2" else -1.0
        problems = match_results(gi[i], sgn * gd[i], oi[i], sgn * od[i], rel=rel, rescore=rs.for_query(q[i], sgn))
        assert not problems, ("query %d" % i, problems[:5])
    assert bad_probe_queries <= max_probe_mismatch
    return gi, gd


CASES = [
    # N, d, nlist, M, nq, nprobe, k, metric, bf16, zipf
    (3000, 64, 16, 16, 9, 4, 10, "l2", False, None),
    (3000, 64, 16, 32, 9, 4, 10, "ip", False, None),
    (5000, 96, 12, 48, 5, 3, 17, "l2", False, None),
    (5000, 128, 20, 64, 7, 20, 33, "l2", False, None),   # nprobe = nlist
    (5000, 128, 20, 64, 7, 5, 8, "ip", True, None),
    (4000, 160, 10, 80, 3, 2, 5, "l2", False, None),
    (6000, 192, 24, 96, 11, 6, 100, "l2", False, 1.1),
    (6000, 192, 24, 96, 11, 6, 100, "ip", True, 1.1),
    (4000, 256, 8, 128, 4, 3, 12, "l2", True, None),
    (2000, 32, 8, 16, 1, 8, 1, "l2", False, None),       # nq = 1, k = 1
    (700, 48, 40, 16, 6, 40, 1024, "l2", False, None),   # k above the candidate count: padding
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "N%d_d%d_nl%d_M%d_%s%s" % (c[0], c[1], c[2], c[3], c[7],
                                                                                   "_bf16" if c[8] else ""))
def test_small_cases_match_oracle(case):
    N, d, nlist, M, nq, nprobe, k, metric, bf16, zipf = case
    data = synth.make_ivfpq(N, d, nlist, M, nq, metric=metric, seed=100 + N + M, zipf=zipf, coarse_bf16=bf16)
    _compare(data, nprobe, k)


LARGE_BATCH_CASES = [
    # N, d, nlist, M, nprobe, k, metric: batches above the limit up to which lookup tables are built by a kernel of
    # their own; beyond it every scan CTA builds the table of each query it meets
    (2500, 64, 8, 16, 2, 5, "l2"),
    (2500, 128, 8, 64, 2, 5, "ip"),     # dsub = 2: the generic table builder
    (2500, 512, 8, 64, 2, 5, "l2"),     # dsub = 8
    (2500, 384, 8, 96, 2, 5, "l2"),     # dsub = 4
]


@pytest.mark.parametrize("case", LARGE_BATCH_CASES, ids=lambda c: "d%d_M%d_%s" % (c[1], c[3], c[6]))
def test_batch_above_the_prebuilt_table_limit(case):
    N, d, nlist, M, nprobe, k, metric = case
    data = synth.make_ivfpq(N, d, nlist, M, 4200, metric=metric, seed=300 + d + M)
    _compare(data, nprobe, k, max_probe_mismatch=8)


def test_empty_lists_and_short_lists():
    data = synth.make_ivfpq(900, 64, 16, 16, 8, metric="l2", seed=5)
    # empty every other list by moving its vectors to the next one
    L = (data.list_offsets[1:] - data.list_offsets[:-1]).clone()
    for l in range(0, 16, 2):
        L[l + 1] += L[l]
        L[l] = 0
    data.list_offsets = synth.offsets_from_lengths(L)
    _compare(data, 16, 20)
    # an entirely empty index
    data0 = synth.make_ivfpq(0, 32, 4, 16, 3, metric="ip", seed=6)
    gi, gd, _, _ = _gpu_search(data0, 2, 5)
    assert (gi == -1).all() and np.isneginf(gd).all()


def test_config1_full_size():
    """Tiny IVF-PQ shape of the benchmark list, all 64 queries."""
    c = synth.CONFIGS[1]
    data = synth.make_config(1)
    _compare(data, c["nprobe"], c["k"])


def test_mid_shape_scaled_down_spans_many_tiles():
    """Mid shape (d = 768, M = 96, Zipf lists) at 1/40 of the vectors: long lists are cut into many
    tiles and split between CTAs, short ones have ragged tails."""
    data = synth.make_ivfpq(250_000, 768, 256, 96, 48, metric="l2", seed=77, zipf=1.1)
    _compare(data, 32, 100, max_probe_mismatch=1)


def test_inner_product_bf16_coarse_hashed_index():
    """Hyperscale shape in miniature: hash-coded M = 64 lists, bf16 centroids, inner product."""
    data = synth.make_ivfpq_hashed(400_000, 768, 512, 64, 32, metric="ip", seed=31, coarse_bf16=True)
    _compare(data, 64, 100, max_probe_mismatch=1)


def test_iterative_small_batches_back_to_back():
    """Latency shape in miniature: batches of 1, 4 and 16 queries issued on one stream reuse one
    workspace; each must equal the oracle's answer for its own queries."""
    data = synth.make_ivfpq_hashed(300_000, 512, 256, 32, 64, metric="l2", seed=41)
    hix = host_index(oracle, data)
    rs = IvfPqRescorer(oracle, hix)
    ix = binding.load_index_from(data, "cuda")
    q = data.queries.cuda()
    outs = []
    pos = 0
    for nb in synth.batch_size_stream(3, 12):
        outs.append((pos, nb) + ix.rago_search(q[pos:pos + nb].contiguous(), 16, 20))
        outs[-1] = (pos, nb, outs[-1][2].clone(), outs[-1][3].clone())
        pos = (pos + nb) % 40
    torch.cuda.synchronize()
    ix.rago_check()
    for pos, nb, gi, gd in outs:
        qh = data.queries[pos:pos + nb].numpy()
        oi, od = oracle.ivfpq_search(hix, qh, 16, 20)
        for i in range(nb):
            assert not match_results(gi[i].cpu().numpy(), gd[i].cpu().numpy(), oi[i], od[i], rel=REL,
                                     rescore=rs.for_query(qh[i]))
    ix.close()


SMALL_BATCH_PATHS = [
    # nq, nprobe, k, metric: batch sizes on both sides of the fused selection + plan (<= 64 queries), of the tiny-batch
    # coarse kernel (<= 16) and of its query groups (8), k on both sides of the one-warp cut (<= 32) and of the two
    # register shapes of the small-batch merge ((CTAs + 1) k <= 4 096 / 16 384) and beyond them
    (1, 40, 33, "l2"), (2, 16, 20, "l2"), (3, 4, 1, "ip"), (8, 16, 27, "ip"), (9, 16, 28, "l2"), (17, 8, 100, "ip"),
    (33, 16, 150, "l2"), (64, 32, 27, "l2"), (65, 16, 20, "ip"),
]


@pytest.mark.parametrize("nq,nprobe,k,metric", SMALL_BATCH_PATHS)
def test_small_batch_paths(nq, nprobe, k, metric):
    """The latency path's kernels change shape with the batch size and k (fused planning, one-warp cuts, ranked
    short buffers, the small-batch merge): every combination must give the oracle's answer."""
    data = synth.make_ivfpq(60_000, 128, 96, 32, nq, metric=metric, seed=500 + nq + k, zipf=1.05)
    _compare(data, nprobe, k, max_probe_mismatch=1)


def test_results_do_not_depend_on_run():
    """The shared per-query threshold makes scheduling vary between runs; results must not."""
    data = synth.make_ivfpq(120_000, 192, 64, 96, 32, metric="l2", seed=8, zipf=1.1)
    ix = binding.load_index_from(data, "cuda")
    q = data.queries.cuda()
    a = ix.rago_search(q, 16, 50)
    a = (a[0].clone(), a[1].clone())
    for _ in range(3):
        b = ix.rago_search(q, 16, 50)
        assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    ix.close()


FLAT_CASES = [(5000, 64, 7, 10), (70_000, 128, 33, 100), (3, 64, 2, 5),
              (200_000, 64, 200, 100),   # two row tiles, lists compacted while streaming
              (300_000, 64, 40, 50),     # large enough for the pilot-threshold pass
              (300_000, 64, 300, 100),   # three row tiles (a pair and a single) behind pilot thresholds
              (40_000, 64, 9, 300),      # wide candidate lists
              (30_000, 64, 5, 1000)]     # k above the fused selection: fp32-pipe fallback
# every case with one row tile per CTA; batches of more than 128 queries also with paired row tiles
FLAT_RUNS = [c + (1,) for c in FLAT_CASES] + [c + (2,) for c in FLAT_CASES if c[2] > 128] + \
            [c + (3,) for c in FLAT_CASES if c[2] > 128]   # 3: a cluster of two CTAs per pair of row tiles


@pytest.mark.parametrize("N,d,nq,k,pairing", FLAT_RUNS)
def test_flat_search_matches_oracle(N, d, nq, k, pairing):
    binding.rago_debug_set_gemm_pairing(pairing)
    try:
        _flat_case(N, d, nq, k)
    finally:
        binding.rago_debug_set_gemm_pairing(0)


def _flat_case(N, d, nq, k):
    db, q = synth.make_flat(N, d, nq, seed=N)
    gi, gs = binding.rago_flat_search(db.cuda(), q.cuda(), k)
    torch.cuda.synchronize()
    oi, osc = oracle.flat_search(db.view(torch.uint16).numpy(), q.view(torch.uint16).numpy(), k,
                                 nthreads=oracle.default_threads())
    gi, gs = gi.cpu().numpy(), gs.cpu().numpy()
    db_bits, q_bits = db.view(torch.uint16).numpy(), q.view(torch.uint16).numpy()
    for i in range(nq):
        def rescore(row, i=i):
            if row < 0 or row >= N:
                raise KeyError(row)
            return -float(oracle.flat_scores(db_bits, q_bits[i], np.array([row], np.int64))[0])
        assert not match_results(gi[i], -gs[i], oi[i], -osc[i], rel=1e-3, rescore=rescore), i


def test_argument_errors_are_reported_before_any_launch():
    data = synth.make_ivfpq(500, 32, 4, 16, 2, seed=1)
    ix = binding.load_index_from(data, "cuda")
    q = data.queries.cuda()
    before = binding.rago_kernel_launches()
    for kwargs in (dict(nprobe=5, k=3), dict(nprobe=0, k=3), dict(nprobe=2, k=0), dict(nprobe=2, k=2000)):
        with pytest.raises(binding.RagoError):
            ix.rago_search(q, **kwargs)
    with pytest.raises(binding.RagoError) as e:
        ix.rago_search(q, 2, 3, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4
    with pytest.raises(binding.RagoError) as e:
        ix.rago_search(torch.zeros(2 * 32 + 1, device="cuda")[1:].view(2, 32), 2, 3)  # 4-byte offset
    assert e.value.status == 2
    assert binding.rago_kernel_launches() == before
    ix.close()
    # unsupported sub-space count, non-monotone offsets
    bad = synth.make_ivfpq(500, 48, 4, 24, 2, seed=1)
    with pytest.raises(binding.RagoError) as e:
        binding.load_index_from(bad, "cuda")
    assert e.value.status == 3
    data.list_offsets = data.list_offsets.clone()
    data.list_offsets[2] = data.list_offsets[1] - 1
    with pytest.raises(binding.RagoError) as e:
        binding.load_index_from(data, "cuda")
    assert e.value.status == 1


def test_search_replays_from_a_cuda_graph():
    """rago_search only enqueues work on the caller's stream (no allocation, no synchronisation), so a call can be
    captured once and replayed; the replay must give the eager call's results."""
    data = synth.make_ivfpq(50_000, 128, 128, 32, 24, metric="l2", seed=12)
    ix = binding.load_index_from(data, "cuda")
    q = data.queries.cuda().contiguous()
    ws = torch.empty(ix.search_workspace_bytes(24, 8, 20), dtype=torch.uint8, device="cuda")
    ids = torch.empty((24, 20), dtype=torch.int64, device="cuda")
    dists = torch.empty((24, 20), dtype=torch.float32, device="cuda")
    ix.rago_search(q, 8, 20, ids, dists, ws)
    torch.cuda.synchronize()
    want_i, want_d = ids.clone(), dists.clone()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            ix.rago_search(q, 8, 20, ids, dists, ws)
    for _ in range(2):
        ids.zero_()
        dists.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(ids, want_i) and torch.equal(dists, want_d)
    ix.rago_check(ws)
    ix.close()


def test_concurrent_searches_on_two_streams_do_not_interfere():
    """Calls on one index from different streams, each with its own workspace and outputs, may overlap on the GPU:
    the index is read-only during a search and all per-call state lives in the workspace."""
    data = synth.make_ivfpq(150_000, 128, 256, 32, 96, metric="ip", seed=19, zipf=1.0)
    ix = binding.load_index_from(data, "cuda")
    qa = data.queries[:64].cuda().contiguous()
    qb = data.queries[64:].cuda().contiguous()
    want_a = [t.clone() for t in ix.rago_search(qa, 12, 30)]
    want_b = [t.clone() for t in ix.rago_search(qb, 20, 50)]
    torch.cuda.synchronize()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    wa = torch.empty(ix.search_workspace_bytes(64, 12, 30), dtype=torch.uint8, device="cuda")
    wb = torch.empty(ix.search_workspace_bytes(32, 20, 50), dtype=torch.uint8, device="cuda")
    outs_a, outs_b = [], []
    for _ in range(6):
        oa = (torch.empty((64, 30), dtype=torch.int64, device="cuda"), torch.empty((64, 30), device="cuda"))
        ob = (torch.empty((32, 50), dtype=torch.int64, device="cuda"), torch.empty((32, 50), device="cuda"))
        with torch.cuda.stream(sa):
            ix.rago_search(qa, 12, 30, oa[0], oa[1], wa)
        with torch.cuda.stream(sb):
            ix.rago_search(qb, 20, 50, ob[0], ob[1], wb)
        outs_a.append(oa)
        outs_b.append(ob)
    torch.cuda.synchronize()
    ix.rago_check(wa)
    ix.rago_check(wb)
    for oa, ob in zip(outs_a, outs_b):
        assert torch.equal(oa[0], want_a[0]) and torch.equal(oa[1], want_a[1])
        assert torch.equal(ob[0], want_b[0]) and torch.equal(ob[1], want_b[1])
    ix.close()


@pytest.mark.parametrize("k", [1000, 100])
def test_single_query_whose_best_list_is_spread_over_many_ctas(k):
    """One query, k large: every scan CTA leaves a partial top-k, and the CTAs that worked on the query's own list
    hold far more than k keys below every other CTA's best one, so the merge cannot finish from the slots' leading
    keys alone and has to select in several rounds."""
    data = synth.make_ivfpq(200_000, 32, 8, 16, 1, metric="l2", seed=23)
    cen = torch.zeros((8, 32))
    cen[1:] = 10.0 * torch.nn.functional.normalize(data.centroids[1:], dim=1)   # list 0 around the origin, the rest far
    data.centroids = cen
    data.queries = 0.01 * data.queries / data.queries.norm()
    _compare(data, 8, k)


@pytest.mark.parametrize("metric", ["l2", "ip"])
@pytest.mark.parametrize("nq", [5, 40])     # tables built ahead of the scan / inside it
def test_query_magnitudes_from_zero_to_huge(metric, nq):
    """The lookup table is fixed-point with a per-query scale: a zero query, tiny and huge queries and one with an
    empty sub-vector must all come out within tolerance."""
    data = synth.make_ivfpq(30_000, 64, 32, 16, nq, metric=metric, seed=77)
    q = data.queries.clone()
    q[0] = 0.0
    q[1] *= 1e-6
    q[2] *= 1e5
    q[3, :8] = 0.0
    q[4, 4:] = 0.0
    data.queries = q
    _compare(data, 6, 15, max_probe_mismatch=1)


def test_small_batch_with_many_probes_builds_tables_in_their_own_launch():
    """30 queries x 150 probes: few enough queries for tables built ahead of the scan, too many (query, list) pairs
    (4 500) for the single planning launch that otherwise hosts the table CTAs."""
    data = synth.make_ivfpq(60_000, 96, 256, 48, 30, metric="ip", seed=41, zipf=0.8)
    _compare(data, 150, 40, max_probe_mismatch=1)


@pytest.mark.parametrize("metric,M,d", [("l2", 16, 64), ("ip", 32, 256)])
def test_batch_beyond_the_prebuilt_table_limit_builds_tables_in_the_scan(metric, M, d):
    """More than 4 096 queries: the scan CTAs build each query's table themselves (exact largest entry for the
    fixed-point scale) instead of fetching an image built ahead."""
    data = synth.make_ivfpq(20_000, d, 64, M, 4200, metric=metric, seed=5)
    _compare(data, 4, 10, max_probe_mismatch=8)


def test_near_duplicate_queries_get_relatively_accurate_l2_distances():
    """Queries that almost coincide with a stored (decoded) vector: the true squared distance is about 1e-4 while
    the terms of the expanded form the scan ranks with are of size 100 (centroid norms near 28 at d = 768), so
    only a final score in the direct form meets a relative tolerance.  Distances are compared at 1e-4 relative
    with the usual tiny floor, i.e. the nearest neighbour's 1e-4 must be right to 1e-8."""
    data = synth.make_ivfpq(40_000, 768, 64, 96, 8, metric="l2", seed=515)
    cen, cb = data.centroids.numpy().astype(np.float64), data.codebooks.numpy().astype(np.float64)
    codes, off = data.codes.numpy(), data.list_offsets.numpy()
    g = np.random.default_rng(7)
    rows = g.choice(data.N, 24, replace=False)
    q = np.empty((24, 768), np.float32)
    for t, pos in enumerate(rows):
        lst = int(np.searchsorted(off, pos, side="right") - 1)
        decoded = cen[lst] + np.concatenate([cb[m, codes[pos, m]] for m in range(96)])
        q[t] = (decoded + 1e-3 * synth.SIGMA * g.standard_normal(768)).astype(np.float32)
    data.queries = torch.from_numpy(q)
    gi, gd = _compare(data, 8, 10)
    assert np.all(gd[:, 0] < 1e-3) and np.all(gd[:, 0] > 0)           # the near-duplicate itself, far below the terms
    assert np.array_equal(gi[:, 0], data.ids.numpy()[rows])


@pytest.mark.parametrize("mode", [1, 2])
def test_thousands_of_identical_centroids_do_not_displace_a_closer_list(mode):
    """2500 coarse centroids are the same vector, so their scores tie bit for bit and the tie group is larger than
    the selection buffer; one further list is strictly closer to each query.  The closer list must always be
    probed first, and the fp32-pipe path fills the rest with the smallest list numbers, as the oracle does."""
    data = synth.make_ivfpq(2000, 32, 3000, 16, 4, metric="l2", seed=90)
    g = torch.Generator().manual_seed(5)
    data.centroids[:2500] = data.centroids[0]
    data.queries = data.centroids[0][None, :] + 0.05 * torch.randn((4, 32), generator=g)
    for i in range(4):
        data.centroids[2700 + i] = data.queries[i]
    hix = host_index(oracle, data)
    q = data.queries.numpy()
    ol, oc = oracle.coarse(hix.centroids, q, 16, "l2")
    for i in range(4):
        assert ol[i].tolist() == [2700 + i] + list(range(15))           # what the definition gives
    ix = binding.load_index_from(data, "cuda")
    ix.rago_set_coarse_mode(mode)
    for _ in range(3):                                                     # the same answer every time
        gl, gc = ix.rago_search_probes(data.queries.cuda().contiguous(), 16)
        torch.cuda.synchronize()
        ix.rago_check()
        gl, gc = gl.cpu().numpy(), gc.cpu().numpy()
        for i in range(4):
            assert gl[i][0] == 2700 + i and gc[i][0] < 1e-9
            assert np.all(gl[i][1:] < 2500) and len(set(gl[i].tolist())) == 16
            assert np.allclose(gc[i][1:], oc[i][1:], rtol=REL)
            if mode == 1:
                assert gl[i].tolist() == ol[i].tolist()
    ix.close()


# ---- 64-byte codes (the Hyperscale code size) on shapes that stress list boundaries and ties ----

CODES64_CASES = [
    # N, d, nlist, nq, nprobe, k, metric, bf16, zipf, hashed
    (60_000, 128, 40, 9, 6, 10, "l2", False, None, False),      # ragged lists (lengths not multiples of 8)
    (60_000, 256, 64, 33, 64, 100, "ip", True, None, True),     # every list probed, bf16 quantiser, k = 100
    (300, 64, 50, 5, 20, 160, "l2", False, None, False),        # lists of a handful of vectors, padding in the results
    (400_000, 768, 96, 20, 24, 100, "l2", False, 1.1, False),   # long skewed lists: many tiles per pair
    (250_000, 64, 7, 1, 7, 50, "ip", False, None, True),        # one query whose lists are spread over all CTAs
]


@pytest.mark.parametrize("case", CODES64_CASES, ids=lambda c: "N%d_d%d_nl%d_nq%d_np%d_k%d_%s" % (c[0], c[1], c[2], c[3], c[4], c[5], c[6]))
def test_64_byte_codes(case):
    N, d, nlist, nq, nprobe, k, metric, bf16, zipf, hashed = case
    if hashed:
        data = synth.make_ivfpq_hashed(N, d, nlist, 64, nq, metric=metric, seed=600 + nlist, coarse_bf16=bf16)
    else:
        data = synth.make_ivfpq(N, d, nlist, 64, nq, metric=metric, seed=600 + nlist, coarse_bf16=bf16, zipf=zipf)
    _compare(data, nprobe, k, max_probe_mismatch=1)


@pytest.mark.parametrize("k", [100, 10])  # the CTA-wide cut / the one-warp cut of small k
def test_thousands_of_identical_vectors_still_give_k_distinct_results(k):
    """Every vector of the probed lists has the same code, so all scores tie: the buffer cuts and the merge must
    still return k distinct vectors of the right score, run after run."""
    data = synth.make_ivfpq(50_000, 64, 8, 64, 3, metric="l2", seed=77)
    data.codes[:] = data.codes[0]
    ix = binding.load_index_from(data, "cuda")
    q = data.queries.cuda().contiguous()
    first = None
    for _ in range(3):
        ids, dists = ix.rago_search(q, 4, k)
        torch.cuda.synchronize()
        ix.rago_check()
        ids, dists = ids.cpu().numpy(), dists.cpu().numpy()
        for i in range(3):
            assert len(set(ids[i].tolist())) == k and ids[i].min() >= 0
            assert np.all(np.diff(dists[i]) >= 0)
        first = dists if first is None else first
        assert np.array_equal(first, dists)
    hix = host_index(oracle, data)
    oi, od = oracle.ivfpq_search(hix, data.queries.numpy(), 4, k)
    rs = IvfPqRescorer(oracle, hix)
    for i in range(3):
        assert not match_results(ids[i], dists[i], oi[i], od[i], rel=REL, rescore=rs.for_query(data.queries[i].numpy())), i
    ix.close()

"""Parity at the full sizes of the benchmark shapes, in the launch configuration bench.py times.

The oracle cannot hold a billion vectors, so each IVF-PQ test checks a sample of at least 64 queries, each of
them through ALL of the lists it probes: the oracle runs on exactly those inverted lists (regenerated on the CPU
from the seed for the hash-coded shapes).  The flat test scores 16 queries against all ten million rows with the
oracle, the database streamed to the host chunk by chunk.
"""

import gc

import numpy as np
import pytest
import torch

import oracle
from paper_2503_14649_b200 import binding, synth
from tests.helpers import IvfPqRescorer, compact_hashed_subindex, host_index, match_results

pytestmark = pytest.mark.gpu

REL = 1e-4


def _free():
    gc.collect()
    torch.cuda.empty_cache()


def _need_gb(gb):
    free, _ = torch.cuda.mem_get_info()
    if free < gb * (1 << 30):
        pytest.skip("needs %d GB of free device memory" % gb)


def _check_sample(data, hix, q_all, sample, gi, gd, gl, nprobe, k):
    """ids / distances of the sampled queries against the oracle on `hix`; probe lists too."""
    sgn = 1.0 if data.metric == "l2" else -1.0
    q = q_all[sample].cpu().numpy()
    oi, od, op = oracle.ivfpq_search(hix, q, nprobe, k, nthreads=oracle.default_threads(), want_probes=True)
    rs = IvfPqRescorer(oracle, hix)
    for t, qi in enumerate(sample):
        if not np.array_equal(gl[qi], op[t]):
            assert set(gl[qi].tolist()) == set(op[t].tolist()), ("probe lists differ", qi)
        problems = match_results(gi[qi], sgn * gd[qi], oi[t], sgn * od[t], rel=REL, rescore=rs.for_query(q[t], sgn))
        assert not problems, ("query", qi, problems[:4])


def test_mid_full_size_sampled():
    """Mid IVF-PQ: 10 M vectors, d = 768, M = 96, Zipf lists, 1024 queries, nprobe 32, k 100."""
    _need_gb(20)
    c = synth.CONFIGS[2]
    data = synth.make_config(2, device="cuda")
    ix = binding.rago_index_load(data.centroids, data.codebooks, data.codes, data.list_offsets.cuda(), data.ids,
                                 data.metric)
    q = data.queries.contiguous()
    ids, dists = ix.rago_search(q, c["nprobe"], c["k"])
    lists, _ = ix.rago_search_probes(q, c["nprobe"])
    torch.cuda.synchronize()
    ix.rago_check()
    gi, gd, gl = ids.cpu().numpy(), dists.cpu().numpy(), lists.cpu().numpy()
    ix.close()
    hix = host_index(oracle, data)
    sample = list(range(0, c["nq"], 8))  # 128 of the 1024 queries
    _check_sample(data, hix, data.queries, sample, gi, gd, gl, c["nprobe"], c["k"])
    del data, ix, q, ids, dists, lists
    _free()


def test_hyperscale_full_size_sampled():
    """Hyperscale shape: 1e9 hash-coded vectors (64 GB of codes), 65 536 bf16 centroids, inner product."""
    _need_gb(100)
    c = synth.CONFIGS[3]
    data = synth.make_config(3, device="cuda")
    ix = binding.rago_index_load(data.centroids, data.codebooks, data.codes, data.list_offsets.cuda(), data.ids,
                                 data.metric)
    q = data.queries.contiguous()
    ids, dists = ix.rago_search(q, c["nprobe"], c["k"])
    lists, _ = ix.rago_search_probes(q, c["nprobe"])
    torch.cuda.synchronize()
    ix.rago_check()
    gi, gd, gl = ids.cpu().numpy(), dists.cpu().numpy(), lists.cpu().numpy()
    sample = list(range(0, c["nq"], 64)) + [4095]  # 65 of the 4096 queries
    small = [0, 1023, 2048, 4095]
    # four queries as a batch of their own: the small-batch path (tables built ahead of the scan)
    qs = q[small].contiguous()
    ids4, dists4 = ix.rago_search(qs, c["nprobe"], c["k"])
    lists4, _ = ix.rago_search_probes(qs, c["nprobe"])
    torch.cuda.synchronize()
    ix.rago_check()
    gi4, gd4, gl4 = ids4.cpu().numpy(), dists4.cpu().numpy(), lists4.cpu().numpy()
    ix.close()
    # the lists the ORACLE's coarse step picks for the sampled queries (nothing here comes from the device)
    cen_h = data.centroids.cpu().view(torch.uint16).numpy()
    want_lists, _ = oracle.coarse(cen_h, data.queries[sorted(set(sample + small))].cpu().numpy(), c["nprobe"], data.metric,
                                  coarse_bf16=True, nthreads=oracle.default_threads())
    hix = compact_hashed_subindex(oracle, data, np.unique(want_lists))
    _check_sample(data, hix, data.queries, sample, gi, gd, gl, c["nprobe"], c["k"])
    _check_sample(data, hix, data.queries[small], [0, 1, 2, 3], gi4, gd4, gl4, c["nprobe"], c["k"])
    del data, ix, q, ids, dists, lists
    _free()


def test_iterative_stream_full_size_sampled():
    """Iterative-retrieval shape: 1e8 vectors, 256 batches of 1, 4 or 16 queries back to back on one stream."""
    _need_gb(12)
    c = synth.CONFIGS[4]
    data = synth.make_config(4, device="cuda", nq=16 * 256)
    ix = binding.rago_index_load(data.centroids, data.codebooks, data.codes, data.list_offsets.cuda(), data.ids,
                                 data.metric)
    sizes = synth.batch_size_stream(data.seed, 256)
    ws = torch.empty(ix.search_workspace_bytes(16, c["nprobe"], c["k"]), dtype=torch.uint8, device="cuda")
    qd = data.queries.contiguous()
    outs, pos = [], 0
    for nb in sizes:
        qb = qd[pos:pos + nb]
        oi = torch.empty((nb, c["k"]), dtype=torch.int64, device="cuda")
        od = torch.empty((nb, c["k"]), dtype=torch.float32, device="cuda")
        ix.rago_search(qb, c["nprobe"], c["k"], oi, od, ws)  # one workspace, one stream, no sync in between
        outs.append((pos, nb, oi, od))
        pos += nb
    torch.cuda.synchronize()
    ix.rago_check(ws)
    picked = list(range(0, 256, 8)) + [37, 255]  # 34 of the 256 batches: well over 64 queries
    assert sum(sizes[b] for b in picked) >= 64
    probes = {}
    for b in picked:
        p0, nb, _, _ = outs[b]
        probes[b] = ix.rago_search_probes(qd[p0:p0 + nb].contiguous(), c["nprobe"])[0].cpu().numpy()
    ix.close()
    qpick = np.concatenate([np.arange(outs[b][0], outs[b][0] + outs[b][1]) for b in picked])
    want_lists, _ = oracle.coarse(data.centroids.cpu().numpy(), data.queries[qpick].cpu().numpy(), c["nprobe"], data.metric,
                                  nthreads=oracle.default_threads())
    hix = compact_hashed_subindex(oracle, data, np.unique(want_lists))
    rs = IvfPqRescorer(oracle, hix)
    for b in picked:
        p0, nb, oi, od = outs[b]
        qh = data.queries[p0:p0 + nb].cpu().numpy()
        ri, rd, rp = oracle.ivfpq_search(hix, qh, c["nprobe"], c["k"], nthreads=oracle.default_threads(), want_probes=True)
        gi, gd = oi.cpu().numpy(), od.cpu().numpy()
        for i in range(nb):
            assert set(probes[b][i].tolist()) == set(rp[i].tolist()), ("probe lists differ", b, i)
            problems = match_results(gi[i], gd[i], ri[i], rd[i], rel=REL, rescore=rs.for_query(qh[i]))
            assert not problems, ("batch", b, "query", i, problems[:4])
    del data, ix, qd, outs, ws
    _free()


def test_iterative_stream_with_two_level_quantiser_full_size_sampled():
    """The iterative-retrieval shape (1e8 vectors, 16 384 lists) with a level of 128 nodes above the coarse
    centroids, 8 nodes kept: 64 single-query searches and 8 batches of 16 against the oracle's two-level search."""
    _need_gb(12)
    c = synth.CONFIGS[4]
    data = synth.make_config(4, device="cuda", nq=192, tree_n1=128)
    ix = binding.rago_index_load(data.centroids, data.codebooks, data.codes, data.list_offsets.cuda(), data.ids,
                                 data.metric)
    top, off = data.extra["level1"].cuda(), data.extra["child_offsets"].cuda()
    ix.rago_index_set_coarse_tree(top, off, 8)
    qd = data.queries.contiguous()
    ws = torch.empty(ix.search_workspace_bytes(16, c["nprobe"], c["k"]), dtype=torch.uint8, device="cuda")
    outs = []
    batches = [(i, 1) for i in range(64)] + [(64 + 16 * j, 16) for j in range(8)]
    for p0, nb in batches:
        oi = torch.empty((nb, c["k"]), dtype=torch.int64, device="cuda")
        od = torch.empty((nb, c["k"]), dtype=torch.float32, device="cuda")
        ix.rago_search(qd[p0:p0 + nb], c["nprobe"], c["k"], oi, od, ws)
        outs.append((oi, od))
    torch.cuda.synchronize()
    ix.rago_check(ws)
    ix.close()
    qh = data.queries.cpu().numpy()
    top_h, off_h = data.extra["level1"].cpu().numpy(), data.extra["child_offsets"].cpu().numpy()
    want_lists, _ = oracle.coarse_tree(data.centroids.cpu().numpy(), top_h, off_h, 8, qh, c["nprobe"], data.metric,
                                       nthreads=oracle.default_threads())
    hix = compact_hashed_subindex(oracle, data, np.unique(want_lists))
    ri, rd = oracle.ivfpq_search_tree(hix, top_h, off_h, 8, qh, c["nprobe"], c["k"], nthreads=oracle.default_threads())
    rs = IvfPqRescorer(oracle, hix)
    for (p0, nb), (oi, od) in zip(batches, outs):
        gi, gd = oi.cpu().numpy(), od.cpu().numpy()
        for i in range(nb):
            problems = match_results(gi[i], gd[i], ri[p0 + i], rd[p0 + i], rel=REL, rescore=rs.for_query(qh[p0 + i]))
            assert not problems, ("query", p0 + i, problems[:4])
    del data, ix, qd, outs, ws
    _free()


def test_flat_full_size_against_the_whole_database():
    """Flat search at 10 M x 1024 bf16: 16 of the 256 queries scored by the oracle against every row.  The database
    goes to the host one chunk at a time; the oracle's best k of every chunk are merged on the host (best first, ties
    to the smaller row), which is the exact answer over all rows."""
    _need_gb(30)
    c = synth.CONFIGS[5]
    k = c["k"]
    db, q = synth.make_flat(c["N"], c["d"], c["nq"], device="cuda")
    gi_t, gs_t = binding.rago_flat_search(db, q, k)
    torch.cuda.synchronize()
    gi, gs = gi_t.cpu().numpy(), gs_t.cpu().numpy()
    sample = list(range(0, c["nq"], 16))  # 16 queries: one per host core where there are 16
    qbits = q.cpu().view(torch.uint16).numpy()[sample]
    chunk = 1_000_000
    best_i = [np.zeros(0, np.int64) for _ in sample]
    best_s = [np.zeros(0, np.float32) for _ in sample]
    for r0 in range(0, c["N"], chunk):
        bits = db[r0:r0 + chunk].cpu().view(torch.uint16).numpy()
        ci, cs = oracle.flat_search(bits, qbits, k, nthreads=oracle.default_threads())
        for t in range(len(sample)):
            ids = np.concatenate([best_i[t], ci[t] + r0])
            sc = np.concatenate([best_s[t], cs[t]])
            order = np.lexsort((ids, -sc.astype(np.float64)))[:k]
            best_i[t], best_s[t] = ids[order], sc[order]
        del bits
    for t, qi in enumerate(sample):
        assert np.all(np.diff(gs[qi]) <= 0), qi                                # best first

        def rescore(row, t=t):
            if row < 0 or row >= c["N"]:
                raise KeyError(row)
            rb = db[row:row + 1].cpu().view(torch.uint16).numpy()
            return -float(oracle.flat_scores(rb, qbits[t], np.array([0], np.int64))[0])
        problems = match_results(gi[qi], -gs[qi], best_i[t], -best_s[t], rel=1e-3, rescore=rescore)
        assert not problems, (qi, problems[:4])
    del db, q, gi_t, gs_t
    _free()

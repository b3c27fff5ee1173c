"""Parity at the full sizes of the benchmark shapes, in the launch configuration bench.py times.

The oracle cannot search a billion vectors, so each test checks a sample: a few queries of the batch
against the oracle run on exactly the inverted lists those queries probe (regenerated on the CPU from
the seed for the hash-coded shapes), and for flat search the returned rows' exact scores plus the
absence of better rows in a sampled part of the database.
"""

import gc

import numpy as np
import pytest
import torch

import oracle
from paper_2503_14649_b200 import binding, synth
from tests.helpers import compact_hashed_subindex, host_index, match_results

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
    for t, qi in enumerate(sample):
        if not np.array_equal(gl[qi], op[t]):
            assert set(gl[qi].tolist()) == set(op[t].tolist()), ("probe lists differ", qi)
        assert not match_results(gi[qi], sgn * gd[qi], oi[t], sgn * od[t], rel=REL), ("query", qi)


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
    sample = list(range(0, c["nq"], 32))  # 32 of the 1024 queries
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
    sample = [0, 1023, 2048, 4095]
    # the same four queries as a batch of their own: the small-batch path (tables built ahead of the scan)
    qs = q[sample].contiguous()
    ids4, dists4 = ix.rago_search(qs, c["nprobe"], c["k"])
    lists4, _ = ix.rago_search_probes(qs, c["nprobe"])
    torch.cuda.synchronize()
    ix.rago_check()
    gi4, gd4, gl4 = ids4.cpu().numpy(), dists4.cpu().numpy(), lists4.cpu().numpy()
    ix.close()
    hix = compact_hashed_subindex(oracle, data, np.unique(gl[sample]))
    _check_sample(data, hix, data.queries, sample, gi, gd, gl, c["nprobe"], c["k"])
    _check_sample(data, hix, data.queries[sample], [0, 1, 2, 3], gi4, gd4, gl4, c["nprobe"], c["k"])
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
    picked = [0, 37, 128, 255]
    probes = {}
    for b in picked:
        p0, nb, _, _ = outs[b]
        probes[b] = ix.rago_search_probes(qd[p0:p0 + nb].contiguous(), c["nprobe"])[0].cpu().numpy()
    ix.close()
    hix = compact_hashed_subindex(oracle, data, np.unique(np.concatenate([probes[b].ravel() for b in picked])))
    for b in picked:
        p0, nb, oi, od = outs[b]
        qh = data.queries[p0:p0 + nb].cpu().numpy()
        ri, rd, rp = oracle.ivfpq_search(hix, qh, c["nprobe"], c["k"], nthreads=oracle.default_threads(), want_probes=True)
        gi, gd = oi.cpu().numpy(), od.cpu().numpy()
        for i in range(nb):
            assert set(probes[b][i].tolist()) == set(rp[i].tolist()), ("probe lists differ", b, i)
            assert not match_results(gi[i], gd[i], ri[i], rd[i], rel=REL), ("batch", b, "query", i)
    del data, ix, qd, outs, ws
    _free()


def test_flat_full_size_sampled():
    """Flat search at 10 M x 1024 bf16: exact scores of the returned rows, and no better row in two samples."""
    _need_gb(30)
    c = synth.CONFIGS[5]
    db, q = synth.make_flat(c["N"], c["d"], c["nq"], device="cuda")
    gi_t, gs_t = binding.rago_flat_search(db, q, c["k"])
    torch.cuda.synchronize()
    gi, gs = gi_t.cpu().numpy(), gs_t.cpu().numpy()
    qbits = q.cpu().view(torch.uint16).numpy()
    g = np.random.default_rng(5)
    rnd_rows = np.sort(g.choice(c["N"], 20_000, replace=False)).astype(np.int64)
    rnd_bits = db[torch.from_numpy(rnd_rows).cuda()].cpu().view(torch.uint16).numpy()
    pre_n = 100_000
    pre_bits = db[:pre_n].cpu().view(torch.uint16).numpy()
    for qi in (0, 100, 255):
        rows = gi[qi]
        assert len(set(rows.tolist())) == c["k"] and rows.min() >= 0 and rows.max() < c["N"]
        got_bits = db[torch.from_numpy(rows).cuda()].cpu().view(torch.uint16).numpy()
        exact = oracle.flat_scores(got_bits, qbits[qi], np.arange(c["k"], dtype=np.int64))
        assert np.allclose(gs[qi], exact, rtol=1e-3, atol=1e-6), qi           # reported scores are the rows' scores
        assert np.all(np.diff(gs[qi]) <= 0), qi                                # best first
        kth = float(gs[qi][-1])
        tol = 1e-3 * abs(kth) + 1e-6
        inres = set(rows.tolist())
        # a random sample of the database and a contiguous prefix: nothing outside the result beats the k-th
        s_rnd = oracle.flat_scores(rnd_bits, qbits[qi], np.arange(len(rnd_rows), dtype=np.int64))
        for r, sc in zip(rnd_rows, s_rnd):
            assert sc <= kth + tol or int(r) in inres, (qi, int(r), sc, kth)
        pi, ps = oracle.flat_search(pre_bits, qbits[qi:qi + 1], c["k"], nthreads=oracle.default_threads())
        for r, sc in zip(pi[0], ps[0]):
            assert sc <= kth + tol or int(r) in inres, (qi, int(r), float(sc), kth)
    del db, q, gi_t, gs_t
    _free()

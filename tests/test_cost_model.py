"""Retrieval cost model and schedule search (paper Sec. 4 retrieval model; Sec. 6.2 Algorithm 1): CPU-only checks
against closed forms, the paper's own printed figures, and a brute-force enumeration written separately."""

import math

import numpy as np

from oracle import schedule as brute
from paper_2503_14649_b200 import cost_model as cm


def test_scan_operator_is_the_larger_of_the_compute_and_memory_legs():
    # 18 GB scanned by one thread at 18 GB/s: one second, whatever the memory system
    assert cm.scan_operator_time(18e9, 1, 18e9, 24, 368e9) == 1.0
    # 24 queries on 24 threads: compute leg 1/24 s, memory leg 18/368 s: memory decides
    assert math.isclose(cm.scan_operator_time(18e9, 24, 18e9, 24, 368e9), 18e9 / 368e9)
    # more queries than threads do not add compute throughput
    assert cm.scan_operator_time(18e9, 100, 1e9, 4, 1e12) == 18e9 / 4e9
    assert cm.scan_operator_time(0.0, 8, 1e9, 4, 1e12) == 0.0
    # levels of a tree add up
    assert math.isclose(cm.tree_search_time([1e9, 2e9], 1, 1e9, 1, 1e12), 3.0)


def test_bytes_model_reproduces_the_papers_batch_one_latency():
    """The paper's database: 64e9 vectors of 96 bytes, 0.1% scanned per query (Sec. 4, methodology), sharded over
    32 servers, one thread per query at the calibrated 18 GB/s: the paper's evaluation quotes about 10 ms of
    retrieval latency at batch size one for that set-up."""
    per_query = cm.retrieval_bytes_per_query(64e9, 96, 0.1)
    assert per_query == 64e9 * 96 * 1e-3
    t = cm.scan_operator_time(per_query / 32, 1, 18e9, 96, 0.8 * 460e9)
    assert 0.009 < t < 0.012
    assert math.isclose(64e9 * 96 / 2 ** 40, 5.59, rel_tol=2e-3)   # the 5.6 TiB the paper states for the PQ codes


def test_fit_recovers_the_constants_it_was_generated_from():
    Q = np.array([1, 2, 4, 8, 16, 32, 64, 128, 256, 512, 1024], np.float64)
    D = Q * 40e6
    T = 90e-6 + D / 4.8e12
    m = cm.fit_retrieval_model(Q, D, T)
    assert abs(m.T0 - 90e-6) < 1e-9 and abs(m.B_mem - 4.8e12) / 4.8e12 < 1e-9
    assert not np.isfinite(m.R_q) and m.max_rel_err < 1e-9
    assert math.isclose(m.time(64, 64 * 40e6), 90e-6 + 64 * 40e6 / 4.8e12)
    # rows whose lists are almost empty (bytes no longer follow the batch size): a per-query rate shows
    Q2 = np.concatenate([Q, Q])
    D2 = np.concatenate([D, np.full_like(D, 1e3)])
    T2 = 90e-6 + np.maximum(D2 / 4.8e12, Q2 / 2.0e6)
    m2 = cm.fit_retrieval_model(Q2, D2, T2)
    assert np.isfinite(m2.R_q) and 1.0e6 < m2.R_q < 4.0e6


def test_pareto_front_keeps_only_non_dominated_points():
    pts = [(1.0, 1.0), (2.0, 3.0), (2.5, 2.0), (3.0, 3.0), (4.0, 5.0)]
    assert cm.pareto_front(pts, lambda p: p) == [(1.0, 1.0), (2.0, 3.0), (4.0, 5.0)]


def _toy_stages():
    """Four stages with differently shaped scaling: a small encoder, retrieval on servers, prefix, decode."""
    def encoder(r, b):
        lat = 0.002 + 0.001 * b / r
        return lat, b / lat

    def retrieval(r, b):
        lat = 0.0001 + 0.004 * b / r
        return lat, b / lat

    def prefix(r, b):
        lat = 0.010 + 0.020 * b / min(r, 8) + 0.001 * r      # communication grows with chips
        return lat, b / lat

    def decode(r, b):
        lat = 0.5 + 0.002 * b / r
        return lat, b / lat
    return [("encode", "inference", True, encoder), ("retrieve", "retrieval", False, retrieval),
            ("prefix", "inference", True, prefix), ("decode", "decode", False, decode)]


def test_placement_keeps_retrieval_and_decode_apart():
    st = [cm.Stage(n, k, p, c) for n, k, c, p in _toy_stages()]
    opts = cm.placement_options(st)
    assert opts == [[[0], [1], [2], [3]]]           # retrieval sits between the two inference stages: nothing to merge
    st3 = [cm.Stage("rewrite", "inference", lambda r, b: (1.0, 1.0)), cm.Stage("rerank", "inference", lambda r, b: (1.0, 1.0)),
           cm.Stage("prefix", "inference", lambda r, b: (1.0, 1.0)), cm.Stage("decode", "decode", lambda r, b: (1.0, 1.0), False)]
    got = sorted(map(str, cm.placement_options(st3)))
    want = sorted(map(str, [[[0], [1], [2], [3]], [[0, 1], [2], [3]], [[0], [1, 2], [3]], [[0, 1, 2], [3]]]))
    assert got == want


def _frontier_values(front):
    return sorted((round(t, 10), round(q, 10)) for t, q in front)


def test_search_equals_brute_force_enumeration():
    toys = _toy_stages()
    st = [cm.Stage(n, k, p, c) for n, k, c, p in toys]
    res = cm.search_schedules(st, chip_budget=16, retrieval_servers=[1, 2, 4], batches=[1, 2, 4, 8, 16])
    all_s = brute.enumerate_schedules(toys, 16, [1, 2, 4, 8, 16], [1, 2, 4], [1, 2, 4, 8, 16])
    want = brute.frontier(all_s)
    assert len(all_s) > 10_000
    assert _frontier_values((s.ttft, s.qps_per_chip) for s in res) == _frontier_values((s[0], s[1]) for s in want)
    assert len(res) >= 3                                                 # a real trade-off curve, not one point
    assert all(s.chips <= 16 for s in res)


def test_search_with_collocation_equals_brute_force():
    def rewrite(r, b):
        lat = 0.004 + 0.010 * b / r
        return lat, b / lat

    def rerank(r, b):
        lat = 0.001 + 0.003 * b / r
        return lat, b / lat

    def prefix(r, b):
        lat = 0.008 + 0.030 * b / r
        return lat, b / lat
    toys = [("rewrite", "inference", True, rewrite), ("rerank", "inference", True, rerank),
            ("prefix", "inference", True, prefix)]
    st = [cm.Stage(n, k, p, c) for n, k, c, p in toys]
    res = cm.search_schedules(st, chip_budget=8, retrieval_servers=[1], batches=[1, 4, 16])
    want = brute.frontier(brute.enumerate_schedules(toys, 8, [1, 2, 4, 8], [1], [1, 4, 16]))
    assert _frontier_values((s.ttft, s.qps_per_chip) for s in res) == _frontier_values((s[0], s[1]) for s in want)
    assert any(len(g) > 1 for s in res for g in s.groups)               # some frontier point collocates stages


def test_retrieval_stage_from_a_fitted_model_shards_the_bytes():
    m = cm.RetrievalModel(T0=100e-6, B_mem=5e12, R_q=float("inf"))
    st = cm.retrieval_stage("retrieve", m, bytes_per_query=62.5e6)
    lat1, thr1 = st.perf(1, 64)
    lat4, thr4 = st.perf(4, 64)
    assert math.isclose(lat1, 100e-6 + 64 * 62.5e6 / 5e12) and math.isclose(thr1, 64 / lat1)
    assert math.isclose(lat4, 100e-6 + 16 * 62.5e6 / 5e12) and thr4 > thr1

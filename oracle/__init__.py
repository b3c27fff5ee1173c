"""ctypes front end of the CPU oracle (oracle/rago_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's cpu_baseline / reference arm.  The product package never imports
this module, and this module never imports the product package.

Inputs and outputs are numpy arrays (bf16 data travels as uint16 bit
patterns).  `build()` compiles the shared object with g++ when it is missing
or older than its source.
"""

from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rago_oracle.cpp")
_LIB = os.path.join(_HERE, "librago_oracle.so")
_lib = None

L2, IP = 0, 1
_METRIC = {"l2": L2, "ip": IP, L2: L2, IP: IP}


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def default_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return os.cpu_count() or 1


class Index:
    """Borrowed views of an IVF-PQ index in host memory."""

    def __init__(self, centroids, codebooks, codes, list_offsets, ids, metric, coarse_bf16=False):
        self.coarse_bf16 = bool(coarse_bf16)
        self.centroids = _c(centroids, np.uint16 if coarse_bf16 else np.float32)
        self.codebooks = _c(codebooks, np.float32)
        self.codes = _c(codes, np.uint8)
        self.offsets = _c(list_offsets, np.int64)
        self.ids = _c(ids, np.int64)
        self.metric = _METRIC[metric]
        self.nlist, self.d = self.centroids.shape
        self.M = self.codebooks.shape[0]
        assert self.codebooks.shape == (self.M, 256, self.d // self.M)
        self.N = int(self.offsets[-1])
        assert self.codes.shape == (self.N, self.M) and self.ids.shape == (self.N,)

    def _head(self):
        return (_p(self.centroids), ctypes.c_int(self.coarse_bf16), _p(self.codebooks), _p(self.codes))


def coarse(centroids, queries, nprobe, metric, coarse_bf16=False, nthreads=1):
    cen = _c(centroids, np.uint16 if coarse_bf16 else np.float32)
    q = _c(queries, np.float32)
    nq, d = q.shape
    lists = np.empty((nq, nprobe), np.int32)
    scores = np.empty((nq, nprobe), np.float64)
    rc = lib().oracle_coarse(_p(cen), ctypes.c_int(bool(coarse_bf16)), d, cen.shape[0], _METRIC[metric], _p(q), nq,
                             nprobe, _p(lists), _p(scores), nthreads)
    if rc:
        raise ValueError("oracle_coarse: bad arguments")
    return lists, scores


def ivfpq_search(ix: Index, queries, nprobe, k, nthreads=1, want_probes=False):
    q = _c(queries, np.float32)
    nq = q.shape[0]
    ids = np.empty((nq, k), np.int64)
    dists = np.empty((nq, k), np.float32)
    probes = np.empty((nq, nprobe), np.int32) if want_probes else None
    rc = lib().oracle_ivfpq_search(*ix._head(), _p(ix.offsets), _p(ix.ids), ctypes.c_int64(ix.N), ix.d, ix.nlist,
                                   ix.M, ix.metric, _p(q), nq, nprobe, k, _p(ids), _p(dists), _p(probes), nthreads)
    if rc:
        raise ValueError("oracle_ivfpq_search: bad arguments")
    return (ids, dists, probes) if want_probes else (ids, dists)


def coarse_tree(centroids, level1, child_offsets, b1, queries, nprobe, metric, coarse_bf16=False, nthreads=1):
    """Coarse step through a two-level quantiser (see rago_oracle.cpp): the best b1 level-1 nodes, then the best
    nprobe of their children.  level1 has the storage type of `centroids`; children of node i are the consecutive
    lists child_offsets[i] .. child_offsets[i + 1] - 1.  Lists come back best first, -1 where the chosen nodes
    have fewer than nprobe children."""
    dt = np.uint16 if coarse_bf16 else np.float32
    cen, top = _c(centroids, dt), _c(level1, dt)
    off = _c(child_offsets, np.int32)
    q = _c(queries, np.float32)
    nq, d = q.shape
    lists = np.empty((nq, nprobe), np.int32)
    scores = np.empty((nq, nprobe), np.float64)
    rc = lib().oracle_coarse_tree(_p(cen), ctypes.c_int(bool(coarse_bf16)), d, cen.shape[0], _METRIC[metric], _p(top),
                                  _p(off), top.shape[0], int(b1), _p(q), nq, nprobe, _p(lists), _p(scores), nthreads)
    if rc:
        raise ValueError("oracle_coarse_tree: bad arguments")
    return lists, scores


def ivfpq_search_tree(ix: Index, level1, child_offsets, b1, queries, nprobe, k, nthreads=1, want_probes=False):
    """ivfpq_search with the probe lists chosen through the two-level quantiser."""
    top = _c(level1, np.uint16 if ix.coarse_bf16 else np.float32)
    off = _c(child_offsets, np.int32)
    q = _c(queries, np.float32)
    nq = q.shape[0]
    ids = np.empty((nq, k), np.int64)
    dists = np.empty((nq, k), np.float32)
    probes = np.empty((nq, nprobe), np.int32) if want_probes else None
    rc = lib().oracle_ivfpq_search_tree(*ix._head(), _p(ix.offsets), _p(ix.ids), ctypes.c_int64(ix.N), ix.d, ix.nlist,
                                        ix.M, ix.metric, _p(top), _p(off), top.shape[0], int(b1), _p(q), nq, nprobe, k,
                                        _p(ids), _p(dists), _p(probes), nthreads)
    if rc:
        raise ValueError("oracle_ivfpq_search_tree: bad arguments")
    return (ids, dists, probes) if want_probes else (ids, dists)


def adc_score(ix: Index, query, list_no, pos) -> float:
    q = _c(query, np.float32)
    out = ctypes.c_double()
    rc = lib().oracle_adc_score(*ix._head(), ix.d, ix.nlist, ix.M, ix.metric, _p(q), int(list_no),
                                ctypes.c_int64(int(pos)), ctypes.byref(out))
    if rc:
        raise ValueError("oracle_adc_score: bad arguments")
    return out.value


def decode_score(ix: Index, query, list_no, pos, want_decoded=False):
    q = _c(query, np.float32)
    out = ctypes.c_double()
    dec = np.empty(ix.d, np.float64) if want_decoded else None
    rc = lib().oracle_decode_score(*ix._head(), ix.d, ix.nlist, ix.M, ix.metric, _p(q), int(list_no),
                                   ctypes.c_int64(int(pos)), ctypes.byref(out), _p(dec))
    if rc:
        raise ValueError("oracle_decode_score: bad arguments")
    return (out.value, dec) if want_decoded else out.value


def flat_search(db_bits, query_bits, k, nthreads=1):
    db = _c(db_bits, np.uint16)
    q = _c(query_bits, np.uint16)
    nq, d = q.shape
    ids = np.empty((nq, k), np.int64)
    sc = np.empty((nq, k), np.float32)
    rc = lib().oracle_flat_search(_p(db), ctypes.c_int64(db.shape[0]), d, _p(q), nq, k, _p(ids), _p(sc), nthreads)
    if rc:
        raise ValueError("oracle_flat_search: bad arguments")
    return ids, sc


def flat_scores(db_bits, query_bits, rows):
    db = _c(db_bits, np.uint16)
    q = _c(query_bits, np.uint16)
    rows = _c(rows, np.int64)
    out = np.empty(rows.shape[0], np.float64)
    lib().oracle_flat_scores(_p(db), db.shape[1], _p(q), _p(rows), rows.shape[0], _p(out))
    return out


def f32_to_bf16_bits(x):
    x = _c(x, np.float32)
    out = np.empty(x.shape, np.uint16)
    lib().oracle_f32_to_bf16(_p(x), _p(out), ctypes.c_int64(x.size))
    return out


def locate(ix: Index, ident: int):
    """(list, position) of the vector with id `ident` (linear search; small inputs only)."""
    pos = int(np.nonzero(ix.ids == ident)[0][0])
    lst = int(np.searchsorted(ix.offsets, pos, side="right") - 1)
    return lst, pos


def merge_results(part_ids, part_dists, k, metric):
    """Aggregate the result lists of independently indexed database shards (paper, Sec. 4, retrieval
    performance model: every shard answers every query and the results are aggregated).

    part_ids / part_dists: [nparts][nq][k_in]; an entry with id -1 is padding.  For each query the
    union of all real entries is ordered best first (smaller L2 distance, larger inner product;
    equal scores by smaller id) and the first k are returned, padded with id -1 and +inf / -inf.
    Plain definition, one query at a time.
    """
    ids = np.asarray(part_ids, np.int64)
    dists = np.asarray(part_dists, np.float32)
    m = _METRIC[metric]
    nparts, nq, _ = ids.shape
    out_ids = np.full((nq, k), -1, np.int64)
    out_d = np.full((nq, k), np.inf if m == L2 else -np.inf, np.float32)
    for q in range(nq):
        entries = []
        for p in range(nparts):
            for ident, dist in zip(ids[p, q], dists[p, q]):
                if ident >= 0:
                    entries.append((float(dist) if m == L2 else -float(dist), int(ident), float(dist)))
        entries.sort(key=lambda e: (e[0], e[1]))
        for t, (_, ident, dist) in enumerate(entries[:k]):
            out_ids[q, t] = ident
            out_d[q, t] = dist
    return out_ids, out_d


def sharded_search(shards, queries, nprobe, k, nthreads=1):
    """Search every shard's own index with the same queries, nprobe and k, then aggregate."""
    parts = [ivfpq_search(ix, queries, nprobe, k, nthreads=nthreads) for ix in shards]
    return merge_results(np.stack([p[0] for p in parts]), np.stack([p[1] for p in parts]), k, shards[0].metric)


# ---- 4-bit product quantisation (the paper's "low-precision" PQ variant, Sec. 2: 4-bit vs 8-bit codes) ----
# Definition, in numpy fp64: each sub-space has 16 codewords, two codes share a byte (sub-space 2j in the low
# nibble of byte j, sub-space 2j + 1 in the high nibble).  Pins in tests/test_oracle_pins.py: a hand-worked
# example, brute force over the decoded vectors, and agreement with the 8-bit oracle on the index whose
# sub-spaces are the pairs and whose 256 codewords per pair are all concatenations.

def unpack_pq4(packed):
    """uint8 [N, M4/2] -> uint8 [N, M4]: code of sub-space 2j = byte j & 15, of sub-space 2j + 1 = byte j >> 4."""
    p = np.asarray(packed, np.uint8)
    out = np.empty((p.shape[0], p.shape[1] * 2), np.uint8)
    out[:, 0::2] = p & 15
    out[:, 1::2] = p >> 4
    return out


def ivfpq4_search(centroids, codebooks4, packed_codes, list_offsets, ids, metric, queries, nprobe, k,
                  coarse_bf16=False):
    """IVF-PQ search with 4-bit codes.  centroids fp32 [nlist, d] (or bf16 bit patterns, uint16, with
    coarse_bf16), codebooks4 fp32 [M4, 16, d / M4], packed_codes uint8 [N, M4 / 2] in list order.

    The nprobe lists come from the same coarse step as the 8-bit search.  A stored vector stands for
    y = centroid + concatenated codewords; its score is ||q - y||^2, or <q, y> with the centroid part
    taken from the coarse step's value (so that a bf16 coarse quantiser enters the same way as in the
    8-bit search).  Best first, ties to the smaller id, padding (-1, +inf / -inf).
    """
    m = _METRIC[metric]
    q = _c(queries, np.float32)
    cb = np.asarray(codebooks4, np.float64)
    M4, ksub, dsub = cb.shape
    assert ksub == 16
    codes = unpack_pq4(packed_codes)
    off = np.asarray(list_offsets, np.int64)
    ids = np.asarray(ids, np.int64)
    lists, cvals = coarse(centroids, q, nprobe, m, coarse_bf16=coarse_bf16)
    if coarse_bf16:
        cen = (np.asarray(centroids, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    else:
        cen = np.asarray(centroids, np.float64)
    nq = q.shape[0]
    out_ids = np.full((nq, k), -1, np.int64)
    out_d = np.full((nq, k), np.inf if m == L2 else -np.inf, np.float32)
    for i in range(nq):
        qi = q[i].astype(np.float64)
        cand_s, cand_id = [], []
        for p in range(nprobe):
            l = int(lists[i, p])
            a, b = int(off[l]), int(off[l + 1])
            if b == a:
                continue
            r = np.concatenate([cb[s][codes[a:b, s]] for s in range(M4)], axis=1)   # [n, d] decoded residuals
            if m == L2:
                s_ = ((qi[None, :] - (cen[l][None, :] + r)) ** 2).sum(1)
            else:
                s_ = float(cvals[i, p]) + r @ qi
            cand_s.append(s_)
            cand_id.append(ids[a:b])
        if not cand_s:
            continue
        s_ = np.concatenate(cand_s)
        id_ = np.concatenate(cand_id)
        order = np.lexsort((id_, s_ if m == L2 else -s_))[:k]
        out_ids[i, :order.size] = id_[order]
        out_d[i, :order.size] = s_[order]
    return out_ids, out_d

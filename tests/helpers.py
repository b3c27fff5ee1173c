"""Shared test helpers: tolerant comparison of result lists and host views of synthetic data."""

import numpy as np
import torch


def host_index(oracle, data):
    """oracle.Index over the CPU copies of a synth.IvfPqData."""
    cen = data.centroids
    if cen.dtype == torch.bfloat16:
        cen_h = cen.cpu().view(torch.uint16).numpy()
    else:
        cen_h = cen.cpu().numpy()
    return oracle.Index(cen_h, data.codebooks.cpu().numpy(), data.codes.cpu().numpy(),
                        data.list_offsets.cpu().numpy(), data.ids.cpu().numpy(), data.metric,
                        coarse_bf16=cen.dtype == torch.bfloat16)


def match_results(ids_a, d_a, ids_o, d_o, rel=1e-4, floor=1e-6, rescore=None):
    """Compare one query's result list (a) with the oracle's (o).

    Distances (smaller = better) must agree position by position within `rel` (relative, with an
    absolute floor).  ids must be equal except inside groups of oracle distances that tie within the
    same tolerance: an id the oracle lists elsewhere must sit in such a tie group with position t; an
    id the oracle does not list at all (the tie group cut by k) is scored by the ORACLE through
    `rescore(id) -> distance` and that value must tie with the oracle's entry at t.  Without a
    `rescore` such an id is reported as unverified.  No id may appear twice (padding excepted).
    Returns a list of problems (empty = match).
    """
    problems = []
    k = len(ids_o)
    real = [int(i) for i, d in zip(ids_a, d_a) if not np.isinf(d)]
    if len(set(real)) != len(real):
        problems.append((-1, "duplicate ids", 0, 0.0, 0, 0.0))
    scale = max(floor, float(np.max(np.abs(d_o[np.isfinite(d_o)]))) if np.isfinite(d_o).any() else floor)
    for t in range(k):
        if np.isinf(d_o[t]) or np.isinf(d_a[t]):
            if not (d_o[t] == d_a[t] and ids_a[t] == ids_o[t]):
                problems.append((t, "pad", int(ids_a[t]), float(d_a[t]), int(ids_o[t]), float(d_o[t])))
            continue
        tol = rel * max(abs(float(d_o[t])), floor * scale)
        if abs(float(d_a[t]) - float(d_o[t])) > tol:
            problems.append((t, "dist", int(ids_a[t]), float(d_a[t]), int(ids_o[t]), float(d_o[t])))
            continue
        if ids_a[t] != ids_o[t]:
            where = np.nonzero(ids_o == ids_a[t])[0]
            if where.size:
                ok = abs(float(d_o[where[0]]) - float(d_o[t])) <= 2 * tol
                what = "id"
            elif rescore is None:
                ok, what = False, "id not in the oracle's list and no rescore given"
            else:
                try:
                    own = float(rescore(int(ids_a[t])))
                    ok = abs(own - float(d_o[t])) <= 2 * tol and abs(own - float(d_o[k - 1])) <= 2 * tol
                    what = "id outside the oracle's list: oracle distance %r" % own
                except KeyError:
                    ok, what = False, "id unknown to the oracle"
            if not ok:
                problems.append((t, what, int(ids_a[t]), float(d_a[t]), int(ids_o[t]), float(d_o[t])))
    return problems


class IvfPqRescorer:
    """Oracle distance of a single stored vector, looked up by id: what match_results needs for ids the
    oracle's own list does not contain.  Built over an oracle.Index (ids are unique)."""

    def __init__(self, oracle, hix):
        self.oracle, self.hix = oracle, hix
        self.order = np.argsort(hix.ids, kind="stable")
        self.sorted_ids = hix.ids[self.order]

    def position(self, ident):
        j = int(np.searchsorted(self.sorted_ids, ident))
        if j >= self.sorted_ids.size or int(self.sorted_ids[j]) != int(ident):
            raise KeyError(ident)
        pos = int(self.order[j])
        return int(np.searchsorted(self.hix.offsets, pos, side="right") - 1), pos

    def for_query(self, query, sign=1.0):
        """callable id -> sign * oracle score of that vector for `query` (KeyError for an unknown id)."""
        def f(ident):
            lst, pos = self.position(ident)
            return sign * self.oracle.adc_score(self.hix, query, lst, pos)
        return f


def coarse_rescorer(oracle, centroids_host, query, metric, coarse_bf16, sign=1.0):
    """callable list number -> sign * oracle coarse score of that list for `query`."""
    def f(lst):
        if lst < 0 or lst >= centroids_host.shape[0]:
            raise KeyError(lst)
        _, sc = oracle.coarse(centroids_host[lst:lst + 1], query[None, :], 1, metric, coarse_bf16=coarse_bf16)
        return sign * float(sc[0, 0])
    return f


def compact_hashed_subindex(oracle, data, lists):
    """Host-side oracle.Index holding only the given inverted lists of a hash-coded synth index.

    The lists' codes and ids are regenerated on the CPU from (seed, position), so nothing comes from
    the device; every other list is empty.  Used for sampled parity at sizes whose codes do not fit
    host memory: a query whose probed lists are all in `lists` gets the same answer as on the full index.
    """
    from paper_2503_14649_b200 import synth
    off = data.list_offsets.cpu().numpy()
    lists = sorted(set(int(l) for l in lists))
    lens = np.zeros(data.nlist, np.int64)
    codes, ids = [], []
    for l in lists:
        n = int(off[l + 1] - off[l])
        lens[l] = n
        if n:
            codes.append(synth.hash_codes(data.seed, int(off[l]), n, data.M).numpy())
            ids.append(synth.hash_ids(int(off[l]), n).numpy())
    new_off = np.zeros(data.nlist + 1, np.int64)
    new_off[1:] = np.cumsum(lens)
    codes = np.concatenate(codes) if codes else np.zeros((0, data.M), np.uint8)
    ids = np.concatenate(ids) if ids else np.zeros((0,), np.int64)
    cen = data.centroids
    cen_h = cen.cpu().view(torch.uint16).numpy() if cen.dtype == torch.bfloat16 else cen.cpu().numpy()
    return oracle.Index(cen_h, data.codebooks.cpu().numpy(), codes, new_off, ids, data.metric,
                        coarse_bf16=cen.dtype == torch.bfloat16)

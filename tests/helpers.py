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


def match_results(ids_a, d_a, ids_o, d_o, rel=1e-4, floor=1e-6):
    """Compare one query's result list (a) with the oracle's (o).

    Distances must agree position by position within `rel` (relative, with an
    absolute floor); ids must be equal except inside groups of oracle
    distances that tie within the same tolerance, where any order and any
    member of the tie group at the list's tail is accepted.
    Returns a list of problems (empty = match).
    """
    problems = []
    k = len(ids_o)
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
            # accept when the oracle has this id at a position whose distance ties with position t,
            # or when position t ties with the last oracle entry (tie group cut by k)
            where = np.nonzero(ids_o == ids_a[t])[0]
            ok = False
            if where.size and abs(float(d_o[where[0]]) - float(d_o[t])) <= 2 * tol:
                ok = True
            elif not where.size and abs(float(d_o[k - 1]) - float(d_o[t])) <= 2 * tol:
                ok = True
            if not ok:
                problems.append((t, "id", int(ids_a[t]), float(d_a[t]), int(ids_o[t]), float(d_o[t])))
    return problems


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

"""Brute-force reference for the schedule search (paper, Sec. 6.2, Algorithm 1).

TEST INFRASTRUCTURE ONLY, like the rest of this package: imported by tests/, never by the product package,
and it imports nothing from the product package.

The search the product implements prunes per-stage operating points to their Pareto front before it
enumerates schedules.  This module does the enumeration with no pruning at all and with its own, separately
written end-to-end arithmetic, so a test can check that both return the same frontier:

  * a schedule cuts the stage sequence into groups of consecutive stages; only inference stages marked
    collocatable may share a group; a retrieval stage and a decode stage are always groups of their own
    (Sec. 6.1, task placement);
  * every group gets an accelerator count (a retrieval group a server count), and the accelerator counts of all
    non-retrieval groups together stay within the chip budget (Sec. 6.1, resource allocation);
  * every stage gets a batch size (Sec. 6.1, batching policy);
  * stages of one group run one after the other on the group's accelerators (time-multiplexing), so a group
    serves one request per  sum over its stages of 1 / throughput  seconds, and the pipeline is as fast as its
    slowest group (Sec. 3, the paper's end-to-end throughput statement: the slowest stage decides);
  * time to first token = sum of the batch latencies of all stages before decode;
  * the result is the set of schedules not dominated in (time to first token down, requests/s per chip up).

Stages are given as plain tuples (name, kind, collocatable, perf) with perf(resource, batch) -> (latency seconds,
throughput requests/s).
"""

from __future__ import annotations

import itertools


def _partitions(n):
    """All ways to cut 0..n-1 into runs of consecutive indices."""
    if n == 0:
        yield []
        return
    for first in range(1, n + 1):
        for rest in _partitions(n - first):
            yield [list(range(0, first))] + [[i + first for i in g] for g in rest]


def enumerate_schedules(stages, chip_budget, accelerator_counts, server_counts, batches):
    """Every legal schedule as (ttft, qps_per_chip, groups, allocation, batch per stage)."""
    out = []
    n = len(stages)
    for groups in _partitions(n):
        legal = True
        for g in groups:
            if len(g) > 1:
                for i in g:
                    _, kind, colloc, _ = stages[i]
                    if kind != "inference" or not colloc:
                        legal = False
        if not legal:
            continue
        choices = [server_counts if stages[g[0]][1] == "retrieval" else accelerator_counts for g in groups]
        for alloc in itertools.product(*choices):
            chips = 0
            for g, r in zip(groups, alloc):
                if stages[g[0]][1] != "retrieval":
                    chips += r
            if chips > chip_budget:
                continue
            for bsel in itertools.product(batches, repeat=n):
                ttft = 0.0
                slowest = None
                for g, r in zip(groups, alloc):
                    seconds_per_request = 0.0
                    for i in g:
                        lat, thr = stages[i][3](r, bsel[i])
                        seconds_per_request += 1.0 / thr
                        if stages[i][1] != "decode":
                            ttft += lat
                    rate = 1.0 / seconds_per_request
                    slowest = rate if slowest is None else min(slowest, rate)
                out.append((ttft, slowest / max(chips, 1), groups, list(alloc), list(bsel)))
    return out


def frontier(schedules):
    """Schedules no other schedule beats in both metrics (equal points are reported once)."""
    keep = []
    for s in schedules:
        dominated = False
        for t in schedules:
            if (t[0] <= s[0] and t[1] >= s[1]) and (t[0] < s[0] or t[1] > s[1]):
                dominated = True
                break
        if not dominated:
            keep.append(s)
    seen, uniq = set(), []
    for s in sorted(keep, key=lambda s: (s[0], -s[1])):
        key = (round(s[0], 12), round(s[1], 12))
        if key not in seen:
            seen.add(key)
            uniq.append(s)
    return uniq

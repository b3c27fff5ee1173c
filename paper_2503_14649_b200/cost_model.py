"""Retrieval cost model and schedule search (CPU-only; no kernel is involved).

Two parts, both restated from the paper:

* The retrieval performance model (Sec. 4, "Retrieval performance modeling"): a search is a sequence of scan
  operators, one per level of a multi-level tree index; an operator that processes D bytes for a batch of Q
  queries takes  max(D / P_comp(Q), D / B_mem)  and the levels' times add up.  `scan_operator_time` and
  `tree_search_time` are that model as printed; `RetrievalModel` is its form for this library on a GPU, where a
  single query already occupies the whole device, so the compute leg does not depend on Q and a launch-bound
  floor T0 appears instead:  T(Q, D) = T0 + max(D / B_mem, Q / R_q).  `fit_retrieval_model` fits its constants to
  measured (batch size, bytes scanned, seconds) rows, e.g. the output of `bench.py --workload sweep`.

* The schedule search (Sec. 6.2, Algorithm 1): profile every pipeline stage over resources and batch sizes,
  keep each stage's Pareto-optimal points, enumerate placement x allocation x batching, assemble the end-to-end
  performance of every schedule, return the Pareto frontier of (time to first token, queries per second per
  chip).  Placement follows Sec. 6.1: consecutive stages up to the prefix may share a group of accelerators
  (time-multiplexed), retrieval always runs on its own servers, prefix and decode are never collocated.
"""

from __future__ import annotations

import itertools
from dataclasses import dataclass, field
from typing import Callable, Dict, Iterable, List, Optional, Sequence, Tuple

import numpy as np


# ---- retrieval performance model ---------------------------------------------------------------------------------

def scan_operator_time(D: float, Q: int, p_unit: float, n_units: int, B_mem: float) -> float:
    """One scan operator (Sec. 4): D bytes for a batch of Q queries, one compute unit (a CPU thread in the
    paper) per query up to n_units, each scanning p_unit bytes/s, against a memory system of B_mem bytes/s."""
    if D <= 0:
        return 0.0
    p_comp = p_unit * max(1, min(int(Q), int(n_units)))
    return max(D / p_comp, D / B_mem)


def tree_search_time(level_bytes: Sequence[float], Q: int, p_unit: float, n_units: int, B_mem: float) -> float:
    """A multi-level tree search is the sum of its levels' scan operators (Sec. 4)."""
    return float(sum(scan_operator_time(D, Q, p_unit, n_units, B_mem) for D in level_bytes))


def retrieval_bytes_per_query(n_dbvec: float, bytes_per_vec: float, p_scan_percent: float) -> float:
    """Bytes of quantised vectors one query scans: N_dbvec x B_vec x P_scan / 100 (RAGSchema section)."""
    return n_dbvec * bytes_per_vec * p_scan_percent / 100.0


@dataclass
class RetrievalModel:
    """T(Q, D) = T0 + max(D / B_mem, Q / R_q): seconds for a batch of Q queries that scans D bytes in total."""
    T0: float      # s: launch-bound floor of one search call
    B_mem: float   # bytes/s: effective scan bandwidth
    R_q: float     # queries/s the per-query stages (coarse step, table build, merge) sustain; inf = never binding
    max_rel_err: float = 0.0

    def time(self, Q: int, D: float) -> float:
        return self.T0 + max(D / self.B_mem, (Q / self.R_q) if np.isfinite(self.R_q) else 0.0)

    def qps(self, Q: int, D: float) -> float:
        return Q / self.time(Q, D)

    def as_dict(self) -> dict:
        return {"T0_us": self.T0 * 1e6, "B_mem_GBs": self.B_mem / 1e9,
                "R_q_per_s": None if not np.isfinite(self.R_q) else self.R_q, "max_rel_err": self.max_rel_err}


def fit_retrieval_model(Q: Sequence[float], D: Sequence[float], T: Sequence[float]) -> RetrievalModel:
    """Relative least squares of T = T0 + D / B_mem over the rows (small batches weigh as much as large ones);
    R_q is then the per-query rate of the rows the bandwidth leg cannot explain (those whose bytes account for less
    than half of their time beyond T0), inf when there are none."""
    Qv, Dv, Tv = (np.asarray(x, np.float64) for x in (Q, D, T))
    A = np.stack([np.ones_like(Dv), Dv], 1)
    coef, *_ = np.linalg.lstsq(A / Tv[:, None], np.ones_like(Tv), rcond=None)
    T0 = max(float(coef[0]), 0.0)
    B = 1.0 / max(float(coef[1]), 1e-30)
    over = Tv - T0                                  # time beyond the floor
    slow = (over > 0) & (Dv / B < 0.5 * over)       # rows whose bytes explain less than half of it
    R_q = float(np.min(Qv[slow] / over[slow])) if slow.any() else float("inf")
    m = RetrievalModel(T0, B, R_q)
    m.max_rel_err = float(np.max(np.abs(np.array([m.time(q, d) for q, d in zip(Qv, Dv)]) - Tv) / Tv))
    return m


# ---- Algorithm 1: exhaustive schedule search --------------------------------------------------------------------

@dataclass(frozen=True)
class StagePerf:
    """One profiled operating point of a stage: `resource` accelerators (or retrieval servers), batch size,
    latency of one batch in seconds, throughput in requests/s."""
    resource: int
    batch: int
    latency: float
    throughput: float


@dataclass
class Stage:
    """A pipeline stage.  kind: "inference" (runs on accelerators; may be collocated with its neighbours when
    `collocatable`), "retrieval" (own servers, never collocated, not counted as chips) or "decode" (accelerators,
    never collocated; its latency does not enter the time to first token)."""
    name: str
    kind: str
    perf: Callable[[int, int], Tuple[float, float]]   # (resource, batch) -> (latency s, throughput req/s)
    collocatable: bool = True


def pareto_front(points: Iterable, key: Callable) -> List:
    """Non-dominated subset; key(p) -> (cost to minimise, value to maximise).  Ties keep the first."""
    pts = sorted(points, key=lambda p: (key(p)[0], -key(p)[1]))
    out, best = [], -float("inf")
    for p in pts:
        v = key(p)[1]
        if v > best:
            out.append(p)
            best = v
    return out


def powers_of_two(limit: int) -> List[int]:
    out, r = [], 1
    while r <= limit:
        out.append(r)
        r *= 2
    return out


def profile_stages(stages: Sequence[Stage], resources: Sequence[int], batches: Sequence[int]) -> Dict[str, List[StagePerf]]:
    """Step 1: every stage at every (resource, batch); per resource only the Pareto points (latency, throughput)
    are kept, since a dominated point cannot be part of a non-dominated schedule with the same allocation."""
    prof = {}
    for st in stages:
        pts = []
        for r in resources:
            cand = []
            for b in batches:
                lat, thr = st.perf(r, b)
                cand.append(StagePerf(r, b, lat, thr))
            pts += pareto_front(cand, lambda p: (p.latency, p.throughput))
        prof[st.name] = pts
    return prof


def placement_options(stages: Sequence[Stage]) -> List[List[List[int]]]:
    """Step 2a: all ways to cut the stage sequence into groups of consecutive stages such that only
    collocatable inference stages share a group (retrieval and decode always stand alone)."""
    n = len(stages)
    out = []
    for cuts in itertools.product((0, 1), repeat=max(0, n - 1)):   # cuts[i] = 1: a boundary after stage i
        groups, cur = [], [0]
        for i in range(1, n):
            if cuts[i - 1]:
                groups.append(cur)
                cur = [i]
            else:
                cur.append(i)
        groups.append(cur)
        ok = all(len(g) == 1 or all(stages[i].kind == "inference" and stages[i].collocatable for i in g) for g in groups)
        if ok:
            out.append(groups)
    return out


@dataclass
class Schedule:
    groups: List[List[int]]
    resources: List[int]            # per group
    batches: List[int]              # per stage
    ttft: float = 0.0
    qps: float = 0.0
    chips: int = 0
    qps_per_chip: float = 0.0


def assemble_perf(stages: Sequence[Stage], groups, resources, points: Sequence[StagePerf]) -> Tuple[float, float, int]:
    """End-to-end performance of one schedule.  A group's stages are time-multiplexed on its accelerators: a
    request occupies the group for the sum of its stages' per-request times, so the group's throughput is the
    reciprocal of that sum; the pipeline runs at its slowest group.  Time to first token adds the batch latency
    of every stage before decode.  Chips are the accelerators of all non-retrieval groups."""
    ttft = 0.0
    qps = float("inf")
    chips = 0
    for g, r in zip(groups, resources):
        per_request = 0.0
        for i in g:
            p = points[i]
            per_request += 1.0 / p.throughput
            if stages[i].kind != "decode":
                ttft += p.latency
        qps = min(qps, 1.0 / per_request)
        if stages[g[0]].kind != "retrieval":
            chips += r
    return ttft, qps, chips


def search_schedules(stages: Sequence[Stage], chip_budget: int, retrieval_servers: Sequence[int],
                     batches: Sequence[int], resources: Optional[Sequence[int]] = None) -> List[Schedule]:
    """Algorithm 1: the Pareto frontier of (TTFT, QPS per chip) over placement x allocation x batching, with
    accelerator counts from `resources` (default: powers of two up to the budget) summing to at most
    `chip_budget` and retrieval stages on one of `retrieval_servers` server counts."""
    resources = list(resources) if resources is not None else powers_of_two(chip_budget)
    prof_acc = profile_stages([s for s in stages if s.kind != "retrieval"], resources, batches)
    prof_ret = profile_stages([s for s in stages if s.kind == "retrieval"], list(retrieval_servers), batches)
    prof = {**prof_acc, **prof_ret}
    found: List[Schedule] = []
    for groups in placement_options(stages):
        opts = [list(retrieval_servers) if stages[g[0]].kind == "retrieval" else resources for g in groups]
        for alloc in itertools.product(*opts):
            chips = sum(r for g, r in zip(groups, alloc) if stages[g[0]].kind != "retrieval")
            if chips > chip_budget:
                continue
            # batching: every stage picks one of its Pareto points at its group's allocation
            per_stage = []
            for g, r in zip(groups, alloc):
                for i in g:
                    per_stage.append([p for p in prof[stages[i].name] if p.resource == r])
            order = [i for g in groups for i in g]
            for combo in itertools.product(*per_stage):
                points = [None] * len(stages)
                for i, p in zip(order, combo):
                    points[i] = p
                ttft, qps, ch = assemble_perf(stages, groups, alloc, points)
                found.append(Schedule([list(g) for g in groups], list(alloc), [p.batch for p in points], ttft, qps,
                                      ch, qps / max(ch, 1)))
    return pareto_front(found, lambda s: (s.ttft, s.qps_per_chip))


def retrieval_stage(name: str, model: RetrievalModel, bytes_per_query: float) -> Stage:
    """A retrieval stage served by this library: with r servers (GPUs) each holding 1/r of the database and every
    query going to every shard (Sec. 4), a batch of b queries scans b x bytes_per_query / r bytes per server."""
    def perf(r: int, b: int):
        t = model.time(b, b * bytes_per_query / r)
        return t, b / t
    return Stage(name, "retrieval", perf, collocatable=False)

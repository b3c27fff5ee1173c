#!/usr/bin/env python
"""Benchmark of the retrieval hot path.

Headline workload: the Hyperscale-shaped IVF-PQ index, the largest of the five shapes that one B200 holds
(1e9 vectors stored as 64-byte PQ codes = 64 GB, 65 536 bf16 coarse centroids, inner product).  A step is one
rago_search over a batch of 4096 queries (coarse distances on the tensor cores + nprobe selection, table build,
list scan, top-k merge), nprobe = 64, k = 100.  The other four shapes (Mid IVF-PQ, flat search, the Hyperscale
coarse step alone, the iterative-retrieval stream) are measured in the same run and nested under "secondary".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

With N > 1 every rank holds a replica of the index and searches its own batch: query batches are independent, so
there is no data-path collective and scaling is weak.  Started without torchrun, `--gpus N` starts the N ranks
itself.  `--impl reference` times the CPU oracle, as it stands, on a bounded sample of the same workload.
Prints one JSON line on rank 0.
"""

from __future__ import annotations

import argparse
import gc
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "retrieval_qps"
UNIT = "queries/s"
HEADLINE = "hyper"
SECONDARY = ("mid", "flat", "coarse_hyper", "iter")

# DRAM bytes per logical (algorithmic) code byte of one scan_kernel launch, from ncu one-pass captures of
# dram__bytes_read.sum + dram__bytes_write.sum (profiles/scan_kernel_hyperscale_sixteenth_scale.md, profiles/scan_kernel_mid_quarter_scale.md).  A figure is only valid for
# the kernel source it was captured from: each entry names the SHA-256 of csrc/scan.cu (first 16 hex digits) and a
# run whose scan.cu hashes differently reports traffic = null.  "hyper" was captured at 1/16 of the vectors (4 GB
# of codes; the capture-size rule) and carries over to the full size because the lists are uniform and no list is
# shared through L2 at either size; "mid" was captured at full size and is not scaled to other sizes.
SCAN_TRAFFIC = {
    "hyper": {"scan_sha": "90e01c4ea3d00589", "dram_per_logical": (15956357120 + 11520000) / 16004289600},   # 0.9977
    "mid": {"scan_sha": "90e01c4ea3d00589", "dram_per_logical": (34071503872 + 9443072) / 42427363200},      # 0.8033
}


def _scan_sha():
    with open(os.path.join(ROOT, "paper_2503_14649_b200", "csrc", "scan.cu"), "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:16]


def _traffic(tag, scan_bytes, scale):
    t = SCAN_TRAFFIC.get(tag)
    if not t or t["dram_per_logical"] is None or t["scan_sha"] != _scan_sha():
        return None
    if tag == "mid" and scale != 1.0:
        return None
    return t["dram_per_logical"] * scan_bytes


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm": float(d["hbm_gbs"]), "burst": float(d["bf16_tflops"]),
                "sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "kind": "measured"}
    return {"hbm": 6650.0, "burst": 1590.0, "sustained": 1400.0, "kind": "fallback"}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons every 200 ms while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        rows = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.3] or [r for (_, r) in self.rows]
        sm, mx, reasons = [], [], set()
        for r in rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def _per_clock(achieved_gbs, clocks, dev):
    """The same rate per SM clock: the step runs under the board's power cap, so the sampled median SM clock says how
    much of a lower rate is the clock's and how much the kernel's.  bytes / clock / SM, and the rate that figure
    gives at the maximum SM clock."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    if not mhz or not mx:
        return {}
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    per = achieved_gbs * 1e9 / (sms * mhz * 1e6)
    return {"bytes_per_clk_per_sm": per, "achieved_at_max_sm_clock": per * sms * mx * 1e6 / 1e9, "sm_mhz": mhz}


def rank_batch_permutation(nq: int, rank: int) -> torch.Tensor:
    """Which of the workload's queries, in which order, rank `rank` searches: a seeded permutation, so every
    replica works on its own batch and any rank's batch can be rebuilt elsewhere (CPU generator: the same on
    every device)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(1000 + rank)
    return torch.randperm(nq, generator=g)


def max_over_ranks(value_ms: float, world: int, device) -> float:
    """The slowest rank's time (the job is as slow as its slowest replica); a no-op for one rank."""
    if world <= 1:
        return float(value_ms)
    t = torch.tensor([value_ms], device=device, dtype=torch.float64)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def whole_job_qps(nq_per_rank: int, world: int, steps: int, total_ms: float) -> float:
    """Queries per second of all replicas together (weak scaling: every rank searches nq_per_rank per step)."""
    return nq_per_rank * world * steps / (total_ms / 1e3)


def _dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def launcher_command(gpus: int, argv, port: int):
    """The command that starts `gpus` ranks of this script on one node (one process per GPU, rendezvous on
    127.0.0.1), as the documented multi-GPU launch does it."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(gpus),
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def check_world(gpus: int, world: int):
    """A run that asks for N GPUs must consist of N ranks: a mislabelled line is worse than none."""
    if max(1, gpus) != world:
        raise SystemExit("bench.py: --gpus %d but %d rank(s) are running; start it as `python bench.py --gpus %d` "
                         "(it spawns the ranks) or under torchrun with --nproc-per-node %d" % (gpus, world, gpus, gpus))


def _init_dist(need_gpu=True):
    rank, world, local = _dist_env()
    if need_gpu and not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device is visible to rank %d; the library has no CPU path" % rank)
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        local = 0
        torch.cuda.set_device(0)
    return rank, world, local, torch.device("cuda", local)


def _free():
    gc.collect()
    torch.cuda.empty_cache()


# ---- workloads -------------------------------------------------------------------------------------------------

IVF = {
    "hyper": dict(cfg=3, name="Hyperscale IVF-PQ (configs[2])", extra="IP, bf16 centroids"),
    "mid": dict(cfg=2, name="Mid IVF-PQ (configs[1])", extra="zipf=1.1 L2"),
}


def _ivf_workload_name(tag, data, c):
    w = IVF[tag]
    return "%s: N=%d d=%d nlist=%d M=%d nq=%d nprobe=%d k=%d %s" % (
        w["name"], data.N, c["d"], c["nlist"], c["M"], c["nq"], c["nprobe"], c["k"], w["extra"])


def _ivf_config(tag, data, c, args, world):
    return {"workload": _ivf_workload_name(tag, data, c), "global_batch": c["nq"] * world,
            "parallelism": "replicas x%d" % world,
            "l2_policy": "inputs larger than L2 (%.2f GB of codes per replica)" % (data.N * c["M"] / 1e9),
            "scale": args.scale}


def _oracle_on_sample(tag, data, c, sample, threads):
    """The oracle's answers for the sampled queries and the seconds it took (index preparation excluded).
    Hash-coded shapes regenerate, on the CPU, exactly the lists those queries probe."""
    import oracle
    from tests.helpers import IvfPqRescorer, compact_hashed_subindex, host_index
    q = data.queries[sample].cpu().numpy()
    if data.hash_coded:
        cen = data.centroids
        cen_h = cen.cpu().view(torch.uint16).numpy() if cen.dtype == torch.bfloat16 else cen.cpu().numpy()
        lists, _ = oracle.coarse(cen_h, q, c["nprobe"], data.metric, coarse_bf16=cen.dtype == torch.bfloat16,
                                 nthreads=threads)
        hix = compact_hashed_subindex(oracle, data, np.unique(lists))
    else:
        hix = host_index(oracle, data)
    t0 = time.perf_counter()
    ids, dists = oracle.ivfpq_search(hix, q, c["nprobe"], c["k"], nthreads=threads)
    return time.perf_counter() - t0, ids, dists, IvfPqRescorer(oracle, hix), q


def bench_ivfpq(tag, args, rank, world, local, dev, want_cpu_baseline):
    """One IVF-PQ shape: device-resident throughput, stage split, host-buffer (end-to-end) throughput, roofline of
    the scan kernel, optionally the oracle on a sample with a result check."""
    from paper_2503_14649_b200 import binding, synth
    c = synth.CONFIGS[IVF[tag]["cfg"]]
    nq, nprobe, k = c["nq"], c["nprobe"], c["k"]
    data = synth.make_config(IVF[tag]["cfg"], device=dev, scale=args.scale)
    if world > 1:  # every rank searches its own batch against its replica
        perm = rank_batch_permutation(nq, rank)
        data.queries = data.queries[perm.to(dev)].contiguous()
    ix = binding.rago_index_load(data.centroids, data.codebooks, data.codes, data.list_offsets.to(dev), data.ids,
                                 data.metric)
    q = data.queries.contiguous()
    ws_bytes = ix.search_workspace_bytes(nq, nprobe, k)
    ws = torch.empty(ws_bytes + ix.host_staging_bytes(nq, k), dtype=torch.uint8, device=dev)
    out_ids = torch.empty((nq, k), dtype=torch.int64, device=dev)
    out_d = torch.empty((nq, k), dtype=torch.float32, device=dev)

    # bytes the scan logically reads: sum over queries of probed-list lengths x M
    lists, _ = ix.rago_search_probes(q, nprobe, workspace=ws)
    L = (data.list_offsets[1:] - data.list_offsets[:-1]).to(dev)
    scanned_vectors = int(L[lists.long()].sum().item())
    scan_bytes = scanned_vectors * c["M"]

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def step():
        ix.rago_search(q, nprobe, k, out_ids, out_d, ws)

    sampler = ClockSampler(local)
    sampler.start()  # before the warm-up, so that nvidia-smi is already reporting when the timed region starts
    for _ in range(max(3, args.warmup)):
        step()
    ix.rago_check(ws)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    launches0 = binding.rago_kernel_launches()
    t0 = time.time()
    ev[0].record()
    for i in range(args.steps):
        step()
        ev[i + 1].record()
    barrier()
    t1 = time.time()
    launches = binding.rago_kernel_launches() - launches0
    total_ms = ev[0].elapsed_time(ev[-1])
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    clocks = sampler.stop(t0, t1)
    ix.rago_check(ws)
    # per-stage device times (events on the launching stream around each stage), read after each of a few steps
    ix.rago_profile_enable(True)
    stage_ms = []
    for _ in range(min(10, max(3, args.steps))):
        step()
        stage_ms.append(ix.rago_profile_read())
    ix.rago_profile_enable(False)
    scan_ms = float(np.mean([s["table_scan"] for s in stage_ms]))

    total_ms = max_over_ranks(total_ms, world, dev)
    qps = whole_job_qps(nq, world, args.steps, total_ms)

    # end to end through the host-buffer entry point: pinned queries in, pinned results out, every step
    hq = q.cpu().pin_memory()
    hids = torch.empty((nq, k), dtype=torch.int64).pin_memory()
    hd = torch.empty((nq, k), dtype=torch.float32).pin_memory()
    for _ in range(2):
        ix.rago_search_host(hq, nprobe, k, hids, hd, ws)
    barrier()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        ix.rago_search_host(hq, nprobe, k, hids, hd, ws)
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    e2e_qps = whole_job_qps(nq, world, args.steps, e2e_ms)
    assert torch.equal(hids, out_ids.cpu()), "host-buffer path disagrees with the device path"

    pk = _peaks()
    achieved = scan_bytes / (scan_ms / 1e3) / 1e9
    traffic = _traffic(tag, scan_bytes, args.scale)
    out = {
        "metric": METRIC, "value": qps, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": _ivf_config(tag, data, c, args, world),
        "clocks": clocks,
        "e2e": {"value": e2e_qps, "unit": UNIT, "h2d_bytes_per_step": nq * c["d"] * 4,
                "d2h_bytes_per_step": nq * k * 12},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "scan_kernel (table fetch + ADC scan + partial top-k)",
                     "achieved": achieved, "peak": pk["hbm"], "peak_kind": pk["kind"], "unit": "GB/s",
                     "frac": achieved / pk["hbm"], "traffic": traffic,
                     "dram_frac": (traffic / (scan_ms / 1e3) / 1e9 / pk["hbm"]) if traffic else None,
                     "algorithmic_bytes_per_launch": scan_bytes, "kernel_ms": scan_ms,
                     "scanned_vectors_per_query": scanned_vectors / nq,
                     **_per_clock(achieved, clocks, dev)},
        "stage_ms": {kk: float(np.mean([s[kk] for s in stage_ms])) for kk in stage_ms[0]},
        "step_ms_p50": float(np.median(step_ms)), "step_ms_max": float(np.max(step_ms)),
    }
    if want_cpu_baseline and rank == 0 and world == 1:
        import oracle
        from tests.helpers import match_results
        threads = oracle.default_threads()
        gi, gd = out_ids.cpu().numpy(), out_d.cpu().numpy()
        if data.hash_coded:   # a fixed, spread sample: every (nq / 64)-th query, each through all its probed lists
            sample = list(range(0, nq, max(1, nq // 64)))[:64]
        else:                 # a first, small sample sizes the real one (about 15 s of oracle time)
            n0 = min(nq, 4 * threads)
            dt0 = _oracle_on_sample(tag, data, c, list(range(n0)), threads)[0]
            sample = list(range(int(min(nq, max(n0, (n0 / dt0) * 15.0)))))
        dt, oi, od, rs, qh = _oracle_on_sample(tag, data, c, sample, threads)
        sgn = 1.0 if data.metric == "l2" else -1.0
        mism = sum(1 for t, qi in enumerate(sample)
                   if match_results(gi[qi], sgn * gd[qi], oi[t], sgn * od[t], rel=1e-4, rescore=rs.for_query(qh[t], sgn)))
        out["cpu_baseline"] = {"value": len(sample) / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
                               "sample": "%d of %d queries (%s), each through all of its probed lists, one query "
                                         "per thread" % (len(sample), nq, "evenly spaced" if data.hash_coded else "the first"),
                               "seconds": dt, "queries_not_matching_gpu": mism}
    ix.close()
    del ix, data, ws, q, out_ids, out_d, lists, L
    _free()
    return out


def _time_steps(fn, steps, warmup):
    """CUDA-event time of `steps` calls of fn on the current stream, after warm-up; returns (total ms, per-step ms)."""
    for _ in range(max(3, warmup)):
        fn()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record()
    for i in range(steps):
        fn()
        ev[i + 1].record()
    torch.cuda.synchronize()
    return ev[0].elapsed_time(ev[-1]), [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]


def bench_flat(args, dev):
    """Exact flat search, N = 10 M x 1024 bf16 rows, 256 queries, k = 100 (cosine on unit rows)."""
    from paper_2503_14649_b200 import binding, synth
    c = synth.CONFIGS[5]
    N = max(1, int(round(c["N"] * args.scale)))
    d, nq, k = c["d"], c["nq"], c["k"]
    db, q = synth.make_flat(N, d, nq, device=dev)
    ws = torch.empty(binding.rago_flat_workspace_bytes(N, d, nq, k), dtype=torch.uint8, device=dev)
    sampler = ClockSampler(dev.index or 0)
    out = {}

    def step():
        out["r"] = binding.rago_flat_search(db, q, k, workspace=ws)

    launches0 = binding.rago_kernel_launches()
    sampler.start()
    t0 = time.time()
    total_ms, step_ms = _time_steps(step, args.steps, args.warmup)
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    launches = (binding.rago_kernel_launches() - launches0) * args.steps // (args.steps + max(3, args.warmup))
    ms = total_ms / args.steps
    pk = _peaks()
    tflops = 2.0 * nq * N * d / (ms / 1e3) / 1e12
    gbs = N * d * 2 / (ms / 1e3) / 1e9
    res = {
        "metric": METRIC, "value": nq / (ms / 1e3), "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": "Exact flat search (configs[4]): N=%d d=%d bf16 unit rows, nq=%d k=%d" % (N, d, nq, k),
                   "l2_policy": "database (%.1f GB) larger than L2" % (N * d * 2 / 1e9), "scale": args.scale},
        "clocks": clocks, "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "kernel": "gemm_select_kernel + flat_merge_kernel (whole call)", "achieved": tflops,
                     "peak": pk["sustained"], "peak_kind": pk["kind"] + " (sustained bf16)", "unit": "TFLOP/s",
                     "frac": tflops / pk["sustained"], "frac_of_burst": tflops / pk["burst"], "traffic": None,
                     "hbm": {"achieved": gbs, "peak": pk["hbm"], "frac": gbs / pk["hbm"], "unit": "GB/s"}},
        "step_ms_p50": float(np.median(step_ms)), "step_ms_max": float(np.max(step_ms))}
    del db, q, ws, out
    _free()
    return res


def bench_coarse_hyper(args, dev):
    """The coarse step of the Hyperscale shape alone: 4096 queries x 65 536 bf16 centroids, d = 768, inner
    product, nprobe = 64 (a 4096 x 768 x 65 536 contraction with the selection fused in)."""
    from paper_2503_14649_b200 import binding, synth
    c = synth.CONFIGS[3]
    nq, nprobe, nlist, d = c["nq"], c["nprobe"], c["nlist"], c["d"]
    data = synth.make_ivfpq_hashed(nlist * 4, d, nlist, c["M"], nq, metric=c["metric"], coarse_bf16=True, device=dev)
    ix = binding.rago_index_load(data.centroids, data.codebooks, data.codes, data.list_offsets.to(dev), data.ids, data.metric)
    q = data.queries.contiguous()
    ws = torch.empty(ix.search_workspace_bytes(nq, nprobe, 1), dtype=torch.uint8, device=dev)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    t0 = time.time()
    total_ms, step_ms = _time_steps(lambda: ix.rago_search_probes(q, nprobe, workspace=ws), args.steps, args.warmup)
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    ix.rago_check(ws)
    ix.rago_profile_enable(True)
    out_i = torch.empty((nq, 1), dtype=torch.int64, device=dev)
    out_d = torch.empty((nq, 1), dtype=torch.float32, device=dev)
    stage = []
    for _ in range(5):
        ix.rago_search(q, nprobe, 1, out_i, out_d, ws)
        stage.append(ix.rago_profile_read())
    gemm_ms = float(np.median([s["coarse_scores"] for s in stage]))
    sel_ms = float(np.median([s["probe_select"] for s in stage]))
    ms = total_ms / args.steps
    pk = _peaks()
    tflops = 2.0 * nq * nlist * d / (gemm_ms / 1e3) / 1e12
    res = {
        "metric": "coarse_qps", "value": nq / (ms / 1e3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "Hyperscale coarse step (configs[2], coarse only): nq=%d nlist=%d d=%d bf16 nprobe=%d IP"
                   % (nq, nlist, d, nprobe), "l2_policy": "centroids 100 MB, L2 flushed by the candidate lists"},
        "clocks": clocks,
        "roofline": {"bound": "tensor", "kernel": "split_bf16_kernel + pilot pass + gemm_select_kernel (the coarse_scores stage)",
                     "achieved": tflops, "peak": pk["burst"], "peak_kind": pk["kind"] + " (burst bf16)", "unit": "TFLOP/s",
                     "frac": tflops / pk["burst"], "frac_of_sustained": tflops / pk["sustained"], "traffic": None,
                     "kernel_ms": gemm_ms},
        "stage_ms": {"coarse_scores": gemm_ms, "probe_select": sel_ms},
        "step_ms_p50": float(np.median(step_ms))}
    ix.close()
    del ix, data, ws, q
    _free()
    return res


def _iter_stream(args, dev, tree):
    """One measurement of the 256-batch stream; tree = (n1, b1) puts a second quantiser level above the coarse
    centroids (the centroids are then drawn as a two-level hierarchy), None is the one-level index."""
    from paper_2503_14649_b200 import binding, synth
    c = synth.CONFIGS[4]
    nprobe, k = c["nprobe"], c["k"]
    sizes = synth.batch_size_stream(synth.MASTER_SEED, 256)
    over = {"tree_n1": tree[0]} if tree else {}
    data = synth.make_config(4, device=dev, scale=args.scale, nq=sum(sizes), **over)
    ix = binding.rago_index_load(data.centroids, data.codebooks, data.codes, data.list_offsets.to(dev), data.ids, data.metric)
    if tree:
        ix.rago_index_set_coarse_tree(data.extra["level1"].to(dev), data.extra["child_offsets"].to(dev), tree[1])
    q = data.queries.contiguous()
    ws = torch.empty(ix.search_workspace_bytes(16, nprobe, k), dtype=torch.uint8, device=dev)
    out_i = torch.empty((16, k), dtype=torch.int64, device=dev)
    out_d = torch.empty((16, k), dtype=torch.float32, device=dev)
    starts = np.concatenate([[0], np.cumsum(sizes)[:-1]])

    def stream(ev=None):
        for b, nb in enumerate(sizes):
            if ev is not None:
                ev[b].record()
            ix.rago_search(q[starts[b]:starts[b] + nb], nprobe, k, out_i[:nb], out_d[:nb], ws)
        if ev is not None:
            ev[len(sizes)].record()

    for _ in range(max(3, args.warmup)):
        stream()
    torch.cuda.synchronize()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    t0 = time.time()
    lat = {1: [], 4: [], 16: []}
    tot = []
    for _ in range(args.steps):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(sizes) + 1)]
        stream(ev)
        torch.cuda.synchronize()
        for b, nb in enumerate(sizes):
            lat[nb].append(ev[b].elapsed_time(ev[b + 1]))
        tot.append(ev[0].elapsed_time(ev[-1]))
    # the same call with nothing between the calls: 240 searches of one batch size back to back, time per call
    b2b = {}
    for nb in (1, 4, 16):
        qs = [q[i * nb:(i + 1) * nb] for i in range(12)] * 20
        oi, od = out_i[:nb], out_d[:nb]
        best = None
        for _ in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for x in qs:
                ix.rago_search(x, nprobe, k, oi, od, ws)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / len(qs)
            best = ms if best is None else min(best, ms)
        b2b[str(nb)] = best
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    ix.rago_check(ws)
    # stage split of a batch of one (events around every stage serialise the launches: shares, not a latency)
    ix.rago_profile_enable(True)
    st1 = []
    for _ in range(20):
        ix.rago_search(q[:1], nprobe, k, out_i[:1], out_d[:1], ws)
        st1.append(ix.rago_profile_read())
    ix.rago_profile_enable(False)
    ms = float(np.mean(tot))
    alll = np.concatenate([lat[1], lat[4], lat[16]])
    res = {"qps": sum(sizes) / (ms / 1e3), "ms_per_stream": ms, "clocks": clocks, "N": data.N, "queries": sum(sizes),
           "latency_ms": {"p50": float(np.percentile(alll, 50)), "p99": float(np.percentile(alll, 99)),
                          "by_batch_size": {str(nb): {"p50": float(np.percentile(v, 50)), "p99": float(np.percentile(v, 99))}
                                            for nb, v in lat.items()},
                          "note": "device time between consecutive batches' start events (launch-to-launch on a busy stream)",
                          "back_to_back_ms_per_call": b2b,
                          "back_to_back_note": "240 calls of one batch size with nothing between them (no event per call), "
                                               "device time / 240, best of 3"},
           "stage_ms_batch_of_1": {kk: float(np.median([s_[kk] for s_ in st1])) for kk in st1[0]}}
    ix.close()
    del ix, data, ws, q
    _free()
    return res


def bench_iter(args, dev):
    """The iterative-retrieval latency shape: N = 1e8, d = 512, nlist = 16 384, M = 32; a stream of 256 batches of
    1, 4 or 16 queries issued back to back on one stream, nprobe = 16, k = 20; per-batch latency from CUDA events
    between the batches.  Measured twice: on the one-level index the shape names, and with a level of 128 nodes
    above the coarse centroids (8 nodes kept), the paper's multi-level index in its smallest form."""
    from paper_2503_14649_b200 import synth
    c = synth.CONFIGS[4]
    one = _iter_stream(args, dev, None)
    two = _iter_stream(args, dev, (128, 8))
    return {
        "metric": METRIC, "value": one["qps"], "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": one["ms_per_stream"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "Iterative-retrieval stream (configs[3]): N=%d d=%d nlist=%d M=%d, 256 batches of 1/4/16 "
                   "queries back to back on one stream, nprobe=%d k=%d L2" % (one["N"], c["d"], c["nlist"], c["M"],
                                                                               c["nprobe"], c["k"]),
                   "step": "one pass over the 256-batch stream (%d queries)" % one["queries"], "scale": args.scale},
        "clocks": one["clocks"], "latency_ms": one["latency_ms"], "stage_ms_batch_of_1": one["stage_ms_batch_of_1"],
        "two_level_coarse": {"n1": 128, "b1": 8, "value": two["qps"], "unit": UNIT, "ms_per_step": two["ms_per_stream"],
                             "latency_ms": two["latency_ms"], "stage_ms_batch_of_1": two["stage_ms_batch_of_1"],
                             "clocks": two["clocks"],
                             "note": "same shape with hierarchical coarse centroids (synth tree_n1 = 128); results "
                                     "follow the two-level definition, not the one-level one"},
        "roofline": {"bound": "latency", "kernel": "whole call", "achieved": None, "peak": None,
                     "unit": None, "frac": None, "traffic": None}}


def bench_sharded(args, rank, world, local, dev):
    """Database-sharded search.  Every rank holds its own Mid-shape shard with an independent index (its own
    seed); all ranks answer rank 0's query batch, exchange their [nq, k] answers with one all-gather and aggregate
    them.  The database grows with the number of ranks, the query batch does not."""
    from paper_2503_14649_b200 import binding, sharded, synth
    c = synth.CONFIGS[2]
    nq, nprobe, k = c["nq"], c["nprobe"], c["k"]
    data = synth.make_config(2, device=dev, scale=args.scale, seed=synth.MASTER_SEED + 7919 * rank)
    ix = binding.rago_index_load(data.centroids, data.codebooks, data.codes, data.list_offsets.to(dev), data.ids,
                                 data.metric)
    q = data.queries.contiguous()
    if world > 1:
        torch.distributed.broadcast(q, 0)
    ws = torch.empty(ix.search_workspace_bytes(nq, nprobe, k), dtype=torch.uint8, device=dev)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def step():
        return sharded.rago_search_sharded(ix, q, nprobe, k, workspace=ws)

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    launches0 = binding.rago_kernel_launches()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    t0 = time.time()
    ev[0].record()
    for _ in range(args.steps):
        step()
    ev[1].record()
    barrier()
    t1 = time.time()
    launches = binding.rago_kernel_launches() - launches0
    clocks = sampler.stop(t0, t1)
    ix.rago_check(ws)
    total_ms = max_over_ranks(ev[0].elapsed_time(ev[1]), world, dev)
    # the aggregation kernel alone, on gathered answers already in place
    ids, dists = ix.rago_search(q, nprobe, k, workspace=ws)
    parts = sharded.gather_parts(ids, dists)
    agg_ms, _ = _time_steps(lambda: binding.rago_merge_results(parts[0], parts[1], k, ix.metric), 20, 3)
    ms = total_ms / args.steps
    return {
        "metric": METRIC, "value": nq / (ms / 1e3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak (database grows with ranks, one shared query batch)", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": "Sharded Mid IVF-PQ: %d shard(s) of N=%d d=%d nlist=%d M=%d, independent indexes; nq=%d "
                               "nprobe=%d k=%d L2; all-gather + aggregation every step"
                               % (world, data.N, c["d"], c["nlist"], c["M"], nq, nprobe, k),
                   "l2_policy": "inputs larger than L2", "scale": args.scale},
        "clocks": clocks, "gpu_launches": launches, "aggregate_kernel_ms": agg_ms / 20,
        "exchange_bytes_per_rank": nq * k * 12}


def bench_sweep(args, dev):
    """Batch-size sweep on the Mid index: the measurements the retrieval cost model is fitted to.  The paper models
    a scan operator as T = max(D / P_comp(Q), D / B_mem) with D the bytes scanned and Q the batch size (Sec. 4);
    here every batch size gets its measured time and scanned bytes, and cost_model.fit_retrieval_model turns the
    rows into the constants of that model on this GPU."""
    from paper_2503_14649_b200 import binding, cost_model, synth
    c = synth.CONFIGS[2]
    nprobe, k = c["nprobe"], c["k"]
    data = synth.make_config(2, device=dev, scale=args.scale)
    ix = binding.rago_index_load(data.centroids, data.codebooks, data.codes, data.list_offsets.to(dev), data.ids,
                                 data.metric)
    Ln = (data.list_offsets[1:] - data.list_offsets[:-1]).to(dev)
    rows = []
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    t0 = time.time()
    for nq in (1, 2, 4, 8, 16, 32, 64, 128, 256, 512, 1024):
        q = data.queries[:nq].contiguous()
        ws = torch.empty(ix.search_workspace_bytes(nq, nprobe, k), dtype=torch.uint8, device=dev)
        out_i = torch.empty((nq, k), dtype=torch.int64, device=dev)
        out_d = torch.empty((nq, k), dtype=torch.float32, device=dev)
        lists, _ = ix.rago_search_probes(q, nprobe, workspace=ws)
        D = int(Ln[lists.long()].sum().item()) * c["M"]
        steps = max(10, min(200, int(2000 / nq)))
        total_ms, step_ms = _time_steps(lambda: ix.rago_search(q, nprobe, k, out_i, out_d, ws), steps, 3)
        ix.rago_check(ws)
        ms = float(np.median(step_ms))
        rows.append({"nq": nq, "ms": ms, "qps": nq / (ms / 1e3), "scanned_bytes": D, "gbs": D / (ms / 1e3) / 1e9})
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    model = cost_model.fit_retrieval_model([r["nq"] for r in rows], [r["scanned_bytes"] for r in rows],
                                           [r["ms"] * 1e-3 for r in rows])
    return {
        "metric": "retrieval_cost_model", "unit": "s = T0 + max(D / B_mem, Q / R_q)", "n_gpus": 1, "data": "synthetic",
        "config": {"workload": "Mid IVF-PQ index (configs[1]), batch sizes 1..1024, nprobe=%d k=%d" % (nprobe, k),
                   "scale": args.scale},
        "fit": model.as_dict(), "rows": rows, "clocks": clocks}


def bench_pq4(args, dev):
    """The Mid shape with 4-bit codes (the paper's low-precision PQ variant): the same corpus recipe, d = 768,
    M4 = 96 sub-spaces of 16 codewords = 48 bytes per vector (half of the 8-bit index's 96)."""
    from paper_2503_14649_b200 import binding, synth
    c = synth.CONFIGS[2]
    nq, nprobe, k, M4 = c["nq"], c["nprobe"], c["k"], args.m4
    N = max(1, int(round(c["N"] * args.scale)))
    data = synth.make_ivfpq4(N, c["d"], c["nlist"], M4, nq, metric=c["metric"], zipf=c["zipf"], device=dev)
    ix = binding.rago_index_load_pq4(data.centroids, data.codebooks, data.codes, data.list_offsets.to(dev), data.ids,
                                     data.metric)
    q = data.queries.contiguous()
    ws = torch.empty(ix.search_workspace_bytes(nq, nprobe, k), dtype=torch.uint8, device=dev)
    out_i = torch.empty((nq, k), dtype=torch.int64, device=dev)
    out_d = torch.empty((nq, k), dtype=torch.float32, device=dev)
    lists, _ = ix.rago_search_probes(q, nprobe, workspace=ws)
    Ln = (data.list_offsets[1:] - data.list_offsets[:-1]).to(dev)
    scanned = int(Ln[lists.long()].sum().item())
    scan_bytes = scanned * (M4 // 2)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    t0 = time.time()
    launches0 = binding.rago_kernel_launches()
    total_ms, step_ms = _time_steps(lambda: ix.rago_search(q, nprobe, k, out_i, out_d, ws), args.steps, args.warmup)
    launches = binding.rago_kernel_launches() - launches0
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    ix.rago_check(ws)
    ix.rago_profile_enable(True)
    stage = []
    for _ in range(5):
        ix.rago_search(q, nprobe, k, out_i, out_d, ws)
        stage.append(ix.rago_profile_read())
    st = {kk: float(np.median([s_[kk] for s_ in stage])) for kk in stage[0]}
    ms = total_ms / args.steps
    pk = _peaks()
    achieved = scan_bytes / (st["table_scan"] / 1e3) / 1e9
    return {
        "metric": METRIC, "value": nq / (ms / 1e3), "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": "Mid shape with 4-bit PQ codes: N=%d d=%d nlist=%d zipf=%.1f M4=%d (%d bytes per vector) "
                               "nq=%d nprobe=%d k=%d L2" % (N, c["d"], c["nlist"], c["zipf"], M4, M4 // 2, nq, nprobe, k),
                   "l2_policy": "inputs larger than L2 (%.2f GB of codes)" % (N * (M4 // 2) / 1e9), "scale": args.scale},
        "clocks": clocks, "gpu_launches": launches,
        "roofline": {"bound": "hbm", "kernel": "scan_kernel (table fetch + ADC scan + partial top-k)", "achieved": achieved,
                     "peak": pk["hbm"], "peak_kind": pk["kind"], "unit": "GB/s", "frac": achieved / pk["hbm"], "traffic": None,
                     "algorithmic_bytes_per_launch": scan_bytes, "kernel_ms": st["table_scan"],
                     "scanned_vectors_per_s": scanned / (st["table_scan"] / 1e3)},
        "stage_ms": st, "step_ms_p50": float(np.median(step_ms))}


# ---- the reference arm: the CPU oracle on a bounded sample ---------------------------------------------------------

def run_reference(args):
    """Each step searches one query per host core of the headline workload with the oracle, every query through
    all of its probed lists (regenerated on the CPU from the seed before the timed steps)."""
    rank, world, _ = _dist_env()
    if rank != 0:
        return
    import oracle
    from paper_2503_14649_b200 import synth
    from tests.helpers import compact_hashed_subindex, host_index
    tag = args.workload if args.workload in IVF else HEADLINE
    c = synth.CONFIGS[IVF[tag]["cfg"]]
    threads = oracle.default_threads()
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    data = synth.make_config(IVF[tag]["cfg"], device=dev, scale=args.scale, materialise=False) \
        if tag == "hyper" else synth.make_config(IVF[tag]["cfg"], device=dev, scale=args.scale)
    nsample = min(c["nq"], threads)  # one query per core per step
    q = data.queries[:nsample].cpu().numpy()
    if data.hash_coded:
        cen_h = data.centroids.cpu().view(torch.uint16).numpy() if data.coarse_bf16 else data.centroids.cpu().numpy()
        lists, _ = oracle.coarse(cen_h, q, c["nprobe"], data.metric, coarse_bf16=data.coarse_bf16, nthreads=threads)
        hix = compact_hashed_subindex(oracle, data, np.unique(lists))
    else:
        hix = host_index(oracle, data)
    for _ in range(args.warmup):
        oracle.ivfpq_search(hix, q, c["nprobe"], c["k"], nthreads=threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.ivfpq_search(hix, q, c["nprobe"], c["k"], nthreads=threads)
    dt = time.perf_counter() - t0
    qps = nsample * args.steps / dt
    sample = "%d of %d queries per step, each through all of its probed lists, one query per thread" % (nsample, c["nq"])
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": qps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": _ivf_config(tag, data, c, args, max(1, args.gpus)),
        "cpu_baseline": {"value": qps, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": qps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---- entry ---------------------------------------------------------------------------------------------------------

def run_ours(args):
    rank, world, local, dev = _init_dist()
    check_world(args.gpus, world)
    wl = args.workload or HEADLINE
    single = {"flat": lambda: bench_flat(args, dev), "coarse_hyper": lambda: bench_coarse_hyper(args, dev),
              "iter": lambda: bench_iter(args, dev), "sweep": lambda: bench_sweep(args, dev),
              "pq4": lambda: bench_pq4(args, dev)}
    if wl in IVF:
        out = bench_ivfpq(wl, args, rank, world, local, dev, want_cpu_baseline=not args.no_cpu_baseline)
        if args.workload is None and world == 1 and not args.no_secondary:
            # the other four shapes, each a full line of its own, so that one run records all five
            sec = {}
            for name in SECONDARY:
                sub = argparse.Namespace(**vars(args))
                sub.steps = min(args.steps, 30)
                try:
                    sec[name] = bench_ivfpq(name, sub, 0, 1, local, dev, want_cpu_baseline=not args.no_cpu_baseline) \
                        if name in IVF else single[name]()
                except Exception as e:  # a failed secondary must not lose the headline
                    sec[name] = {"error": "%s: %s" % (type(e).__name__, e)}
                    _free()
            out["secondary"] = sec
    elif wl == "sharded":
        out = bench_sharded(args, rank, world, local, dev)
    else:
        if world > 1:
            raise SystemExit("bench.py: --workload %s runs on one GPU" % wl)
        out = single[wl]()
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        torch.distributed.destroy_process_group()


def main(argv=None):
    argv = list(sys.argv[1:] if argv is None else argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scale", type=float, default=1.0, help="shrink N (development only; 1.0 = the named workload)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="headline workload only")
    ap.add_argument("--m4", type=int, default=96, help="--workload pq4: number of 4-bit sub-spaces")
    ap.add_argument("--workload", default=None,
                    choices=["hyper", "mid", "flat", "coarse_hyper", "iter", "sharded", "sweep", "pq4"],
                    help="default: the Hyperscale headline plus the four secondary shapes; a name runs that one alone")
    args = ap.parse_args(argv)
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "RANK" not in os.environ:
        # started plainly: start the ranks ourselves, one process per GPU, and hand over
        port = 29400 + os.getpid() % 500
        raise SystemExit(subprocess.call(launcher_command(args.gpus, argv, port)))
    run_ours(args)


if __name__ == "__main__":
    main()

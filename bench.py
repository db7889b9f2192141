#!/usr/bin/env python
"""Benchmark of the FROG search hot path: mixed-selectivity QPS at recall@10 >= 0.95 on one B200,
with the achieved fraction of the HBM roofline and the CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one frog_search call over the whole query batch (every row of the hot path: endpoint
lookup, hotspot localization, entry points, the expansion loop with EN identification, lazy hash
check, vector gather + L2, sort/merge, output).  The index and the queries are resident in HBM
when the timed region starts; the ``e2e`` figure repeats the measurement through the host-buffer
call, transfers included.

The headline workload is the largest configuration (``deep10m``: 10M x 96, 10,000 queries, width
fraction log-uniform in 2^-12..1, k = 10).  Without ``--workload`` the run then also measures the
other configurations (tiny, sift, deep1m at each fixed width fraction, deep10m at k = 100, text)
and reports them under ``config.per_workload``: the (budget, beam width) reaching the recall target,
queries/s, algorithmic bytes, fraction of the HBM peak and the CPU oracle's rate on a bounded sample.

With N > 1 every rank holds a full replica and answers its own copy of the batch (no data-path
collective); only the headline is measured.  ``--impl reference`` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import shutil
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "mixed-selectivity QPS at recall@10>=0.95"
UNIT = "queries/s"
SWEEP = [16, 24, 32, 40, 44, 48, 52, 56, 64, 80, 96, 112, 128, 160, 192, 256, 320, 384, 448, 512]
SECONDARY_BUDGETS = [32, 64, 96, 128]  # ... for the entries of config.per_workload and the reference arm's choice
BUDGETS = [16, 32, 48, 64, 96]  # expansion budget B of Alg. 2: from the paper's default upwards (the kernels take up to 128)
RECALL_TARGET = 0.95
HBM_FALLBACK_GBS = 6650.0
HEADLINE = "deep10m"
DEEP1M_FRACTIONS = [2.0 ** -10, 2.0 ** -7, 2.0 ** -4, 2.0 ** -1, 1.0]
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "dram_traffic_per_launch.txt")
DEBUG_FLAGS = 0
RANGE_TEXT = {"tiny": "2^-8..1", "sift": "2^-10..1", "deep1m": "2^-10..1", "deep10m": "2^-12..1", "text": "2^-10..1"}


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return HBM_FALLBACK_GBS, "fallback"


def workload_text(wl, fraction=None) -> str:
    """One string per workload, the same in both arms."""
    if fraction is None:
        sel = f"mixed selectivity (width fraction log-uniform {RANGE_TEXT.get(wl.name, '?')})"
    else:
        sel = f"fixed width fraction 2^{int(round(math.log2(fraction)))}"
    return f"{wl.name}: n={wl.n} d={wl.d} nq={wl.nq} k={wl.k} {sel}"


def ncu_traffic(name: str, n: int, k: int, budget: int, beam: int, fraction=None):
    """DRAM bytes (read + write) of one search-kernel launch from the tracked table of ncu captures,
    or None when no capture exists for exactly this batch and operating point."""
    name = f"{name}:mixed" if fraction is None else f"{name}:2^{int(round(math.log2(fraction)))}"
    try:
        with open(TRAFFIC_TABLE) as f:
            for ln in f:
                t = ln.split()
                if len(t) >= 6 and not ln.startswith("#"):
                    if (t[0], int(t[1]), int(t[2]), int(t[3]), int(t[4])) == (name, n, k, budget, beam):
                        return float(t[5])
    except Exception:
        pass
    return None


def prepare_index(frog, wl, cache_dir, builder="auto", device=0):
    """Build (or reuse) the index file of a workload.  The cache is an optimisation only.
    builder: "gpu" (CUDA builder), "cpu" (host builder) or "auto" (gpu when a device is there)."""
    os.makedirs(cache_dir, exist_ok=True)
    from paper_2608_16491_b200 import build as b
    if builder == "auto":
        try:
            import torch
            builder = "gpu" if torch.cuda.is_available() else "cpu"
        except Exception:
            builder = "cpu"
    src = "frog_build_gpu.cu" if builder == "gpu" else "frog_build.cpp"
    h = hashlib.sha1()
    h.update(open(os.path.join(b.CSRC, src), "rb").read())
    h.update(open(os.path.join(b.CSRC, "frog_device.cuh"), "rb").read() if builder == "gpu" else b"")
    h.update(open(os.path.join(ROOT, "datagen", "__init__.py"), "rb").read())
    tag = h.hexdigest()[:12]
    path = os.path.join(cache_dir, f"{wl.name}_{wl.n}_{builder}_{tag}.idx")
    secs = 0.0
    if not os.path.exists(path):
        need = wl.n * (8 + 4 * wl.d + 4 * 20 * wl.m) + (1 << 30)
        free = shutil.disk_usage(cache_dir).free
        if free < need:
            raise SystemExit(f"not enough disk under {cache_dir} for the index of {wl.name}: {free >> 30} GiB free, "
                             f"about {need >> 30} GiB needed")
        t = time.time()
        tmp = path + f".tmp{os.getpid()}"
        if builder == "gpu":
            frog.build_index_gpu(wl.vectors, wl.attrs, tmp, device=device, seed=wl.seed)
        else:
            frog.build_index(wl.vectors, wl.attrs, tmp, seed=wl.seed)
        os.replace(tmp, path)
        secs = time.time() - t
    return path, secs


def recall_at_k(ids: np.ndarray, gt: np.ndarray) -> float:
    """|R ∩ GT| / |GT| averaged over the queries with a non-empty GT (rows are sorted per chunk to keep
    the comparison small at k = 100)."""
    valid = gt >= 0
    denom = valid.sum(axis=1)
    per_q = np.zeros(ids.shape[0], dtype=np.int64)
    step = max(1, (1 << 24) // max(1, ids.shape[1] * gt.shape[1]))
    for s in range(0, ids.shape[0], step):
        hit = (ids[s:s + step, :, None] == gt[s:s + step, None, :]) & valid[s:s + step, None, :]
        per_q[s:s + step] = hit.any(axis=1).sum(axis=1)
    ok = denom > 0
    return float((per_q[ok] / denom[ok]).mean()) if ok.any() else 1.0


def recall_tie_aware(dists: np.ndarray, gt_d: np.ndarray) -> float:
    fin = np.isfinite(gt_d)
    denom = fin.sum(axis=1)
    kth = np.where(fin, gt_d, -np.inf).max(axis=1)
    hit = (dists <= kth[:, None] * (1 + 1e-6)) & np.isfinite(dists)
    ok = denom > 0
    return float((np.minimum(hit.sum(axis=1), denom)[ok] / denom[ok]).mean()) if ok.any() else 1.0


class ClockSampler:
    """SM clock and throttle reasons read through NVML (read-only queries) by a background thread
    every millisecond or so while the timed region runs."""

    REASONS = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
               "sw_thermal_slowdown": 0x20}

    def __init__(self, device: int):
        self.samples = []          # (time, sm_mhz, reasons bitmask)
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            # NVML enumerates physical devices: honour CUDA_VISIBLE_DEVICES when it lists indices
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            idx = device
            if vis and all(t.strip().isdigit() for t in vis.split(",")):
                idx = int(vis.split(",")[device])
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        except Exception as e:           # no NVML: the clocks entry stays empty
            log(f"[bench] clock sampling unavailable: {e}")

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                mhz = float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    rs = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    rs = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                self.samples.append((time.time(), mhz, rs))
            except Exception:
                pass
            time.sleep(0.001)

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)

    def summary(self, t0, t1):
        rows = [s for s in self.samples if t0 <= s[0] <= t1]
        scope = "timed region"
        if not rows:
            rows = [s for s in self.samples if t0 - 0.5 <= s[0] <= t1 + 0.5]
            scope = "within 0.5 s of the timed region"
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        bits = 0
        for _, _, r in rows:
            bits |= r
        return {"sm_mhz": float(np.median([r[1] for r in rows])), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(k for k, v in self.REASONS.items() if bits & v), "samples": len(rows),
                "scope": scope}


def algorithmic_bytes(stats: np.ndarray, n: int, d: int, d_pad: int, m: int, k: int) -> float:
    """Bytes the method must move per batch: query vector, endpoint probes, ENC rows scanned,
    vectors whose distance is evaluated, and the result rows."""
    nq = stats.shape[0]
    per_q = 4 * d + 8 * math.ceil(math.log2(max(n, 2))) + 8 * k
    return float(nq * per_q + 4.0 * m * stats[:, 1].astype(np.float64).sum()
                 + 4.0 * d_pad * stats[:, 3].astype(np.float64).sum())


def ensure_built():
    """Compile the libraries if they are missing (rank 0 builds, the others wait for the files)."""
    from paper_2608_16491_b200 import build as b
    rank = int(os.environ.get("RANK", "0"))
    missing = [p for p in (b.LIB_SEARCH, b.LIB_BUILD) if not os.path.exists(p)]
    if missing and rank == 0:
        b.build_all()
    t0 = time.time()
    while any(not os.path.exists(p) for p in (b.LIB_SEARCH, b.LIB_BUILD)):
        if time.time() - t0 > 900:
            raise SystemExit("shared libraries missing and not built within 15 minutes")
        time.sleep(1.0)


# ------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle
# ------------------------------------------------------------------------------------------------
def oracle_operating_point(oracle, ix, wl, sample: int, budgets):
    """The rule of the other arm (per budget the smallest beam of the sweep whose recall reaches the
    target; among those the cheapest, here by distance evaluations), applied by the oracle alone on the
    first `sample` queries with the oracle's exact slab scan as ground truth."""
    S = min(sample, wl.nq)
    Q, lo, hi = wl.queries[:S], wl.lo[:S], wl.hi[:S]
    gt, _, _ = oracle.exact_slab(ix, Q, lo, hi, wl.k, mode=1)
    best = None
    for B in budgets:
        for ef in SWEEP:
            if ef < wl.k:
                continue
            r = oracle.search(ix, Q, lo, hi, wl.k, ef, B=B)
            rec = recall_at_k(r.ids, gt)
            if rec >= RECALL_TARGET:
                cost = float(r.stats[:, 3].sum()) + 4.0 * float(r.stats[:, 0].sum())
                if best is None or cost < best[2]:
                    best = (ef, B, cost, rec)
                break
    if best is None:
        return SWEEP[-1], budgets[-1], None
    return best[0], best[1], best[3]


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: K steps over a bounded query sample."""
    from paper_2608_16491_b200 import replicas
    rank, _, ws = replicas.world()
    if rank != 0:
        return
    import datagen
    import oracle
    from paper_2608_16491_b200 import build as frog_build
    frog_build.build_all()              # the index builder (tooling); no-op when up to date
    import paper_2608_16491_b200 as frog
    name = args.workload or HEADLINE
    wl = datagen.make_workload(name, n=args.n or None, nq=args.nq or None)
    path, build_s = prepare_index(frog, wl, args.cache_dir, args.builder)
    ix = oracle.load_index(path)
    S = min(args.ref_sample, wl.nq)
    Q, lo, hi = wl.queries[:S], wl.lo[:S], wl.hi[:S]
    beam, budget, rec = args.beam, args.budget, None
    if beam <= 0 or budget <= 0:
        budgets = [args.budget] if args.budget > 0 else SECONDARY_BUDGETS
        beam, budget, rec = oracle_operating_point(oracle, ix, wl, 300, budgets)
    for _ in range(args.warmup):
        oracle.search(ix, Q, lo, hi, wl.k, beam, B=budget)
    t0 = time.perf_counter()
    threads = 1
    for _ in range(args.steps):
        threads = oracle.search(ix, Q, lo, hi, wl.k, beam, B=budget).threads
    dt = time.perf_counter() - t0
    qps = S * args.steps / dt
    out = {
        "impl": "reference", "metric": METRIC, "value": qps, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": workload_text(wl), "beam_width": beam, "budget": budget, "epn": 16},
        "cpu_baseline": {"value": qps, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"first {S} of {wl.nq} queries per step, beam_width={beam}, budget={budget}"
                                   + ("" if rec is None else f" (operating point chosen by the oracle on 300 queries, "
                                                             f"recall@{wl.k} {rec:.4f} there)")},
        "e2e": {"value": qps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
class Batch:
    """One workload resident on the device: index, queries, ranges, exact answers."""

    def __init__(self, frog, torch, wl, path, dev, local_rank):
        self.wl, self.path, self.dev = wl, path, dev
        self.ix = frog.Index.load(path, local_rank)
        self.q = torch.from_numpy(wl.queries).to(dev)
        self.lo = torch.from_numpy(wl.lo).to(dev)
        self.hi = torch.from_numpy(wl.hi).to(dev)
        nq, k = wl.nq, wl.k
        self.out_ids = torch.empty((nq, k), dtype=torch.int32, device=dev)
        self.out_d = torch.empty((nq, k), dtype=torch.float32, device=dev)
        # ground truth: exact filtered kNN by slab scan on the GPU (parity-tested against the oracle)
        gt_ids, gt_d = self.ix.exact_search(self.q, self.lo, self.hi, k)
        torch.cuda.synchronize()
        self.gt_ids, self.gt_d = gt_ids.cpu().numpy(), gt_d.cpu().numpy()

    def search(self, beam, prm, **kw):
        return self.ix.search(self.q, self.lo, self.hi, self.wl.k, beam, out_ids=self.out_ids, out_dists=self.out_d,
                              params=prm, **kw)

    def close(self):
        self.ix.close()


def sweep_operating_point(frog, torch, b: Batch, budgets, beams, tag=""):
    """Per budget the smallest beam width of the sweep reaching the recall target; the fastest of those
    is the operating point.  Returns (chosen row or None, all rows)."""
    rows, best = [], None
    k = b.wl.k
    for B in budgets:
        prm = frog.Params(budget=B, debug_flags=DEBUG_FLAGS)
        for ef in beams:
            if ef < k:
                continue
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            b.search(ef, prm)   # warm
            evs[0].record()
            for i in range(3):  # the median of three launches ranks the candidates
                b.search(ef, prm)
                evs[i + 1].record()
            torch.cuda.synchronize()
            ms = sorted(evs[i].elapsed_time(evs[i + 1]) for i in range(3))[1]
            ids = b.out_ids.cpu().numpy()
            rec = recall_at_k(ids, b.gt_ids)
            rec_t = recall_tie_aware(b.out_d.cpu().numpy(), b.gt_d)
            row = {"budget": B, "beam_width": ef, "recall": round(rec, 4), "recall_tie_aware": round(rec_t, 4),
                   "qps": round(b.wl.nq / (ms * 1e-3))}
            rows.append(row)
            log(f"[bench]{tag} B={B} ef_s={ef}: recall@{k}={rec:.4f} (tie-aware {rec_t:.4f}) {row['qps']} q/s")
            if rec >= RECALL_TARGET or len(beams) == 1:
                if best is None or row["qps"] > best["qps"]:
                    best = row
                break
    return best, rows


def timed_launches(torch, b: Batch, beam, prm, steps, warmup):
    """K launches on the current stream with an event after each: per-launch milliseconds."""
    stream = torch.cuda.current_stream()
    for _ in range(max(warmup, 3)):
        b.search(beam, prm)
    torch.cuda.synchronize()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    evs[0].record(stream)
    for i in range(steps):
        b.search(beam, prm)
        evs[i + 1].record(stream)
    torch.cuda.synchronize()
    return [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)], evs[0].elapsed_time(evs[-1])


def kernel_only_ms(frog, torch, b: Batch, beam, budget, steps):
    """Device time of the search kernel alone (the step also runs two small planning kernels), launch by
    launch, from CUDA events the library records around that kernel on the launching stream."""
    prm = frog.Params(budget=budget, debug_flags=16 | DEBUG_FLAGS)
    out = []
    for _ in range(steps):
        b.search(beam, prm)
        out.append(b.ix.kernel_ms())
    return out


def counters(torch, b: Batch, beam, prm):
    stats = torch.zeros((b.wl.nq, 4), dtype=torch.int32, device=b.dev)
    status = torch.zeros(b.wl.nq, dtype=torch.int32, device=b.dev)
    b.search(beam, prm, status=status, stats=stats)
    torch.cuda.synchronize()
    return stats.cpu().numpy().view(np.uint32), status.cpu().numpy().view(np.uint32)


def cpu_oracle_rate(b: Batch, beam, budget, sample, passes, st=None):
    """The oracle on the first `sample` queries with all host threads; also compares ids and counters."""
    import oracle
    oix = oracle.load_index(b.path)
    wl = b.wl
    S = min(sample, wl.nq)
    t0 = time.perf_counter()
    for _ in range(passes):
        ref = oracle.search(oix, wl.queries[:S], wl.lo[:S], wl.hi[:S], wl.k, beam, B=budget)
    dt = (time.perf_counter() - t0) / passes
    out = {"value": S / dt, "unit": UNIT, "cores": ref.threads, "kind": "oracle",
           "sample": f"first {S} of {wl.nq} queries, beam_width={beam}, budget={budget}, mean of {passes} pass(es) "
                     f"(about {dt * passes * ref.threads:.0f} core-seconds)",
           "ids_equal_to_gpu": bool(np.array_equal(b.out_ids.cpu().numpy()[:S], ref.ids))}
    if st is not None:
        out["counters_equal_to_gpu"] = bool(np.array_equal(st[:S], ref.stats))
    return out, oix


def measure_secondary(frog, torch, datagen, args, name, k, fraction, dev, local_rank, peak, steps):
    """One entry of config.per_workload."""
    t = time.time()
    wl = datagen.make_workload(name, k=k, fractions=None if fraction is None else [fraction])
    path, build_s = prepare_index(frog, wl, args.cache_dir, args.builder, local_rank)
    b = Batch(frog, torch, wl, path, dev, local_rank)
    try:
        tag = f" [{name} k={k}" + ("" if fraction is None else f" f=2^{int(round(math.log2(fraction)))}") + "]"
        best, rows = sweep_operating_point(frog, torch, b, SECONDARY_BUDGETS, SWEEP, tag)
        reached = best is not None
        if not reached:
            best = max(rows, key=lambda r: r["recall"])
        beam, budget = best["beam_width"], best["budget"]
        prm = frog.Params(budget=budget, debug_flags=DEBUG_FLAGS)
        st, status = counters(torch, b, beam, prm)
        info = b.ix.info
        alg = algorithmic_bytes(st, info.n, info.d, info.d_pad, info.m, k)
        per_ms, _ = timed_launches(torch, b, beam, prm, steps, 3)
        mean_ms, med_ms = float(np.mean(per_ms)), float(np.median(per_ms))
        k_ms = float(np.mean(kernel_only_ms(frog, torch, b, beam, budget, 10)))
        b.search(beam, prm)
        torch.cuda.synchronize()
        cpu, _ = cpu_oracle_rate(b, beam, budget, args.cpu_sample_secondary, 1, st)
        out = {"workload": workload_text(wl, fraction), "k": k,
               "operating_point": {"budget": budget, "beam_width": beam} if reached else "not reached",
               "recall": best["recall"], "recall_tie_aware": best["recall_tie_aware"],
               "qps": wl.nq / (mean_ms * 1e-3), "qps_median": wl.nq / (med_ms * 1e-3), "launches_timed": steps,
               "ms_per_launch": mean_ms, "search_kernel_ms": k_ms, "algorithmic_bytes_per_launch": alg,
               "roofline_frac": alg / (k_ms * 1e-3) / 1e9 / peak,
               "traffic": ncu_traffic(wl.name, wl.n, k, budget, beam, fraction),
               "row_bytes": info.d_pad * 4, "expansions_per_query": float(st[:, 0].mean()),
               "distances_per_query": float(st[:, 3].mean()),
               "cpu_oracle_qps": cpu["value"], "cpu_cores": cpu["cores"], "cpu_sample": cpu["sample"],
               "ids_equal_to_oracle_on_sample": cpu["ids_equal_to_gpu"],
               "counters_equal_to_oracle_on_sample": cpu.get("counters_equal_to_gpu"),
               "index_build_seconds": round(build_s, 1), "seconds": None}
        if not reached:
            out["best_budget"], out["best_beam_width"] = budget, beam
        out["seconds"] = round(time.time() - t, 1)
        return out
    finally:
        b.close()


def run_ours(args):
    import torch
    from paper_2608_16491_b200 import replicas
    rank, local_rank, ws = replicas.world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the search path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    replicas.init("nccl")
    import datagen
    from paper_2608_16491_b200 import build as frog_build
    if local_rank == 0:
        frog_build.build_all()          # no-op when the in-tree libraries are up to date
    replicas.barrier()
    import paper_2608_16491_b200 as frog
    peak, peak_src = measured_hbm_peak()
    t_start = time.time()

    name = args.workload or HEADLINE
    t = time.time()
    wl = datagen.make_workload(name, n=args.n or None, nq=args.nq or None, k=args.k)
    gen_s = time.time() - t
    if rank == 0:
        path, build_s = prepare_index(frog, wl, args.cache_dir, args.builder, local_rank)
    replicas.barrier()
    if rank != 0:
        path, build_s = prepare_index(frog, wl, args.cache_dir, args.builder, local_rank)
    t = time.time()
    b = Batch(frog, torch, wl, path, dev, local_rank)
    load_s = time.time() - t
    info = b.ix.info
    nq, k = wl.nq, wl.k
    log(f"[bench] workload {wl.name} n={wl.n} d={wl.d} nq={wl.nq}: gen {gen_s:.1f}s build {build_s:.1f}s "
        f"load+ground truth {load_s:.1f}s")

    # sweep (budget B, beam width ef_s): per budget the smallest ef_s reaching the recall target; the
    # configuration with the highest throughput among those is the one that gets timed
    budgets = [args.budget] if args.budget > 0 else BUDGETS
    beams = [args.beam] if args.beam > 0 else SWEEP
    best, sweep = sweep_operating_point(frog, torch, b, budgets, beams)
    reached = best is not None
    if not reached:
        best = max(sweep, key=lambda r: r["recall"])
    chosen = best
    beam, budget = chosen["beam_width"], chosen["budget"]
    prm = frog.Params(budget=budget, debug_flags=DEBUG_FLAGS)

    # counters of the chosen configuration -> algorithmic bytes per launch
    st, status = counters(torch, b, beam, prm)
    alg_bytes = algorithmic_bytes(st, info.n, info.d, info.d_pad, info.m, k)
    launch = b.ix.launch_info(beam, prm)

    # ---- timed region: K launches, device-resident inputs ----------------------------------------
    sampler = ClockSampler(local_rank) if rank == 0 else None
    stream = torch.cuda.current_stream()
    for _ in range(max(args.warmup, 3)):
        b.search(beam, prm)
    torch.cuda.synchronize()
    replicas.barrier()
    torch.cuda.synchronize()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    t_wall0 = time.time()
    evs[0].record(stream)
    for i in range(args.steps):
        b.search(beam, prm)
        evs[i + 1].record(stream)
    torch.cuda.synchronize()
    replicas.barrier()
    torch.cuda.synchronize()
    t_wall1 = time.time()
    total_ms = evs[0].elapsed_time(evs[-1])
    per_launch_ms = [evs[i].elapsed_time(evs[i + 1]) for i in range(args.steps)]
    total_ms_max = replicas.max_over_ranks(total_ms, dev)
    clocks = sampler.summary(t_wall0, t_wall1) if sampler else None

    # the search kernel alone, launch by launch (the roofline's kernel time)
    k_only = kernel_only_ms(frog, torch, b, beam, budget, args.steps)

    # the paper's protocol (Sec. 8.1): 30 repetitions, mean and median, when K is smaller than that
    proto_ms = per_launch_ms
    if args.steps < 30:
        proto_ms, _ = timed_launches(torch, b, beam, prm, 30, 0)

    # ---- the same K launches handed to two streams in turn (batches of a serving loop overlap: the
    # tail of one launch, where its last queries leave warps idle, is filled by the next) -----------
    out_ids = b.out_ids
    pipe_ms_max = None
    if args.streams > 1:
        streams = [torch.cuda.Stream(device=dev) for _ in range(args.streams)]
        outs = [(torch.empty_like(b.out_ids), torch.empty_like(b.out_d)) for _ in streams]
        torch.cuda.synchronize()
        for j, sj in enumerate(streams):
            b.ix.search(b.q, b.lo, b.hi, k, beam, out_ids=outs[j][0], out_dists=outs[j][1], params=prm, stream=sj)
        torch.cuda.synchronize()
        replicas.barrier()
        p0 = torch.cuda.Event(enable_timing=True)
        pends = [torch.cuda.Event(enable_timing=True) for _ in streams]
        p0.record(streams[0])
        for sj in streams[1:]:
            sj.wait_event(p0)
        for i in range(args.steps):
            j = i % len(streams)
            b.ix.search(b.q, b.lo, b.hi, k, beam, out_ids=outs[j][0], out_dists=outs[j][1], params=prm,
                        stream=streams[j])
        for j, sj in enumerate(streams):
            pends[j].record(sj)
        torch.cuda.synchronize()
        replicas.barrier()
        pipe_ms = max(p0.elapsed_time(e) for e in pends)
        pipe_ms_max = replicas.max_over_ranks(pipe_ms, dev)
        pipe_same = all(bool(torch.equal(o[0], out_ids)) for o in outs)
        del outs

    # ---- end to end: host buffers in, host buffers out, transfers inside the timed region ----------
    hq = torch.from_numpy(wl.queries).pin_memory()
    hlo = torch.from_numpy(wl.lo).pin_memory()
    hhi = torch.from_numpy(wl.hi).pin_memory()
    h_ids = torch.empty((nq, k), dtype=torch.int32).pin_memory()
    h_d = torch.empty((nq, k), dtype=torch.float32).pin_memory()
    for _ in range(3):
        b.ix.search_host(hq, hlo, hhi, k, beam, out_ids=h_ids, out_dists=h_d, params=prm)
    replicas.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        b.ix.search_host(hq, hlo, hhi, k, beam, out_ids=h_ids, out_dists=h_d, params=prm)
    e2e_s = time.perf_counter() - t0
    replicas.barrier()
    e2e_s_max = replicas.max_over_ranks(e2e_s, dev)
    if sampler:
        sampler.stop()
    e2e_same = bool(np.array_equal(h_ids.numpy(), out_ids.cpu().numpy()))

    if rank != 0:
        b.close()
        return
    mean_launch_ms = float(np.mean(per_launch_ms))
    kernel_ms = float(np.mean(k_only))
    achieved = alg_bytes / (kernel_ms * 1e-3) / 1e9
    value = ws * nq * args.steps / (total_ms_max * 1e-3)

    # ---- CPU oracle on the host cores, bounded sample; doubles as a parity check ------------------
    cpu = None
    if not args.no_cpu_baseline and ws == 1:      # rank 0 at N = 1 only
        cpu, oix = cpu_oracle_rate(b, beam, budget, args.cpu_sample, 2, st)
        # the ground truth used for the recall figures, checked against the oracle's own slab scan
        import oracle
        S = min(48, nq)
        sel = np.argsort(wl.hi[:512].astype(np.int64) - wl.lo[:512].astype(np.int64))[:S]   # the narrowest: cheap to scan
        g_ids, _, _ = oracle.exact_slab(oix, wl.queries[sel], wl.lo[sel], wl.hi[sel], k, mode=1)
        cpu["ground_truth_equal_to_oracle_on_sample"] = bool(np.array_equal(g_ids, b.gt_ids[sel]))
    b.close()

    per_workload = None
    if not args.workload and ws == 1 and not args.no_per_workload:
        per_workload = []
        todo = [("tiny", 10, None), ("sift", 10, None)]
        todo += [("deep1m", 10, f) for f in DEEP1M_FRACTIONS]
        todo += [("deep10m", 100, None), ("text", 10, None)]
        for wname, wk, frac in todo:
            try:
                row = measure_secondary(frog, torch, datagen, args, wname, wk, frac, dev, local_rank, peak, 30)
            except SystemExit as e:
                row = {"workload": wname, "k": wk, "skipped": str(e)}
            log(f"[bench] per-workload {json.dumps(row)}")
            per_workload.append(row)
        # the headline itself, in the same shape
        per_workload.insert(7, {
            "workload": workload_text(wl), "k": k,
            "operating_point": {"budget": budget, "beam_width": beam} if reached else "not reached",
            "recall": chosen["recall"], "recall_tie_aware": chosen["recall_tie_aware"],
            "qps": nq / (float(np.mean(proto_ms)) * 1e-3), "qps_median": nq / (float(np.median(proto_ms)) * 1e-3),
            "launches_timed": len(proto_ms), "ms_per_launch": float(np.mean(proto_ms)),
            "algorithmic_bytes_per_launch": alg_bytes,
            "search_kernel_ms": kernel_ms, "roofline_frac": alg_bytes / (kernel_ms * 1e-3) / 1e9 / peak,
            "traffic": ncu_traffic(wl.name, wl.n, k, budget, beam), "row_bytes": info.d_pad * 4,
            "expansions_per_query": float(st[:, 0].mean()), "distances_per_query": float(st[:, 3].mean()),
            "cpu_oracle_qps": None if cpu is None else cpu["value"], "cpu_cores": None if cpu is None else cpu["cores"],
            "cpu_sample": None if cpu is None else cpu["sample"], "headline": True})
        # deep1m pooled over its five fixed fractions (same query vectors, five batches)
        d1 = [r for r in per_workload if r.get("workload", "").startswith("deep1m") and "qps" in r]
        if d1:
            tot_q = sum(10_000 for _ in d1)
            per_workload.append({"workload": "deep1m: pooled over the five fixed width fractions", "k": 10,
                                 "qps": tot_q / sum(10_000 / r["qps"] for r in d1),
                                 "recall": float(np.mean([r["recall"] for r in d1])),
                                 "roofline_frac": sum(r["algorithmic_bytes_per_launch"] for r in d1)
                                 / sum(r["search_kernel_ms"] * 1e-3 for r in d1) / 1e9 / peak})

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": ws, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms_max / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_text(wl),
                   "beam_width": beam, "budget": budget, "epn": 16,
                   "recall_at_k": chosen["recall"], "recall_target_reached": reached,
                   "recall_tie_aware": chosen["recall_tie_aware"],
                   "index": {"H": info.H, "m": info.m, "bytes": info.device_bytes, "build_seconds": round(build_s, 1),
                             "file": os.path.basename(path),
                             "builder": "CUDA builder, paper parameters plus reverse edges and RNG-ordered ENC selection"},
                   "l2": "inputs larger than L2 (%.1f GB index, ~%.1f GB gathered per launch)"
                         % (info.device_bytes / 1e9, alg_bytes / 1e9),
                   "parallelism": "replicas" if ws > 1 else "single GPU",
                   "launch": launch, "sweep": sweep, "per_workload": per_workload},
        "e2e": {"value": ws * nq * args.steps / e2e_s_max, "unit": UNIT,
                "h2d_bytes_per_step": nq * info.d * 4 + 2 * nq * 4, "d2h_bytes_per_step": 2 * nq * k * 4,
                "same_ids_as_device_path": e2e_same,
                "transfer": "pinned host buffers, read and written by the kernels across the bus inside the "
                            "timed region (frog_search_host); wall clock per call including its stream sync"},
        "pipelined": None if pipe_ms_max is None else {
            "streams": args.streams, "value": ws * nq * args.steps / (pipe_ms_max * 1e-3), "unit": UNIT,
            "ms_per_step": pipe_ms_max / args.steps,
            "roofline_frac": alg_bytes * args.steps / (pipe_ms_max * 1e-3) / 1e9 / peak,
            "same_ids_as_single_stream": pipe_same,
            "note": "the same K launches issued on the streams in turn; launches of different streams "
                    "overlap on the GPU (own scratch set each), not part of `value`"},
        "gpu_launches": 3 * args.steps,   # per step: endpoint/plan kernel, order kernel, search kernel
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": peak_src,
                     "traffic": ncu_traffic(wl.name, wl.n, k, budget, beam),
                     "algorithmic_bytes_per_launch": alg_bytes, "kernel_ms": kernel_ms,
                     "kernel_ms_median": float(np.median(k_only)), "kernel_launches_timed": len(k_only),
                     "step_ms": mean_launch_ms, "step_frac": alg_bytes / (mean_launch_ms * 1e-3) / 1e9 / peak,
                     "note": "kernel_ms: CUDA events around the search kernel alone, one launch at a time; "
                             "step_ms: a whole frog_search call (planning kernels included) in the timed region",
                     "kernel": "frog_search_lean_kernel" if info.d_pad * 4 in (384, 512) else "frog_search_kernel"},
        "protocol_30": {"launches": len(proto_ms), "qps_mean": nq / (float(np.mean(proto_ms)) * 1e-3),
                        "qps_median": nq / (float(np.median(proto_ms)) * 1e-3)},
        "clocks": clocks,
        "expansions_per_query": float(st[:, 0].mean()), "distances_per_query": float(st[:, 3].mean()),
        "enc_rows_per_query": float(st[:, 1].mean()),
        "status_flags": {"iteration_cap": int((status & 4).astype(bool).sum()),
                         "copy_timeout": int((status & 32).astype(bool).sum())},
        "seconds_total": round(time.time() - t_start, 1),
    }
    if cpu:
        out["cpu_baseline"] = cpu
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="", help="measure this workload only (default: deep10m as the headline, "
                                                   "then the other configurations under config.per_workload)")
    ap.add_argument("--k", type=int, default=10)
    ap.add_argument("--n", type=int, default=0, help="override the number of base vectors (profiling on a small case)")
    ap.add_argument("--nq", type=int, default=0, help="override the number of queries")
    ap.add_argument("--beam", type=int, default=0, help="beam width; 0 = smallest reaching the recall target")
    ap.add_argument("--budget", type=int, default=0, help="expansion budget B; 0 = best of 16, 32, 48, 64, 96")
    ap.add_argument("--debug-flags", type=int, default=0,
                    help="frog_params_t.debug_flags for every search of the run (8: visited hash table on small "
                         "indexes too, for profiling that form on a small case)")
    ap.add_argument("--cache-dir", default=os.environ.get("FROG_CACHE", "/tmp/frog_cache"))
    ap.add_argument("--builder", default="auto", choices=["auto", "gpu", "cpu"],
                    help="index builder used when the cache has no file for the workload")
    ap.add_argument("--cpu-sample", type=int, default=10000)
    ap.add_argument("--cpu-sample-secondary", type=int, default=2000)
    ap.add_argument("--ref-sample", type=int, default=1000)
    ap.add_argument("--streams", type=int, default=2,
                    help="streams of the extra pipelined measurement (1 = skip it)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-workload", action="store_true")
    args = ap.parse_args()
    global DEBUG_FLAGS
    DEBUG_FLAGS = args.debug_flags
    ensure_built()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

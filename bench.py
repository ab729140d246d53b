#!/usr/bin/env python
"""Throughput of the DS-FACTO epoch on B200: nonzero-updates/s = nnz x epochs / seconds.

A step is one dsfacto_epoch (w0 step, the p strata, the recompute pass, the objective) over the
C4 synthetic workload (hashed categorical, n = 45M, d = 2^20, 39 entries per row, K = 16, p = 512).
  value      inputs resident in HBM; CUDA events around exactly K epochs on the library's stream
  e2e        dsfacto_load_csr from host buffers (host->device copies, tile bucketing) + one epoch +
             the objective read back, through the C ABI
  roofline   dominant kernel (stratum SGD): algorithmic bytes / measured launch time vs the
             measured HBM copy peak
  cpu_baseline   the CPU oracle, as it stands, on a bounded row sample of the same workload

--impl reference times the CPU oracle alone.  --gpus N (under torchrun) runs N independent
replicas (the path is single-GPU; no collective on the data path)."""
from __future__ import annotations

import argparse
import datetime
import json
import os
import statistics
import subprocess
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "nonzero-updates/sec"
UNIT = "updates/s"
ORACLE_SAMPLE_ROWS = 1_000_000
# dram__bytes_read.sum + dram__bytes_write.sum of sgd_sweep_kernel per stored entry, by factor width K, from
# the ncu captures summarised in profiles/ (scaled cases; DRAM traffic of the sweep grows with the entries).
# A width without a capture of the current kernel reports traffic = null.
SGD_DRAM_BYTES_PER_ENTRY = {16: 22.0, 128: 186.0}


def peaks():
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        try:
            return float(json.loads(f.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Ends the sampling; keeps the samples taken between the two datetimes (the timed region).
        The sampler is started before the warm-up so that it is already running when the region
        begins; a region shorter than the sampling period keeps the samples closest to it."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = []   # (time, sm MHz, max MHz, active reasons)
        for line in out.splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                when = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f")
                rows.append((when, float(parts[1]), float(parts[2]),
                             [nm for nm, val in zip(names, parts[4:8]) if val.lower().startswith("active")]))
            except ValueError:
                continue
        window = "timed region"
        inside = [r for r in rows if t_begin is None or (t_begin <= r[0] <= t_end)]
        if not inside and rows:
            mid = t_begin + (t_end - t_begin) / 2
            inside = sorted(rows, key=lambda r: abs((r[0] - mid).total_seconds()))[:3]
            window = "nearest samples (region shorter than the sampling period)"
        sm = [r[1] for r in inside]
        reasons = sorted({nm for r in inside for nm in r[3]})
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(r[2] for r in inside) if inside else None,
                "samples": len(sm), "window": window, "reasons": reasons}


def oracle_leg(wl_name: str, rows: int, min_seconds: float, max_epochs: int):
    """Times oracle epochs (as the oracle stands) on the first `rows` rows' worth of the workload."""
    from oracle import dsfacto_oracle as O
    from paper_2004_13940_b200 import workloads as W

    wl = W.make(wl_name, n=rows)
    o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    o.epoch()                                   # untimed: page in, OpenMP team start
    t0 = time.perf_counter()
    epochs = 0
    while epochs < max_epochs and (epochs == 0 or time.perf_counter() - t0 < min_seconds):
        o.epoch()
        epochs += 1
    dt = time.perf_counter() - t0
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    return {"value": wl.nnz * epochs / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%s generator, first %d rows (nnz %d), p=%d, %d oracle epochs in %.1f s (fp64, OpenMP over the "
                      "tiles of a round)" % (wl_name, wl.n, wl.nnz, wl.p, epochs, dt),
            "seconds": dt, "epochs": epochs, "nnz": wl.nnz}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import dsfacto_oracle as O
    from paper_2004_13940_b200 import workloads as W

    wl = W.make(args.workload, n=args.oracle_rows)
    o = O.Oracle(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
    o.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
    per_step = []
    for step in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        o.epoch()
        if step >= args.warmup:
            per_step.append(time.perf_counter() - t0)
    total = sum(per_step)
    value = wl.nnz * len(per_step) / total
    info = {"cores": int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))}
    cfg = workload_config(args.workload, sample_rows=args.oracle_rows)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(per_step),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": cfg,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": info["cores"], "kind": "oracle",
                             "sample": "each step = one oracle epoch on the first %d rows of the %s generator"
                                       % (args.oracle_rows, args.workload)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def take_turns(rank, world, barrier, fn):
    """Runs fn() on one rank at a time (rank order), a barrier after each turn; returns this rank's result.
    Used for the loads, so that the host-side bucketing buffers of the replicas never coexist."""
    out = None
    for turn in range(world):
        if turn == rank:
            out = fn()
        barrier()
    return out


def max_over_ranks(values, world, device):
    """Element-wise maximum of a list of floats over all ranks (identity for one rank)."""
    if world == 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_rate(world, units_per_rank, steps, ms):
    """Units all replicas processed per second, given the slowest rank's time for `steps` steps."""
    return world * units_per_rank * steps / (ms * 1e-3)


def workload_config(name, sample_rows=None):
    from paper_2004_13940_b200 import workloads as W
    c = W.CONFIGS[name]
    cfg = {"workload": name, "n": c["n"], "d": c["d"], "K": c["K"], "p": c["p"],
           "loss": "logistic" if c["loss"] else "squared", "eta": c["eta"], "lambda": 1e-3,
           "l2": "inputs larger than L2 (no flush needed)"}
    if sample_rows is not None:
        cfg["sample_rows"] = sample_rows
    return cfg


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2004_13940_b200 import dsfacto as D
    from paper_2004_13940_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()

    D.lib()
    # pinned host buffers for the CSR arrays: they are the e2e leg's source
    def pinned_empty(count, dtype):
        t = torch.empty(int(count), dtype={np.int64: torch.int64, np.int32: torch.int32,
                                          np.float32: torch.float32}[np.dtype(dtype).type], pin_memory=args.pin)
        return t.numpy()

    t_gen = time.perf_counter()
    wl = W.make(args.workload, n=args.rows, p=args.p, empty=pinned_empty)
    if args.K is not None:
        wl.K = int(args.K)
    t_gen = time.perf_counter() - t_gen
    nnz = wl.nnz
    stream = torch.cuda.current_stream()

    def new_handle():
        g = D.DSFacto(wl.n, wl.d, wl.K, wl.p, wl.loss, wl.lambda_w, wl.lambda_v, wl.eta, wl.init_seed)
        g.set_stream(stream.cuda_stream)
        if args.refresh_every > 0:
            g.set_refresh_every(args.refresh_every)
        return g

    # ranks load one after another so that the host-side bucketing buffers never coexist
    def first_load():
        t0 = time.perf_counter()
        gg = new_handle()
        gg.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
        return gg, time.perf_counter() - t0

    g, t_load = take_turns(rank, world, barrier, first_load)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(args.warmup):
        g.epoch()
    launches0 = g.launch_count()
    barrier(); torch.cuda.synchronize()
    t_begin = datetime.datetime.now()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    phase = np.zeros(4)
    ev0.record(stream)
    epoch_log = []
    for step in range(args.steps):
        g.epoch()
        ph = np.asarray(g.last_epoch_ms())
        phase += ph
        if args.log and rank == 0:
            epoch_log.append({"epoch": args.warmup + step + 1, "objective": g.objective(), "loss": g.stats()[0],
                              "seconds": ph[0] * 1e-3, "nnz_updates_per_s": nnz / (ph[0] * 1e-3),
                              "ms": {"sgd_strata": float(ph[1]), "refresh": float(ph[2]), "norms": float(ph[3])}})
    ev1.record(stream)
    torch.cuda.synchronize(); barrier()
    clocks = sampler.stop(t_begin, datetime.datetime.now()) if rank == 0 else None
    if args.log and rank == 0:
        with open(args.log, "a") as fh:
            for rec in epoch_log:
                fh.write(json.dumps(rec) + "\n")
    ms = ev0.elapsed_time(ev1)
    launches = g.launch_count() - launches0
    load_path, load_h2d, load_d2h = g.last_load()   # how the tile lists were built and what crossed the link for it
    objective = g.objective()
    g.close()

    # ---- e2e: host buffers -> load_csr -> epoch -> objective, through the C ABI ----
    def e2e_leg():
        per_step = []
        for _ in range(args.e2e_steps):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            hh = new_handle()
            hh.load_csr(wl.indptr, wl.indices, wl.values, wl.y)
            hh.epoch()
            _ = hh.objective()
            hh.close()
            torch.cuda.synchronize()
            per_step.append(1e3 * (time.perf_counter() - t0))
        return per_step

    e2e_steps_ms = take_turns(rank, world, barrier, e2e_leg) or [0.0]
    e2e_ms = float(sum(e2e_steps_ms))
    e2e_min, e2e_med = float(min(e2e_steps_ms)), float(statistics.median(e2e_steps_ms))
    ms, e2e_ms, e2e_min, e2e_med = max_over_ranks([ms, e2e_ms, e2e_min, e2e_med], world, "cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    phase /= args.steps
    peak, peak_kind = peaks()
    K, n, d, p = wl.K, wl.n, wl.d, wl.p
    # Stratum SGD, algorithmic bytes per epoch.  Row-block sweep (default): every array once - the 8-byte
    # entry records, A and G once (all entries of a row meet in one launch), w and V read + written.
    # Round sweep: the p tiles of a round own disjoint row blocks, so every entry re-reads G_i and a_i.
    # A plan cut into segments (--refresh-every) keeps the row-block sweep: one launch per segment, each of
    # which reads A and G of all rows and reads and writes w and V once.
    sweep = os.environ.get("DSFACTO_SWEEP", "rowblock")
    segments = -(-p // args.refresh_every) if 0 < args.refresh_every < p else 1
    sgd_gather = nnz * (8 + 4 * K + 4) + 8 * d * (K + 1)
    sgd_floor = 8 * nnz + segments * (4 * n * (K + 1) + 8 * d * (K + 1))
    sgd_bytes = sgd_gather if sweep == "round" else sgd_floor
    ref_bytes = 8 * nnz + 8 * (n + 1) + 4 * d * (K + 2) + 4 * n * K + 8 * n
    sgd_s, ref_s = phase[1] * 1e-3, phase[2] * 1e-3
    # the counters were taken on the default schedule (row-block sweep, one launch per sweep)
    per_entry = SGD_DRAM_BYTES_PER_ENTRY.get(K)
    traffic = None if (per_entry is None or sweep != "rowblock" or segments != 1) else per_entry * nnz
    roof = {"bound": "hbm", "kernel": "sgd_sweep_kernel", "launches_per_step": segments, "sweep": sweep,
            "achieved": sgd_bytes / sgd_s / 1e9, "peak": peak, "unit": "GB/s", "frac": sgd_bytes / sgd_s / 1e9 / peak,
            "peak_kind": "of " + peak_kind, "traffic": traffic,
            "algorithmic_bytes_per_launch": sgd_bytes / segments, "avg_launch_us": 1e6 * sgd_s / segments,
            "model": ("gather: nnz*(8+4K+4) + 8d(K+1)" if sweep == "round" else "stream floor: 8nnz + 4n(K+1) + 8d(K+1)")
                     + ("; one launch covers the whole sweep" if segments == 1 else
                        "; %d launches per sweep, A, G, w, V once per launch" % segments),
            # bytes the sweep asks its caches for when nothing is reused in registers; most of them are served
            # by L2, so this rate is NOT a fraction of the HBM peak and is given for context only
            "cache_request_model": {"bytes_per_step": sgd_gather, "rate_GBps": sgd_gather / sgd_s / 1e9},
            "refresh_kernel": {"algorithmic_bytes_per_step": ref_bytes, "ms": phase[2],
                               "achieved": ref_bytes / ref_s / 1e9, "frac": ref_bytes / ref_s / 1e9 / peak}}
    value = whole_job_rate(world, nnz, args.steps, ms)
    e2e = {"value": whole_job_rate(world, nnz, args.e2e_steps, e2e_ms) if args.e2e_steps > 0 else None, "unit": UNIT, "h2d_bytes_per_step": int(load_h2d),
           "d2h_bytes_per_step": int(load_d2h) + 32, "steps": args.e2e_steps, "ms_per_step": e2e_ms / max(args.e2e_steps, 1),
           "ms_per_step_min": e2e_min, "ms_per_step_median": e2e_med,
           "tile_lists": ("bucketed on the host, one copy", "bucketed on the host, streamed to the device",
                          "CSR arrays copied, bucketed on the device")[load_path],
           "what": "dsfacto_create + dsfacto_load_csr (H2D of the CSR arrays, tile bucketing, launch plan, first recompute pass) + dsfacto_epoch + dsfacto_objective"}
    cfg = workload_config(args.workload)
    if args.refresh_every > 0:
        cfg["refresh_every"] = args.refresh_every
    cfg.update({"n": n, "p": p, "nnz": nnz, "parallelism": "replicas x%d" % world if world > 1 else "single GPU",
                "pinned_host": bool(args.pin)})
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg, "clocks": clocks, "e2e": e2e,
            "gpu_launches": int(launches), "roofline": roof,
            "phase_ms": {"epoch": phase[0], "sgd_strata": phase[1], "refresh": phase[2], "norms": phase[3]},
            "objective": objective, "setup_s": {"generate": t_gen, "create+load_csr": t_load}}
    if world == 1 and not args.no_cpu_baseline:
        cb = oracle_leg(args.workload, args.oracle_rows, args.oracle_seconds, 50)
        line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C4")
    ap.add_argument("--rows", type=int, default=None, help="override the workload's row count (profiling)")
    ap.add_argument("--p", type=int, default=None, help="override the tile grid (profiling)")
    ap.add_argument("--K", type=int, default=None, help="override the number of factors (profiling)")
    ap.add_argument("--refresh-every", type=int, default=0,
                    help="second schedule: recompute G, A after every R inner rounds (0: once per epoch)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--log", default=None, help="append one JSON line per timed epoch to this file: epoch, objective, "
                                                "mean loss, seconds, updates/s, per-phase ms")
    ap.add_argument("--oracle-rows", type=int, default=ORACLE_SAMPLE_ROWS)
    ap.add_argument("--oracle-seconds", type=float, default=10.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-pin", dest="pin", action="store_false")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

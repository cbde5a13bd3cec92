#!/usr/bin/env python
"""Benchmark of the CoCoA round on one B200 (or N independent replicas on N GPUs).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

A step is one pass of the whole hot path over the workload: the round's visiting orders, the K local SCD
solvers, the aggregation of their updates, and the duality-gap evaluation. The workload is the sparse hinge-SVM
configuration (n = 1 000 000 rows, d = 100 000 features, about 50 non-zeros per row, K = 16 partitions, one
local epoch per round), synthetic and seeded. Prints one JSON line.

`--impl reference` times the CPU oracle (as it stands, on the host cores) on the same workload and metric.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "scd_coordinate_updates_per_s"
UNIT = "updates/s"
WORKLOAD = "hinge_csr"


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--scale", type=int, default=1, help="divide rows and columns (for quick checks only)")
    ap.add_argument("--e2e-steps", type=int, default=3, help="0 skips the end-to-end leg")
    ap.add_argument("--cpu-rounds", type=int, default=0,
                    help="oracle rounds for cpu_baseline (0 = pick from a probe round, negative = skip)")
    return ap.parse_args(argv)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


def workload_config(w, n_gpus):
    ph = w.phases[0]
    return {"workload": "config 2: hinge-SVM dual on sparse CSR, n=%d d=%d nnz=%d (Poisson(50)/row, Zipf(1.1) ids), "
                        "lambda=%g, K=%d random equal partitions, H=1 local epoch, sigma'=%g; step = visiting orders + "
                        "local solvers + aggregation + duality gap" % (w.n_rows, w.n_cols, w.nnz, w.lam, ph.K, ph.sigma_prime),
            "n": w.n_rows, "d": w.n_cols, "nnz": w.nnz, "K": ph.K, "H": "one local epoch",
            "l2": "inputs (%.0f MB of CSR) larger than the 126 MB L2" % ((w.nnz * 8 + w.n_rows * 8) / 1e6),
            "parallelism": "1 GPU" if n_gpus == 1 else "%d independent replicas, no collective" % n_gpus}


def algorithmic_bytes_per_round(w):
    """Compulsory HBM bytes of one local-solver launch: the row stream (value + index per non-zero, two indptr
    entries per coordinate) plus per-coordinate state (visiting-order entry, label, squared norm, alpha read and
    write). Second value: the same plus the v_local gathers and scatters (4 bytes each per non-zero)."""
    row_stream = w.nnz * 8 + w.n_coord * 16 + w.n_coord * 20
    return row_stream, row_stream + w.nnz * 8


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.path = tempfile.mktemp(prefix="clocks_", suffix=".csv")
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [t.strip() for t in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def max_over_ranks(dist, value, device=None):
    """Largest value over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized():
        return value
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate(units_per_rank, world, seconds_max):
    """Whole-job throughput: the units all ranks processed divided by the slowest rank's time."""
    return units_per_rank * world / seconds_max


def read_traffic():
    """DRAM bytes per local-solver launch from the committed ncu summary; None once the solver source has changed
    since the counters were taken."""
    import hashlib
    try:
        kv = dict(l.split() for l in open(os.path.join(ROOT, "profiles", "local_scd_traffic.txt")) if l.strip() and l[0] != "#")
        src = b"".join(open(os.path.join(ROOT, "paper_1909_04885_b200", "csrc", f), "rb").read()
                       for f in ("lookahead.cu", "solver_common.cuh"))
        if hashlib.sha256(src).hexdigest() != kv["solver_source_sha256"]:
            return None
        return int(kv["dram_bytes_per_launch"])
    except Exception:
        return None


def time_oracle(w, ph, rounds_arg):
    """The oracle, untuned, on a bounded sample of the workload: whole rounds (+ gap) on min(K, cores) threads."""
    import oracle
    cores = os.cpu_count() or 1
    threads = min(ph.K, cores)
    orc = oracle.CocoaOracle(w.loss, w.fmt, w.n_rows, w.n_cols, w.values, w.labels, w.lam, w.indptr, w.indices, threads=threads)
    orc.partition(ph.K, ph.seed)
    t0 = time.perf_counter()
    orc.cocoa_round(w.H, ph.sigma_prime)
    orc.duality_gap()
    probe = time.perf_counter() - t0
    rounds = rounds_arg or max(1, min(20, int(15.0 / max(probe, 1e-3))))
    t0 = time.perf_counter()
    for _ in range(rounds):
        orc.cocoa_round(w.H, ph.sigma_prime)
        orc.duality_gap()
    dt = time.perf_counter() - t0
    return {"value": w.n_coord * rounds / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "%d full rounds + gap of the whole workload after 1 probe round" % rounds}


def run_reference(args):
    """The oracle, as it stands, on the host cores: a step is one round plus the gap on the full workload."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    from paper_1909_04885_b200 import datagen
    w = datagen.make(WORKLOAD, args.scale)
    ph = w.phases[0]
    threads = min(ph.K, os.cpu_count() or 1)
    orc = oracle.CocoaOracle(w.loss, w.fmt, w.n_rows, w.n_cols, w.values, w.labels, w.lam, w.indptr, w.indices, threads=threads)
    orc.partition(ph.K, ph.seed)
    for _ in range(args.warmup):
        orc.cocoa_round(w.H, ph.sigma_prime)
        orc.duality_gap()
    t0 = time.perf_counter()
    g = None
    for _ in range(args.steps):
        orc.cocoa_round(w.H, ph.sigma_prime)
        g = orc.duality_gap()
    dt = time.perf_counter() - t0
    value = w.n_coord * args.steps / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(w, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": "%d full rounds + gap of the whole workload" % args.steps},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "final_gap": g["gap"] if g else None}
    print(json.dumps(line))


def run_b200(args):
    import torch

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", str(rank)))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the library has no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    from paper_1909_04885_b200 import binding, build, datagen
    if rank == 0:
        build.build()
    if dist is not None:
        dist.barrier()

    w = datagen.make(WORKLOAD, args.scale)
    ph = w.phases[0]
    comp_bytes, eff_bytes = algorithmic_bytes_per_round(w)
    warmup = max(args.warmup, 3)

    # ---- inputs resident in HBM before the timed region
    glm = binding.from_workload(w, device=local, on_device=True)
    glm.partition(ph.K, ph.seed)
    for _ in range(warmup):
        glm.cocoa_round(w.H, ph.sigma_prime)
        glm.duality_gap()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stats, gap = [], None
    torch.cuda.synchronize()
    start.record()
    gap_events = []
    for _ in range(args.steps):
        stats.append(glm.cocoa_round(w.H, ph.sigma_prime, stats=True))
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        gap = glm.duality_gap()
        g1.record()
        gap_events.append((g0, g1))
    stop.record()
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop)
    clocks = sampler.stop() if sampler else None
    if dist is not None:
        dist.barrier()
    ms_max = max_over_ranks(dist, ms, dev)
    value = aggregate(w.n_coord * args.steps, world, ms_max / 1e3)
    # outside the timed region: the prepare kernel alone. A long round is cut into slices whose prepare kernels run
    # beside the chain kernels; with the slicing off the prepare kernel has the GPU to itself and can be timed.
    os.environ["CHICLE_LA_SLICES"] = "1"
    alone = [glm.cocoa_round(w.H, ph.sigma_prime, stats=True) for _ in range(3)]
    del os.environ["CHICLE_LA_SLICES"]
    glm.close()

    # ---- time to a duality gap of 1e-3 from the zero state (the second half of the metric): rounds of one local
    #      epoch with the gap evaluated after every round, device time by CUDA events, at most 100 rounds
    time_to_gap = None
    if rank == 0:
        g3 = binding.from_workload(w, device=local, on_device=True)
        g3.partition(ph.K, ph.seed)
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        reached, gap_now, rounds_done = False, None, 0
        for r in range(100):
            g3.cocoa_round(w.H, ph.sigma_prime)
            gap_now = g3.duality_gap()["gap"]
            rounds_done = r + 1
            if gap_now <= 1e-3:
                reached = True
                break
        t1.record()
        torch.cuda.synchronize()
        time_to_gap = {"threshold": 1e-3, "reached": reached, "rounds": rounds_done, "ms": t0.elapsed_time(t1),
                       "gap": gap_now, "what": "absolute gap of the (1/n)-normalised objective, from alpha = 0; the "
                       "workload's own schedule has %d rounds" % w.rounds}
        g3.close()

    # ---- end to end through the C ABI with host buffers: create (H2D) + partition + round + gap + read-back (D2H)
    e2e = None
    if args.e2e_steps > 0:
        pinned = [torch.from_numpy(a).pin_memory().numpy() for a in (w.values, w.labels, w.indptr, w.indices)]
        h2d = sum(a.nbytes for a in pinned)
        v_host = torch.empty(w.n_cols, dtype=torch.float32).pin_memory().numpy()
        d2h = v_host.nbytes + 24
        e2e_ms = []
        for it in range(args.e2e_steps + 1):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            g2 = binding.Glm(w.loss, w.fmt, w.n_rows, w.n_cols, pinned[0], pinned[1], w.lam, pinned[2], pinned[3], device=local)
            g2.partition(ph.K, ph.seed)
            g2.cocoa_round(w.H, ph.sigma_prime)
            g2.duality_gap()
            g2.get_v(v_host)
            torch.cuda.synchronize()
            if it > 0:
                e2e_ms.append(1e3 * (time.perf_counter() - t0))
            g2.close()
        e2e_max = max_over_ranks(dist, statistics.mean(e2e_ms), dev)
        e2e = {"value": aggregate(w.n_coord, world, e2e_max / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_max,
               "what": "create from pinned host arrays + partition + one round + gap + read-back of v, per step"}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks, peak_kind = measured_peaks()
    ms_local = statistics.mean(s["ms_local"] for s in stats)
    ms_prep = statistics.mean(s["ms_prepare"] for s in stats)   # until the first chain launch starts
    ms_chain = ms_local - ms_prep                   # the latency-bound kernel: one CTA per partition; a long round's
    #                                                 launches of it (one per slice) together
    ms_prep_alone = statistics.mean(s["ms_prepare"] for s in alone)
    ms_local_alone = statistics.mean(s["ms_local"] for s in alone)
    n_k = w.n_coord // ph.K
    sliced = w.n_coord // 32 >= 4096 and n_k // 32 >= 64 and 2 * ph.K <= 148
    ms_perm = statistics.mean(s["ms_permutation"] for s in stats)
    ms_red = statistics.mean(s["ms_reduce"] for s in stats)
    ms_gap = statistics.mean(a.elapsed_time(b) for a, b in gap_events)
    gap_bytes = w.nnz * 8 + w.n_coord * 16          # row stream + label and alpha per coordinate
    red_bytes = (2 * ph.K + 2) * w.n_cols * 4       # reads and clears the K update rows, reads and writes v
    achieved = comp_bytes / (ms_chain * 1e-3) / 1e9
    # the prepare kernel reads every row once and writes (then the chain kernel reads) a record of about 16 bytes per
    # non-zero plus a 5.7 KB head per block of 32 steps
    prep_bytes = comp_bytes + w.nnz * 16 + (w.n_coord // 32) * 5728
    traffic = read_traffic() if args.scale == 1 else None
    owner_passes = 1 if ph.K <= 256 else 2
    solver_launches = 9 if sliced else 3            # per slice: block table, prepare, chain
    launches = 1 + 5 * (4 + owner_passes) + 1 + solver_launches + 1 + 2   # order keys, radix passes, run fix-up, solver, aggregation, gap (2)

    cpu_baseline = time_oracle(w, ph, args.cpu_rounds) if args.cpu_rounds >= 0 else None

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms_max / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": workload_config(w, world),
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches * args.steps,
            "roofline": {"bound": "hbm", "kernel": "k_lookahead_chain (local SCD solvers, one CTA per partition)", "achieved": achieved,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                         "peak_kind": "of " + peak_kind, "traffic": traffic,
                         "algorithmic_bytes_per_launch": comp_bytes,
                         "effective_gbs_with_gathers_and_scatters": eff_bytes / (ms_chain * 1e-3) / 1e9,
                         "whole_solver_gbs": comp_bytes / (ms_local * 1e-3) / 1e9,
                         "launches_per_round": 3 if sliced else 1,
                         "prepare_kernel": {"ms": ms_prep_alone, "bytes": prep_bytes, "gbs": prep_bytes / (ms_prep_alone * 1e-3) / 1e9,
                                            "frac": prep_bytes / (ms_prep_alone * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                            "note": "timed alone in 3 extra rounds with the slicing off (local solvers then "
                                                    "%.3f ms); in the timed rounds only the first slice's prepare is exposed" % ms_local_alone},
                         "note": "a partition is walked strictly in order: K dependent chains bound this kernel, not HBM"},
            "kernel_ms": {"visiting_orders": ms_perm, "local_solvers": ms_local, "local_solvers_prepare_exposed": ms_prep,
                          "local_solvers_chain": ms_chain, "aggregation": ms_red,
                          "gap_call": ms_gap, "host_and_sync": ms_max / args.steps - ms_perm - ms_local - ms_red - ms_gap},
            "streaming_kernels": {"gap_call_gbs": gap_bytes / (ms_gap * 1e-3) / 1e9,
                                  "gap_frac_of_hbm_peak": gap_bytes / (ms_gap * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                  "aggregation_gbs": red_bytes / (ms_red * 1e-3) / 1e9,
                                  "note": "gap_call = both gap kernels + the 24-byte read-back and its synchronise"},
            "chain": {"partitions": ph.K, "ns_per_coordinate_step": 1e6 * ms_chain / (w.n_coord / ph.K)},
            "cpu_baseline": cpu_baseline,
            "time_to_gap": time_to_gap,
            "final_gap": gap["gap"] if gap else None}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_b200(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the CoCoA round on one B200 (or one job spread over N GPUs: partitions k mod N on rank k).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--configs 4,1,2,3,5]

A step is one pass of the whole hot path over the workload: the round's visiting orders, the K local SCD solvers,
the aggregation of their updates, and the duality-gap evaluation. The headline workload is the largest one that
fits one GPU: the hinge-SVM dual on hashed sparse data with the shape of the paper's Criteo set (Table 1: 45 M rows,
1 M features, 39 non-zeros per row), synthetic and seeded, on its own elastic schedule (K = 64 partitions for the
first third of the steps, then a repartition into K = 16). The other four configurations are timed in the same run
and reported under "configs". Prints one JSON line.

`--impl reference` times the CPU oracle (as it stands, on the host cores) on the headline workload and metric.
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
CONFIGS = {1: "hinge_dense", 2: "hinge_csr", 3: "logistic_dense", 4: "hinge_hashed", 5: "ridge_csc"}
HEADLINE = 4
ON_GPU = {"hinge_hashed", "ridge_csc", "logistic_dense"}  # drawn with torch on the GPU (the CPU draw takes minutes)


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=12)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--scale", type=int, default=1, help="divide rows and columns (for quick checks and ncu captures only)")
    ap.add_argument("--configs", default="4,1,2,3,5", help="configurations to time; the first one is the headline")
    ap.add_argument("--e2e-steps", type=int, default=1, help="0 skips the end-to-end leg")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="oracle time per configuration (0 skips cpu_baseline)")
    ap.add_argument("--no-time-to-gap", action="store_true")
    return ap.parse_args(argv)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


def describe(w, cfg, n_gpus):
    shapes = {1: "config 1: hinge-SVM dual, dense N(0,1) rows", 2: "config 2: hinge-SVM dual on sparse CSR (Poisson(50) per row, Zipf(1.1) ids)",
              3: "config 3: logistic-regression dual on tall dense data (the shape of Higgs, Table 1)",
              4: "config 4: hinge-SVM dual on hashed sparse CSR with the shape of Criteo (Table 1), 39 Zipf(1.05) ids per row, elastic",
              5: "config 5: ridge regression primal, feature partitions on CSC"}
    sched = ", ".join("K=%d from round %d (sigma'=%g)" % (p.K, p.start, p.sigma_prime) for p in w.phases)
    data_mb = (w.nnz * 8 + w.n_coord * 8) / 1e6 if w.indptr is not None else w.values.size * 4 / 1e6
    return {"workload": "%s: n=%d d=%d nnz=%d, lambda=%g, %s, H=1 local epoch; step = visiting orders + local solvers + "
                        "aggregation + duality gap" % (shapes[cfg], w.n_rows, w.n_cols, w.nnz, w.lam, sched),
            "n": w.n_rows, "d": w.n_cols, "nnz": w.nnz, "H": "one local epoch",
            "l2": "inputs (%.0f MB) %s the 126 MB L2%s" % (data_mb, "larger than" if data_mb > 126 else "smaller than",
                                                          "" if data_mb > 126 else ": every round also rewrites the K x d update rows and the solver's records"),
            "parallelism": "1 GPU" if n_gpus == 1 else "one job on %d GPUs: rank g runs the partitions k mod %d = g; one all-gather of the "
                           "summed updates per round, one all-reduce of the per-coordinate state per gap evaluation" % (n_gpus, n_gpus)}


def algorithmic_bytes_per_round(w):
    """Compulsory HBM bytes of one round's local solvers: the row stream (value + index per non-zero, two indptr
    entries per coordinate; dense rows: the values) plus per-coordinate state (visiting-order entry, label, squared
    norm, alpha read and write). Second value: the same plus the local-model gathers and scatters (4 bytes each per
    non-zero)."""
    if w.indptr is None:
        row_stream = w.values.size * 4 + w.n_coord * 20
    else:
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


def throughput(units, seconds_max):
    """Whole-job throughput: the units the job processed divided by the slowest rank's time (with several ranks the
    job is one: its units are not multiplied by the number of ranks)."""
    return units / seconds_max


def read_profile_numbers():
    """Figures taken from committed ncu / timing-build summaries: DRAM bytes of the local solvers' kernels per
    coordinate step for the headline shape (captured at reduced size; None once the solver source has changed since),
    and the on-chip cost of one dependent step of the recurrence."""
    import hashlib
    out = {"traffic_bytes_per_step": None, "t_step_ns": None}
    try:
        kv = dict(l.split(None, 1) for l in open(os.path.join(ROOT, "profiles", "local_scd_traffic.txt")) if l.strip() and l[0] != "#")
        kv = {k: v.strip() for k, v in kv.items()}
        out["t_step_ns"] = float(kv["t_step_ns"])
        src = b"".join(open(os.path.join(ROOT, "paper_1909_04885_b200", "csrc", f), "rb").read()
                       for f in ("lookahead.cu", "solver_common.cuh"))
        if hashlib.sha256(src).hexdigest() == kv.get("solver_source_sha256"):
            out["traffic_bytes_per_step"] = float(kv["dram_bytes_per_step_config4"])
            out["traffic_note"] = kv.get("note")
    except Exception:
        pass
    return out


def schedule(w, steps):
    """The workload's own schedule squeezed into `steps` rounds: phase boundaries keep their share of the rounds."""
    bounds = []
    for i, p in enumerate(w.phases):
        at = 0 if i == 0 else max(1, min(steps - 1, round(p.start * steps / w.rounds)))
        bounds.append((at, p))
    return bounds


def make_workload(cfg, scale):
    from paper_1909_04885_b200 import datagen
    import torch
    name = CONFIGS[cfg]
    dev = "cuda" if (name in ON_GPU and scale == 1 and torch.cuda.is_available()) else "cpu"
    return datagen.make(name, scale, device=dev)


def time_oracle(w, seconds, min_rounds=3):
    """The oracle, untuned, on a bounded sample of the workload: whole rounds (+ gap) on min(K, cores) threads, on
    the workload's first phase. At least `min_rounds` rounds unless one round already exceeds the budget."""
    import oracle
    ph = w.phases[0]
    cores = os.cpu_count() or 1
    threads = min(ph.K, cores)
    orc = oracle.CocoaOracle(w.loss, w.fmt, w.n_rows, w.n_cols, w.values, w.labels, w.lam, w.indptr, w.indices, threads=threads)
    orc.partition(ph.K, ph.seed)
    rounds, t0 = 0, time.perf_counter()
    while True:
        orc.cocoa_round(w.H, ph.sigma_prime)
        orc.duality_gap()
        rounds += 1
        dt = time.perf_counter() - t0
        if (rounds >= min_rounds and dt >= seconds) or dt >= 3 * seconds or rounds >= 20:
            break
    return {"value": w.n_coord * rounds / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "%d full rounds + gap of the whole workload at K=%d (%.1f s); a round costs the same at every K, so "
                      "the figure stands for the whole schedule" % (rounds, ph.K, dt),
            "s_per_round": dt / rounds}


def run_reference(args):
    """The oracle, as it stands, on the host cores, on the headline workload: a step is one round plus the gap."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    cfg = int(args.configs.split(",")[0])
    w = make_workload(cfg, args.scale)
    threads_of = lambda K: min(K, os.cpu_count() or 1)
    ph0 = w.phases[0]
    orc = oracle.CocoaOracle(w.loss, w.fmt, w.n_rows, w.n_cols, w.values, w.labels, w.lam, w.indptr, w.indices, threads=threads_of(ph0.K))
    orc.partition(ph0.K, ph0.seed)
    for _ in range(args.warmup):
        orc.cocoa_round(w.H, ph0.sigma_prime)
        orc.duality_gap()
    bounds = schedule(w, args.steps)
    t0 = time.perf_counter()
    g = None
    for s in range(args.steps):
        for at, p in bounds:
            if at == s and s > 0:
                orc.threads = threads_of(p.K)
                orc.partition(p.K, p.seed)
        ph = [p for at, p in bounds if at <= s][-1]
        orc.cocoa_round(w.H, ph.sigma_prime)
        g = orc.duality_gap()
    dt = time.perf_counter() - t0
    value = w.n_coord * args.steps / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": describe(w, cfg, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads_of(ph0.K), "kind": "oracle",
                             "sample": "%d full rounds + gap of the whole workload on its schedule" % args.steps},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "final_gap": g["gap"] if g else None}
    print(json.dumps(line))


def run_config(cfg, w, steps, warmup, local, dist, dev, world, peaks, want_ttg, sampler_rank0):
    """Times `steps` rounds (+ gap) of one configuration on its own schedule, inputs resident in HBM. Returns the
    figures of that configuration."""
    import torch
    from paper_1909_04885_b200 import binding
    comp_bytes, eff_bytes = algorithmic_bytes_per_round(w)
    bounds = schedule(w, steps)
    handle = binding.from_workload(w, device=local, on_device=True)
    glm = handle
    if world > 1:
        # one job over the ranks: every rank holds the data and the replicated shared vector and runs the partitions
        # k mod world; the summed updates are exchanged once per round (strong scaling: the work is fixed)
        from paper_1909_04885_b200 import sharded
        glm = sharded.ShardedGlm(sharded.GlmBackend(handle), sharded.Comm(dist))
    ph0 = w.phases[0]
    glm.partition(ph0.K, ph0.seed)
    for _ in range(warmup):
        glm.cocoa_round(w.H, ph0.sigma_prime)
        glm.duality_gap()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local) if sampler_rank0 else None
    ev = lambda: torch.cuda.Event(enable_timing=True)
    start, stop = ev(), ev()
    stats, gap, gap_events, part_events, Ks = [], None, [], [], []
    torch.cuda.synchronize()
    start.record()
    for s in range(steps):
        for at, p in bounds:
            if at == s and s > 0:   # the elastic step: a new partition between two rounds, state kept
                p0, p1 = ev(), ev()
                p0.record()
                glm.partition(p.K, p.seed)
                p1.record()
                part_events.append((p0, p1))
        ph = [p for at, p in bounds if at <= s][-1]
        Ks.append(ph.K)
        stats.append(glm.cocoa_round(w.H, ph.sigma_prime, stats=True))
        g0, g1 = ev(), ev()
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
    value = throughput(w.n_coord * steps, ms_max / 1e3)
    handle.close()

    def mean(key, sel=None):
        xs = [s[key] for s, K in zip(stats, Ks) if sel is None or K == sel]
        return statistics.mean(xs) if xs else None

    ms_gap = statistics.mean(a.elapsed_time(b) for a, b in gap_events)
    per_phase = {}
    for K in sorted(set(Ks), reverse=True):
        loc, prep = mean("ms_local", K), mean("ms_prepare", K)
        chain = loc - prep
        per_phase["K=%d" % K] = {
            "rounds": Ks.count(K), "ms_local_solvers": loc, "ms_prepare_exposed": prep, "ms_chain_launches": chain,
            "ms_visiting_orders": mean("ms_permutation", K), "ms_aggregation": mean("ms_reduce", K),
            "updates_per_s_solvers_only": w.n_coord / (loc * 1e-3),
            "ns_per_coordinate_step_and_chain": 1e6 * chain / (w.n_coord / K),
            "hbm_gbs": comp_bytes / (chain * 1e-3) / 1e9, "hbm_frac": comp_bytes / (chain * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "aggregation_gbs": (2 * K + 2) * (w.n_rows if w.loss == "ridge" else w.n_cols) * 4 / (mean("ms_reduce", K) * 1e-3) / 1e9,
            "solver_slices": stats[Ks.index(K)]["solver_slices"], "cluster_ctas": stats[Ks.index(K)]["cluster_ctas"],
            "solver_variant": stats[Ks.index(K)]["solver_variant"]}
    gap_bytes = (w.nnz * 8 + w.n_coord * 16) if w.indptr is not None else (w.values.size * 4 + w.n_coord * 8)
    launches = sum(s["solver_launches"] + s["order_launches"] + 1 + 2 for s in stats)  # + aggregation + gap (2)
    out = {"value": value, "ms_per_step": ms_max / steps, "steps": steps, "per_phase": per_phase,
           "ms_gap_call": ms_gap, "gap_gbs": gap_bytes / (ms_gap * 1e-3) / 1e9,
           "gap_frac_of_hbm_peak": gap_bytes / (ms_gap * 1e-3) / 1e9 / peaks["hbm_gbs"],
           "ms_repartition": [a.elapsed_time(b) for a, b in part_events], "final_gap": gap["gap"] if gap else None,
           "gpu_launches": launches, "clocks": clocks, "algorithmic_bytes_per_round": comp_bytes,
           "effective_bytes_per_round_with_gathers_and_scatters": eff_bytes}

    # ---- time to a duality gap of 1e-3 from the zero state (the second half of the metric): the workload's own
    #      schedule, the gap evaluated after every round, device time by CUDA events; ridge: relative to P(0)
    if want_ttg:
        g3 = binding.from_workload(w, device=local, on_device=True)
        g3.partition(ph0.K, ph0.seed)
        p_zero = g3.duality_gap()["primal"]
        thr = 1e-3 * (p_zero if w.loss == "ridge" else 1.0)
        torch.cuda.synchronize()
        t0, t1 = ev(), ev()
        t0.record()
        reached, gap_now, done = False, None, 0
        for r in range(min(3 * w.rounds, 100)):
            ph = w.phase_at(r)
            if r > 0 and r == ph.start:
                g3.partition(ph.K, ph.seed)
            g3.cocoa_round(w.H, ph.sigma_prime)
            gap_now = g3.duality_gap()["gap"]
            done = r + 1
            if gap_now <= thr:
                reached = True
                break
        t1.record()
        torch.cuda.synchronize()
        out["time_to_gap"] = {"threshold": thr, "reached": reached, "rounds": done, "ms": t0.elapsed_time(t1), "gap": gap_now,
                              "what": "gap of the (1/n)-normalised objective%s, from the zero state, on the workload's own "
                                      "schedule (%d rounds), continued at the last K" % (" relative to P(0)" if w.loss == "ridge" else "", w.rounds)}
        g3.close()
    return out


def run_e2e(w, n_steps, local, dist, dev, world):
    """End to end through the C ABI with host buffers: create (host-to-device copies of the whole matrix from pinned
    memory) + partition + one round + gap + read-back of the shared vector, per step."""
    import torch
    from paper_1909_04885_b200 import binding
    ph = w.phases[0]
    arrays = [w.values, w.labels] + ([w.indptr, w.indices] if w.indptr is not None else [])
    pinned = [torch.from_numpy(a).pin_memory().numpy() for a in arrays]
    h2d = sum(a.nbytes for a in pinned)
    out_len = w.n_rows if w.loss == "ridge" else w.n_cols
    v_host = torch.empty(out_len, dtype=torch.float32).pin_memory().numpy()
    d2h = v_host.nbytes + 24
    times = []
    for it in range(n_steps + 1):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        g2 = binding.Glm(w.loss, w.fmt, w.n_rows, w.n_cols, pinned[0], pinned[1], w.lam,
                         pinned[2] if len(pinned) > 2 else None, pinned[3] if len(pinned) > 2 else None, device=local)
        job = g2
        if world > 1:   # the same job over the ranks (every rank uploads the data and keeps a replica of v)
            from paper_1909_04885_b200 import sharded
            job = sharded.ShardedGlm(sharded.GlmBackend(g2), sharded.Comm(dist))
        job.partition(ph.K, ph.seed)
        job.cocoa_round(w.H, ph.sigma_prime)
        job.duality_gap()
        g2.get_v(v_host)
        torch.cuda.synchronize()
        if it > 0:
            times.append(1e3 * (time.perf_counter() - t0))
        g2.close()
    e2e_max = max_over_ranks(dist, statistics.mean(times), dev)
    return {"value": throughput(w.n_coord, e2e_max / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": e2e_max,
            "what": "create from pinned host arrays + partition (K=%d) + one round + gap + read-back of v, per step" % ph.K}


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
    from paper_1909_04885_b200 import build
    if rank == 0:
        build.build()
    if dist is not None:
        dist.barrier()

    peaks, peak_kind = measured_peaks()
    cfgs = [int(c) for c in args.configs.split(",") if c.strip()]
    head = cfgs[0]
    warmup = max(args.warmup, 3)
    results, e2e, cpu = {}, None, {}
    for cfg in cfgs:
        if cfg != head and rank != 0:
            continue   # the other configurations are single-GPU figures, taken on rank 0
        w = make_workload(cfg, args.scale)
        is_head = cfg == head
        steps = args.steps if is_head else max(3, min(args.steps, 3 * len(w.phases) + 3))
        res = run_config(cfg, w, steps, warmup, local, dist if is_head else None, dev, world if is_head else 1, peaks,
                         want_ttg=(rank == 0 and not args.no_time_to_gap), sampler_rank0=(is_head and rank == 0))
        res["config"] = describe(w, cfg, world if is_head else 1)
        if is_head and args.e2e_steps > 0:
            e2e = run_e2e(w, args.e2e_steps, local, dist, dev, world)
        if rank == 0 and args.cpu_seconds > 0:
            res["cpu_baseline"] = time_oracle(w, args.cpu_seconds)
        results[cfg] = res
        del w
        torch.cuda.empty_cache()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    H = results[head]
    prof = read_profile_numbers()
    # the dominant kernel of the headline workload: the chain launches of its longest phase (smallest K)
    dom_key = sorted(H["per_phase"], key=lambda k: H["per_phase"][k]["ms_chain_launches"] * H["per_phase"][k]["rounds"])[-1]
    dom = H["per_phase"][dom_key]
    n_head = H["config"]["n"]
    K_dom = int(dom_key.split("=")[1])
    chain_roof = None
    if prof["t_step_ns"]:
        peak_updates = K_dom / (prof["t_step_ns"] * 1e-9)
        got = n_head / (dom["ms_chain_launches"] * 1e-3)
        chain_roof = {"t_step_ns": prof["t_step_ns"], "chains": K_dom, "peak_updates_per_s": peak_updates,
                      "achieved_updates_per_s": got, "frac": got / peak_updates,
                      "what": "K dependent chains, each bounded by the on-chip cost of one step of the scalar recurrence "
                              "(measured with cycle counters in the recurrence warp, see profiles/)"}
    traffic = prof["traffic_bytes_per_step"] * n_head if (prof["traffic_bytes_per_step"] and args.scale == 1 and head == HEADLINE) else None
    line = {"metric": METRIC, "value": H["value"], "unit": UNIT, "n_gpus": world, "steps": H["steps"], "warmup": warmup,
            "ms_per_step": H["ms_per_step"], "higher_is_better": True, "scaling": "weak" if world == 1 else "strong", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": H["config"], "clocks": H["clocks"], "e2e": e2e,
            "gpu_launches": H["gpu_launches"],
            "roofline": {"bound": "hbm", "kernel": "k_lookahead_chain at %s (local SCD solvers: one thread-block cluster per partition)" % dom_key,
                         "achieved": dom["hbm_gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": dom["hbm_frac"],
                         "peak_kind": "of " + peak_kind, "traffic": traffic, "traffic_note": prof.get("traffic_note"),
                         "traffic_detail": None if traffic is None else {
                             "bytes": traffic, "captured_at_scale": 16, "extrapolated": True,
                             "covers": "all chain launches of one round (19 at full size); bytes per coordinate step "
                                       "from the ncu capture at 1/16 size times the steps of a round"},
                         "algorithmic_bytes_per_launch": H["algorithmic_bytes_per_round"],
                         "note": "a partition is walked strictly in order: K dependent chains and the throughput of the "
                                 "prepare kernel bound the local solvers, not HBM; achieved = algorithmic bytes of a round / time "
                                 "of the round's chain launches"},
            "chain_roofline": chain_roof,
            "per_phase": H["per_phase"], "ms_repartition": H["ms_repartition"],
            "streaming_kernels": {"gap_call_ms": H["ms_gap_call"], "gap_call_gbs": H["gap_gbs"], "gap_frac_of_hbm_peak": H["gap_frac_of_hbm_peak"],
                                  "aggregation_gbs": {k: v["aggregation_gbs"] for k, v in H["per_phase"].items()},
                                  "note": "gap_call = both gap kernels + the 24-byte read-back and its synchronise"},
            "cpu_baseline": H.get("cpu_baseline"), "time_to_gap": H.get("time_to_gap"), "final_gap": H["final_gap"],
            "configs": {str(c): {k: v for k, v in r.items() if k != "clocks"} for c, r in results.items() if c != head}}
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

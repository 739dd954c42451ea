#!/usr/bin/env python
"""Benchmark of the LAQ hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
                    [--no-configs] [--no-cpu-baseline] [--sustained-steps S]

A step is one LAQ iteration (Algorithm 2: local gradients, quantizer, norms, skip rule, lazy aggregate and
theta step) over all M workers of the workload.  Prints one JSON line (rank 0).  Workloads:
c4_b8 (default: M = 64, p = 25.6 M, b = 8, gradients generated in the kernels), c4_b4, c4_b2,
c4_b8_stored (the same stream written to memory by step 1 and read back by the sweeps),
c4_b8_xi0 (every worker uploads), c4_b8_frozen (no drift: uploads die out), c4_b8_M8 (8 workers: a small case
for profiler captures), c0, c1, c2, c3 (model workloads).
The default run (one GPU) also reports, under "configs", a short run of every other configuration and, under
"sustained", a longer run of the headline workload with the clocks it settled at.
With N > 1 (torchrun) every rank runs an independent replica of the workload on its own GPU: the path does
not shard across GPUs and has no collective; the timing is the maximum over ranks.
"""
import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "LAQ iters/s for M workers on 1 B200; quantize+trigger GB/s vs HBM peak"
FALLBACK_HBM_GBS = 6650.0
STAGES = ["local_gradient", "radius", "quantize_norms_trigger", "aggregate_theta_step"]
STAGE_KERNELS = {"radius": "radius_kernel", "quantize_norms_trigger": "quantize_kernel",
                 "aggregate_theta_step": "aggregate_kernel", "local_gradient": "grad_*_kernel"}
TRAJ_RTOL = 1e-4          # band of theta and loss around the fp64 oracle's while skip decisions agree

MODE_FLAGS = {"lag": 1, "qgd": 2, "gd": 3, "stored": 4, "sparse": 8, "sharded": 0}   # quantizer off, trigger off, both, g through memory (LAQ_FLAG_*)

# short runs of the other configurations in the default line: (workload, timed steps)
CONFIG_RUNS = [("c0", 2000), ("c1", 500), ("c2", 1000), ("c3", 300), ("c4_b4", 100), ("c4_b2", 100),
               ("c4_b8_stored", 100)]
# iterations of the free-running fp64 oracle per model workload (timed: its cost is that workload's CPU baseline)
ORACLE_ITERS = {"c0": 200, "c1": 16, "c2": 120, "c3": 2}


def make_workload(name):
    """c4_b8 (default), c4_b{2,3,4}, c4_b8_M8, c0..c3; suffixes _lag, _qgd, _gd select the baseline modes,
    _stored the stored-gradient mode of the synthetic stream, and _batchN minibatch gradients (model workloads),
    e.g. c1_b3_batch500."""
    w = _base_workload(name)
    w.flags, w.batch = 0, 0
    for part in name.split("_")[1:]:
        if part in MODE_FLAGS:
            w.flags |= MODE_FLAGS[part]
        elif part.startswith("batch") and part[5:].isdigit():
            w.batch = int(part[5:])
        elif part.startswith("b") and part[1:].isdigit() and not name.startswith("c4"):
            w.b = int(part[1:])
    return w


def _base_workload(name):
    from paper_1909_07588_b200 import workloads as W
    if name.startswith("c4"):
        parts = name.split("_")
        b = int(parts[1][1:]) if len(parts) > 1 else 8
        kw = {}
        if "xi0" in parts:
            kw["xi_scale"] = 0.0
        if "frozen" in parts:
            kw["eta0"] = 0.0
        for part in parts:                      # e.g. c4_b8_M8: fewer workers, a 1 GB case for profiler captures
            if part.startswith("M") and part[1:].isdigit():
                kw["M"] = int(part[1:])
        return W.c4(b=b, **kw)
    base = name.split("_")[0]
    if base == "c2":
        # a small random start: at theta = 0 every residual is +-1/2 and the gradient of a rarely active one-hot
        # column can cancel to exactly 0, a point midway between two grid values, where fp32 and fp64 may pick
        # different, equally near codes in the very first iteration
        return W.c2(theta0_scale=0.01)
    return {"c0": W.c0, "c1": W.c1, "c3": W.c3}[base]()


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


def tensor_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json bf16_tflops_sustained)"
    except Exception:
        return 1400.0, "fallback (earlier measurement on this pool, sustained)"


def algorithmic_bytes(w, u):
    """Bytes the method must move per iteration, per stage: Q_prev (and a stored g) read once per sweep, codes
    written once, and per uploader codes read and Q_prev rewritten; theta and the aggregate read and written.
    u = uploading fraction |M^k| / M averaged over the timed iterations."""
    Mp = float(w.M) * w.p
    flags = getattr(w, "flags", 0)
    stored = w.model != 3 or bool(flags & 4)
    g_bytes = 4.0 if stored else 0.0                # g read from HBM unless generated in the sweeps
    batch = getattr(w, "batch", 0)
    rows = [min(n, batch) if batch else n for n in w.N]
    X_bytes = sum(n * w.n_features * 4.0 + n * 4.0 for n in rows) if w.X else 0.0
    grad = X_bytes + (Mp * 4.0 if stored else 0.0)  # step 1: the shard read once, g written once
    if flags & 1:                                   # quantizer off: one sweep for radius and norm, raw innovations
        return {"local_gradient": grad, "radius": 0.0, "quantize_norms_trigger": Mp * (4.0 + g_bytes),
                "aggregate_theta_step": u * Mp * (8.0 + g_bytes) + 16.0 * w.p}
    return {"local_gradient": grad, "radius": Mp * (4.0 + g_bytes),
            "quantize_norms_trigger": Mp * (4.0 + g_bytes + w.b / 8.0),
            "aggregate_theta_step": u * Mp * (8.0 + w.b / 8.0) + 16.0 * w.p}


def max_over_ranks(x, world, device="cuda"):
    """The slowest rank's time decides: maximum of a per-rank scalar over all ranks (identity for one rank)."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replicas_throughput(world, steps, ms):
    """Whole-job iterations/s of `world` independent replicas that each ran `steps` iterations in `ms` (max over ranks)."""
    return world * steps / (ms * 1e-3)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index, period_ms=100):
        self.rows, self.proc, self.index, self.period_ms = [], None, index, period_ms

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], None, set(), []
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
                power.append(float(r[2]))
            except Exception:
                continue
            for name, col in (("hw_slowdown", 4), ("hw_thermal_slowdown", 5), ("sw_thermal_slowdown", 6),
                              ("sw_power_cap", 7)):
                if len(r) > col and r[col].lower().startswith("active"):
                    reasons.add(name)
        busy = [v for v in sm if mx and v > 0.5 * mx] or sm
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power) if power else None}


def traffic_for(stage, w):
    """DRAM bytes per launch from the committed ncu capture, or None if the kernel source changed since."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            rec = json.load(f)
        h = hashlib.sha256()
        for name in rec["sources"]:
            h.update(open(os.path.join(ROOT, "paper_1909_07588_b200", "csrc", name), "rb").read())
        if h.hexdigest() != rec["sources_sha256"]:
            return None
        key = "c4_b%d%s" % (w.b, "_stored" if getattr(w, "flags", 0) & 4 else "")
        per_coord = rec["bytes_per_worker_coordinate"][key][stage]
        return None if per_coord is None or w.model != 3 else per_coord * float(w.M) * w.p
    except Exception:
        return None


# ------------------------------------------------------------------------------------------------------------
# CPU legs: the oracle as it stands, timed on the host cores
# ------------------------------------------------------------------------------------------------------------
def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def _available_host_bytes():
    try:
        import psutil
        return int(psutil.virtual_memory().available)
    except Exception:
        return 0


def _oracle_for(w, p=None, precision=None):
    import oracle
    if w.model == 3:
        return oracle.OracleLaq(32 if precision is None else precision, oracle.MODEL_SYNTH, w.M, w.p if p is None else p,
                                alpha=w.alpha, b=w.b, D=w.D, xi=w.xi, tbar=w.tbar, seed=w.seed,
                                synth_sigma=w.synth_sigma, synth_eta0=w.synth_eta0, flags=w.flags & 3)
    o = oracle.OracleLaq(64 if precision is None else precision, w.model, w.M, w.p, N=w.N, n_features=w.n_features,
                         n_classes=w.n_classes, n_hidden=w.n_hidden, alpha=w.alpha, lam=w.lam, b=w.b, D=w.D, xi=w.xi,
                         tbar=w.tbar, bf16_ops=w.bf16_ops, theta0=w.theta0, seed=w.seed, flags=w.flags & 3, batch=w.batch)
    for m in range(w.M):
        o.set_shard(m, w.X[m], w.y[m])
    return o


def cpu_baseline(w, name, steps=None, warmup=1, budget_s=30.0):
    """The oracle as it stands on ONE host thread.  The large synthetic workload runs at full size when the host
    has the memory for the oracle's state (it keeps Q_prev, g, dQ and the codes as plain arrays: about 20 bytes per
    worker-coordinate), at least two iterations; otherwise on the first 1.6 M coordinates of every worker, scaled,
    and the sample text says so.  With `steps` given (the reference arm) it runs that many iterations after
    `warmup`, but stops when `budget_s` is used up."""
    import oracle
    oracle.build()
    scale, what = 1.0, "fp64 oracle, full workload"
    if w.model == 3:
        need = 24.0 * w.M * w.p
        if _available_host_bytes() > 1.5 * need:
            o = _oracle_for(w)
            what = "fp32 mirror, M=%d workers, all %d coordinates (full size)" % (w.M, w.p)
        else:
            p_s = min(w.p, 1_600_000)
            o = _oracle_for(w, p=p_s)
            scale = p_s / float(w.p)
            what = ("fp32 mirror, M=%d workers, first %d of %d coordinates (the host lacks the %.0f GB the oracle's "
                    "state needs at full size)" % (w.M, p_s, w.p, need / 1e9))
    else:
        o = _oracle_for(w)
    t_w = time.time()
    for _ in range(max(1, warmup)):
        o.step()
        if time.time() - t_w > budget_s / 3:
            break
    t0 = time.time()
    n = 0
    limit = steps if steps is not None else 10 ** 9
    while n < limit and (n < 2 or time.time() - t0 < budget_s):
        o.step()
        n += 1
    dt = time.time() - t0
    return {"value": n / dt * scale, "unit": "iters/s", "cores": 1, "host_cores": host_cores(), "kind": "oracle",
            "steps_timed": n, "seconds": dt,
            "sample": "%s, %d iterations after warm-up%s" % (
                what, n, "; iterations/s scaled by %g (cost is linear in p)" % scale if scale != 1.0 else "")}


def _all_core_worker(args):
    """One worker's steps 1-3 with the oracle's stateless routines (runs in a pool process)."""
    import oracle
    seed, m, M, p, b, sigma, eta0 = args
    g = oracle.synth_gradient(seed, m, M, p, 1, sigma, eta0)
    r = oracle.quantize(g, np.zeros(p, np.float32), b, np.float32)
    return float(r["n_dq"])


def cpu_all_cores(w, budget_workers=None):
    """The untouched oracle on every host core: its stateless generator and quantizer (steps 1-3 of an iteration,
    which are independent per worker) over disjoint workers in a process pool started with `spawn`.  Steps 4-5 (a
    few scalars and one pass over the uploaders) stay out: what is reported is workers/s turned into iterations/s of
    steps 1-3."""
    import multiprocessing as mp
    import oracle
    oracle.build()
    cores = host_cores()
    # a pool process holds one worker's vectors (g, Q_prev, codes, dQ, Q_new, eps): about 28 bytes per coordinate
    by_memory = max(1, int(_available_host_bytes() * 0.5 / (28.0 * w.p))) if _available_host_bytes() else 4
    cores = max(1, min(cores, by_memory))
    n_workers = w.M if budget_workers is None else min(w.M, budget_workers)
    jobs = [(w.seed, m, w.M, w.p, w.b, w.synth_sigma, w.synth_eta0) for m in range(n_workers)]
    ctx = mp.get_context("spawn")
    with ctx.Pool(processes=min(cores, n_workers)) as pool:      # leaving the block terminates the pool
        # start-up, library load, page faults; every wait on the pool is bounded
        pool.map_async(_all_core_worker, jobs[:min(cores, n_workers)]).get(timeout=120)
        t0 = time.time()
        pool.map_async(_all_core_worker, jobs, chunksize=1).get(timeout=240)
        dt = time.time() - t0
    return {"value": (n_workers / dt) / w.M, "unit": "iters/s (steps 1-3 only)", "cores": min(cores, n_workers),
            "host_cores": host_cores(), "kind": "oracle",
            "sample": "stateless generator + quantizer of the fp32 mirror, %d of %d workers at full p = %d with Q_prev = 0, "
                      "one worker per pool process" % (n_workers, w.M, w.p)}


def first_disagreement(w, n):
    """The free-running fp64 oracle (timed: this is the workload's CPU baseline) against a fresh context stepped one
    iteration at a time: first iteration at which a skip bit differs or theta / the loss leaves the 1e-4 band."""
    from paper_1909_07588_b200 import laq
    o = _oracle_for(w)
    rows = []
    t0 = time.time()
    for _ in range(n):
        st = o.step()
        rows.append((st["skip"].astype(np.uint8), float(st["loss"]), o.state(big=False)["theta"]))
    dt = time.time() - t0
    ctx = laq.from_workload(w, trace_capacity=1, flags=w.flags, batch=w.batch)
    first = None
    for k in range(n):
        tr = ctx.step(1, trace=True)
        th = ctx.get_state(big=False)["theta"]
        skip, loss, th64 = rows[k]
        if (not np.array_equal(skip, tr["skip"][0]) or np.linalg.norm(th - th64) > TRAJ_RTOL * np.linalg.norm(th64)
                or abs(tr["loss"][0] - loss) > TRAJ_RTOL * abs(loss)):
            first = k + 1
            break
    ctx.close()
    return first, {"value": n / dt, "unit": "iters/s", "cores": 1, "host_cores": host_cores(), "kind": "oracle",
                   "sample": "fp64 oracle, full workload, %d iterations from the start" % n}


def run_reference(args, w, name, rank):
    """--impl reference: the paper ships no code, so the reference arm is the CPU oracle (rank 0 only)."""
    if rank != 0:
        return
    t0 = time.time()
    base = cpu_baseline(w, name, steps=args.steps, warmup=1, budget_s=150.0)
    val = base["value"]
    # the oracle runs full-size iterations until the requested number is done or its time budget is used up:
    # "steps" is what was timed, so that ms_per_step x steps is the timed region
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "iters/s", "n_gpus": args.gpus,
            "steps": base["steps_timed"], "steps_requested": args.steps, "warmup": 1, "ms_per_step": 1000.0 / val,
            "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(w, name, 1, None),
            "cpu_baseline": base,
            "e2e": {"value": val, "unit": "iters/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": time.time() - t0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------------------
# GPU legs
# ------------------------------------------------------------------------------------------------------------
def workload_config(w, name, world, ctx):
    cfg = {"workload": name, "name": w.name, "M": w.M, "p": w.p, "b": w.b, "D": w.D, "tbar": w.tbar,
           "alpha": w.alpha, "flags": w.flags, "batch": w.batch, "parallelism": "replicas x%d" % world}
    if ctx is not None:
        cfg["l2"] = ("no flush: the state swept every iteration (%.1f GB) exceeds the 126 MB L2" % (ctx.workspace_bytes / 1e9)
                     if ctx.workspace_bytes > 4e8 else "no flush: working set is L2 resident by design of the workload")
    return cfg


def stage_table(w, stage_ms, stage_n, u, peak):
    """Per-stage milliseconds (averaged over the bracketed iterations), algorithmic bytes and fraction of the copy peak."""
    abytes = algorithmic_bytes(w, u)
    stages = []
    iters_recorded = int(stage_n[3])          # one aggregate launch per iteration; at most 512 iterations are bracketed
    for i, name in enumerate(STAGES):
        if stage_n[i] == 0 or iters_recorded == 0:
            continue
        if (w.flags & 1) and name == "radius":
            continue                            # quantizer off: radius and norm share one sweep (the next slot)
        avg_ms = stage_ms[i] / iters_recorded  # per iteration (the gradient stage may be several launches)
        gbs = abytes[name] / (avg_ms * 1e-3) / 1e9 if avg_ms > 0 else 0.0
        kern = STAGE_KERNELS[name]
        if w.flags & 1:
            kern = {"quantize_kernel": "innovation_kernel", "aggregate_kernel": "aggregate_raw_kernel"}.get(kern, kern)
        if name == "local_gradient" and w.model == 3:
            kern = "synth_fill_kernel"
        stages.append({"stage": name, "kernel": kern, "ms": avg_ms, "bytes": abytes[name],
                       "GB/s": gbs, "frac": gbs / peak, "share": stage_ms[i] / max(stage_ms.sum(), 1e-12)})
    if w.model != 3 and w.M * ((w.p + 15) // 16 * 16) <= 8192 and not (w.flags & 1):
        # small problems run steps 2-5 in one single-block kernel: its time sits in the last slot, the radius and
        # quantize slots are empty; it moves the bytes of all three sweeps
        last = stages[-1]
        last.update({"stage": "steps_2_to_5_single_block", "kernel": "small_iteration_kernel",
                     "bytes": abytes["radius"] + abytes["quantize_norms_trigger"] + abytes["aggregate_theta_step"]})
        last["GB/s"] = last["bytes"] / (last["ms"] * 1e-3) / 1e9 if last["ms"] > 0 else 0.0
        last["frac"] = last["GB/s"] / peak
        stages = [st for st in stages if st["stage"] not in ("radius", "quantize_norms_trigger")]
    return stages


def roofline_of(w, stages, u, peak, peak_src, timing_note):
    dom = max(stages, key=lambda s: s["ms"])
    path_bytes = sum(s["bytes"] for s in stages)
    path_ms = sum(s["ms"] for s in stages)
    roofline = {"bound": "hbm", "kernel": dom["kernel"], "achieved": dom["GB/s"], "peak": peak, "unit": "GB/s",
                "frac": dom["frac"], "traffic": traffic_for(dom["stage"], w), "peak_source": peak_src,
                "bytes_per_launch": dom["bytes"], "ms_per_launch": dom["ms"], "upload_fraction": u,
                "stage_timing": timing_note, "stages": stages,
                "whole_path": {"bytes_per_iter": path_bytes, "GB/s": path_bytes / (path_ms * 1e-3) / 1e9,
                               "frac": path_bytes / (path_ms * 1e-3) / 1e9 / peak}}
    if w.model == 2:
        # the network's gradient stage is two dense bf16 products (X W1^T and dH^T X): a tensor-core roofline
        g_stage = [st for st in stages if st["stage"] == "local_gradient"][0]
        rows = [min(n, w.batch) if w.batch else n for n in w.N]
        flops = 4.0 * sum(rows) * w.n_features * w.n_hidden
        tpeak, tsrc = tensor_peak()
        tf = flops / (g_stage["ms"] * 1e-3) / 1e12
        roofline.update({"bound": "tensor", "kernel": "network gradient stage (hidden-layer product with fused epilogue, W1-gradient product)",
                         "achieved": tf, "peak": tpeak, "unit": "TFLOP/s", "frac": tf / tpeak, "traffic": None,
                         "peak_source": tsrc, "flops_per_launch": flops, "ms_per_launch": g_stage["ms"]})
    return roofline


def run_timed(w, K, Wm, world, local_rank, barrier):
    """W warm-up and K timed iterations of one workload (inputs resident), per-stage CUDA events on the library's
    stream.  Returns (ctx, result dict)."""
    import torch
    from paper_1909_07588_b200 import laq
    ctx = laq.from_workload(w, trace_capacity=1, flags=w.flags, batch=w.batch)
    ctx.step(Wm)
    ctx.sync()
    s0 = ctx.get_state(big=False)
    sampler = ClockSampler(local_rank)
    sampler.start()
    # Per-stage CUDA events (on the library's stream) cost a few microseconds per iteration: nothing against the
    # millisecond iterations of the large-p workload, where they bracket the stages of the timed region itself;
    # for the small model workloads they would distort the number, so there the stages are timed over the K
    # iterations that follow the timed region.
    inline_events = w.model == 3
    launches0 = ctx.kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if inline_events:
        ctx.set_profiling(True)
        ctx.kernel_times()
    barrier()
    e0.record()
    ctx.step(K)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = ctx.kernel_launches() - launches0
    if inline_events:
        stage_ms, stage_n = ctx.kernel_times()
        ctx.set_profiling(False)
        s1, s2 = s0, ctx.get_state(big=False)
    else:
        s1 = ctx.get_state(big=False)
        ctx.set_profiling(True)
        ctx.kernel_times()
        ctx.step(min(K, 512))
        stage_ms, stage_n = ctx.kernel_times()
        ctx.set_profiling(False)
        s2 = ctx.get_state(big=False)
    clocks = sampler.stop()
    ms = max_over_ranks(ms, world)
    n_staged = K if inline_events else min(K, 512)
    u = (s2["uploads"] - s1["uploads"]) / float(n_staged * w.M)       # of the iterations whose stages were timed
    peak, peak_src = hbm_peak()
    stages = stage_table(w, stage_ms, stage_n, u, peak)
    note = ("CUDA events around every stage inside the timed region" if inline_events else
            "CUDA events around every stage over the %d iterations that follow the timed region" % n_staged)
    return ctx, {"ms": ms, "launches": int(launches), "clocks": clocks, "u": u,
                 "roofline": roofline_of(w, stages, u, peak, peak_src, note)}


def run_sustained(ctx, w, steps, local_rank):
    """A longer run of the same context: the power cap pulls the SM clock down within a second or two, and the
    issue-bound quantize sweep follows the clock.  Reports the stage fractions beside the median SM clock and the
    clock-normalised step time (ms x MHz), so that burst and capped figures can be told apart."""
    import torch
    peak, peak_src = hbm_peak()
    sampler = ClockSampler(local_rank, period_ms=50)
    sampler.start()
    ctx.step(steps)                               # settle under load
    ctx.sync()
    s1 = ctx.get_state(big=False)
    ctx.set_profiling(True)
    ctx.kernel_times()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = min(steps, 512)
    e0.record()
    ctx.step(n)
    e1.record()
    torch.cuda.synchronize()
    stage_ms, stage_n = ctx.kernel_times()
    ctx.set_profiling(False)
    clocks = sampler.stop()
    s2 = ctx.get_state(big=False)
    u = (s2["uploads"] - s1["uploads"]) / float(n * w.M)
    ms = e0.elapsed_time(e1) / n
    stages = stage_table(w, stage_ms, stage_n, u, peak)
    out = {"steps_before": steps, "steps": n, "ms_per_step": ms, "value": 1000.0 / ms, "unit": "iters/s",
           "clocks": clocks, "upload_fraction": u,
           "ms_x_mhz": ms * clocks["sm_mhz"] if clocks.get("sm_mhz") else None,
           "stages": [{k: s[k] for k in ("stage", "kernel", "ms", "GB/s", "frac")} for s in stages]}
    dom = max(stages, key=lambda s: s["ms"])
    out.update({"kernel": dom["kernel"], "frac": dom["frac"], "peak": peak, "peak_source": peak_src})
    return out


def run_e2e(w, Ke, world, barrier):
    """The same metric end to end through the C ABI with host buffers: context creation (theta0 and the shards
    cross PCIe), one laq_step with its report read back per iteration, the final iterate read back."""
    import torch
    from paper_1909_07588_b200 import laq
    theta0_pin = torch.zeros(w.p, dtype=torch.float32).pin_memory()           # pinned host memory both ways
    if w.theta0 is not None:
        theta0_pin.copy_(torch.from_numpy(np.asarray(w.theta0, np.float32)))
    theta_out_pin = torch.empty(w.p, dtype=torch.float32).pin_memory()
    barrier()
    t0 = time.perf_counter()
    ctx2 = laq.from_workload(w, trace_capacity=1, theta0=theta0_pin.numpy(), flags=w.flags, batch=w.batch)
    tr_bytes = 0
    for _ in range(Ke):
        tr = ctx2.step(1, trace=True)                                     # per-step report read back to the host
        tr_bytes = sum(v.nbytes for v in tr.values())
    final = ctx2.get_state(big=False, agg=False, buffers={"theta": theta_out_pin.numpy()})   # the iterate comes back
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s, world)
    ctx2.close()
    shard_bytes = sum(x.nbytes + y.nbytes for x, y in zip(w.X, w.y))
    return {"value": world * Ke / e2e_s, "unit": "iters/s", "steps": Ke,
            "h2d_bytes_per_step": (w.p * 4 + shard_bytes) / float(Ke),
            "d2h_bytes_per_step": tr_bytes + final["theta"].nbytes / float(Ke),
            "includes": "laq_init (theta0 H2D from pinned memory), laq_load_shards (H2D), laq_step(1, trace) per step, "
                        "final laq_get_state (theta D2H into pinned memory)"}


def run_sharded(args, w, K, Wm, world, rank, local_rank, barrier):
    """Workload suffix _sharded: the M workers are spread over the ranks (strong scaling) and every iteration
    exchanges the uploaders' messages (radius + code stream) over NCCL; see paper_1909_07588_b200/sharded.py.
    With one rank it runs the same split iteration without a collective."""
    import torch
    from paper_1909_07588_b200 import laq, sharded
    job = sharded.ShardedLaq(lambda wd, r: laq.from_workload(w, flags=w.flags, batch=w.batch, world=wd if wd > 1 else 0,
                                                             rank=r if wd > 1 else 0), world, rank)
    job.step(Wm)
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = job.ctx.kernel_launches()
    sent0 = job.sent_payload_bytes
    barrier()
    e0.record()
    job.step(K)
    e1.record()
    barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), world)
    clocks = sampler.stop()
    s = job.ctx.get_state(big=False)
    line = {"metric": METRIC, "value": K / (ms * 1e-3), "unit": "iters/s", "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": dict(workload_config(w, args.workload, world, job.ctx),
                                                parallelism="workers spread over %d ranks, (R, codes) exchange" % world),
            "clocks": clocks, "gpu_launches": int(job.ctx.kernel_launches() - launches0),
            "exchange": {"payload_bytes_sent_per_step_this_rank": (job.sent_payload_bytes - sent0) / float(K),
                         "uploads_per_step_all_ranks": None, "bits_counted": int(s["bits"]),
                         "host_round_trips_per_step": 1},
            "e2e": None, "roofline": None, "cpu_baseline": None}
    job.close()
    if rank == 0:
        print(json.dumps(line), flush=True)


def two_kernel_graph_floor_us(iters=2000):
    """Launch floor of a two-kernel iteration on this machine: a CUDA graph of eight iterations of two dependent,
    almost empty kernels (torch element-wise adds on one float), replayed back to back; microseconds per iteration."""
    import torch
    x = torch.zeros(1, device="cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for _ in range(3):
            x.add_(1.0)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for _ in range(8):
                x.add_(1.0)
                x.mul_(0.5)
        for _ in range(20):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s)
        for _ in range(iters // 8):
            g.replay()
        e1.record(s)
        e1.synchronize()
    return e0.elapsed_time(e1) * 1000.0 / (iters // 8 * 8)


def config_summary(name, K, local_rank, with_oracle):
    """One short run of another configuration for the default line's "configs" key."""
    w = make_workload(name)
    ctx, r = run_timed(w, K, 20 if w.model == 3 else 50, 1, local_rank, lambda: __import__("torch").cuda.synchronize())
    ctx.close()
    rf = r["roofline"]
    out = {"value": replicas_throughput(1, K, r["ms"]), "unit": "iters/s", "steps": K, "ms_per_step": r["ms"] / K,
           "gpu_launches": r["launches"], "upload_fraction": r["u"], "clocks": r["clocks"],
           "roofline": {k: rf[k] for k in ("bound", "kernel", "achieved", "peak", "unit", "frac")},
           "stages": [{k: s[k] for k in ("stage", "kernel", "ms", "GB/s", "frac")} for s in rf["stages"]],
           "whole_path_frac": rf["whole_path"]["frac"]}
    base = name.split("_")[0]
    if name == "c0":
        try:
            out["launch_floor"] = {"us_per_iteration": two_kernel_graph_floor_us(),
                                   "what": "graph replay of two dependent, almost empty kernels per iteration (eight "
                                           "iterations per graph, as laq_step replays them): the floor of a two-kernel "
                                           "iteration that is bound by launches and kernel boundaries"}
        except Exception as e:
            out["launch_floor"] = {"error": repr(e)[:200]}
    if with_oracle and base in ORACLE_ITERS and name == base:
        n = ORACLE_ITERS[base]
        first, cpu = first_disagreement(w, n)
        out["first_disagreement"] = {"iteration": first, "within": n,
                                     "rule": "first iteration at which a skip bit differs from the free-running fp64 "
                                             "oracle's, or theta / the loss leaves its %g band; null = none within "
                                             "the iterations compared" % TRAJ_RTOL}
        out["cpu_baseline"] = cpu
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="c4_b8")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="leave out the short runs of the other configurations")
    ap.add_argument("--sustained-steps", type=int, default=400,
                    help="headline workload only: iterations to settle under the power cap before the sustained figure (0 = off)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w = make_workload(args.workload)
    sharded_run = "sharded" in args.workload.split("_")

    if args.impl == "reference":
        run_reference(args, w, args.workload, rank)
        return

    extras = world == 1 and args.workload == "c4_b8"       # the default line carries the whole picture
    cpu_all = None
    if extras and not args.no_cpu_baseline:
        # the pool is started (spawn) and done before the first GPU call of this process
        try:
            cpu_all = cpu_all_cores(w)
        except Exception as e:                      # the all-core leg must not take the GPU legs down with it
            cpu_all = {"value": None, "unit": "iters/s (steps 1-3 only)", "kind": "oracle", "error": repr(e)[:200]}

    import torch
    import torch.distributed as dist
    from paper_1909_07588_b200 import build, laq
    if not os.path.exists(laq.LIB_PATH):
        build.build()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    K, Wm = args.steps, args.warmup
    if sharded_run:
        run_sharded(args, w, K, Wm, world, rank, local_rank, barrier)
        if world > 1:
            dist.destroy_process_group()
        return
    ctx, r = run_timed(w, K, Wm, world, local_rank, barrier)
    sustained = run_sustained(ctx, w, args.sustained_steps, local_rank) if extras and args.sustained_steps > 0 else None
    cfg = workload_config(w, args.workload, world, ctx)
    ctx.close()
    del ctx
    torch.cuda.empty_cache()
    e2e = run_e2e(w, K, world, barrier)

    line = {"metric": METRIC, "value": replicas_throughput(world, K, r["ms"]), "unit": "iters/s", "n_gpus": world,
            "steps": K, "warmup": Wm, "ms_per_step": r["ms"] / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg, "clocks": r["clocks"], "e2e": e2e,
            "gpu_launches": r["launches"], "roofline": r["roofline"]}
    if sustained is not None:
        line["sustained"] = sustained
    if extras and not args.no_configs:
        configs = {}
        for name, Kc in CONFIG_RUNS:
            torch.cuda.empty_cache()
            try:
                configs[name] = config_summary(name, Kc, local_rank, with_oracle=not args.no_cpu_baseline)
            except Exception as e:
                configs[name] = {"error": repr(e)[:300]}
        line["configs"] = configs
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, args.workload)
        if cpu_all is not None:
            line["cpu_baseline"]["all_cores"] = cpu_all
    elif rank == 0:
        line["cpu_baseline"] = None
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the LAQ hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one LAQ iteration (Algorithm 2: local gradients, quantizer, norms, skip rule, lazy aggregate and
theta step) over all M workers of the workload.  Prints one JSON line (rank 0).  Workloads:
c4_b8 (default: M = 64, p = 25.6 M, b = 8, gradients generated in the kernels), c4_b4, c4_b2,
c4_b8_xi0 (every worker uploads), c4_b8_frozen (no drift: uploads die out), c4_b8_M8 (8 workers: a small case
for profiler captures), c0, c1, c2, c3 (model workloads).
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


MODE_FLAGS = {"lag": 1, "qgd": 2, "gd": 3}          # quantizer off, trigger off, both (LAQ_FLAG_*)


def make_workload(name):
    """c4_b8 (default), c4_b{2,3,4}, c4_b8_M8, c0..c3; suffixes _lag, _qgd, _gd select the baseline modes and
    _batchN minibatch gradients (model workloads), e.g. c1_b3_batch500."""
    w = _base_workload(name)
    w.flags, w.batch = 0, 0
    for part in name.split("_")[1:]:
        if part in MODE_FLAGS:
            w.flags = MODE_FLAGS[part]
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
    return {"c0": W.c0, "c1": W.c1, "c2": W.c2, "c3": W.c3}[name.split("_")[0]]()


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
    g_bytes = 0.0 if w.model == 3 else 4.0          # g read from HBM unless generated in the kernel
    batch = getattr(w, "batch", 0)
    rows = [min(n, batch) if batch else n for n in w.N]
    X_bytes = sum(n * w.n_features * 4.0 + n * 4.0 for n in rows) if w.X else 0.0
    if getattr(w, "flags", 0) & 1:                  # quantizer off: one sweep for radius and norm, raw innovations
        return {
            "local_gradient": X_bytes + (Mp * 4.0 if w.X else 0.0),
            "radius": 0.0,
            "quantize_norms_trigger": Mp * (4.0 + g_bytes),
            "aggregate_theta_step": u * Mp * (8.0 + g_bytes) + 16.0 * w.p,
        }
    return {
        "local_gradient": X_bytes + (Mp * 4.0 if w.X else 0.0),
        "radius": Mp * (4.0 + g_bytes),
        "quantize_norms_trigger": Mp * (4.0 + g_bytes + w.b / 8.0),
        "aggregate_theta_step": u * Mp * (8.0 + w.b / 8.0) + 16.0 * w.p,
    }


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

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
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
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except Exception:
                continue
            for name, col in (("hw_slowdown", 4), ("hw_thermal_slowdown", 5), ("sw_thermal_slowdown", 6),
                              ("sw_power_cap", 7)):
                if len(r) > col and r[col].lower().startswith("active"):
                    reasons.add(name)
        busy = [v for v in sm if mx and v > 0.5 * mx] or sm
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


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
        per_coord = rec["bytes_per_worker_coordinate"]["c4_b%d" % w.b][stage]
        return None if per_coord is None or w.model != 3 else per_coord * float(w.M) * w.p
    except Exception:
        return None


def cpu_baseline(w, name, steps=None, warmup=1, budget_s=12.0):
    """The oracle as it stands, one thread, on a bounded sample of the workload.  With `steps` given (the
    reference arm) it runs that many sample iterations after `warmup`, but stops when `budget_s` is used up."""
    import oracle
    oracle.build()
    if w.model == 3:
        p_s = min(w.p, 1_600_000)
        o = oracle.OracleLaq(32, oracle.MODEL_SYNTH, w.M, p_s, alpha=w.alpha, b=w.b, D=w.D, xi=w.xi, tbar=w.tbar,
                             seed=w.seed, synth_sigma=w.synth_sigma, synth_eta0=w.synth_eta0, flags=w.flags)
        scale = p_s / float(w.p)
        what = "fp32 mirror, M=%d workers, first %d of %d coordinates" % (w.M, p_s, w.p)
    else:
        o = oracle.OracleLaq(64, w.model, w.M, w.p, N=w.N, n_features=w.n_features, n_classes=w.n_classes,
                             n_hidden=w.n_hidden, alpha=w.alpha, lam=w.lam, b=w.b, D=w.D, xi=w.xi, tbar=w.tbar,
                             bf16_ops=w.bf16_ops, theta0=w.theta0, seed=w.seed, flags=w.flags, batch=w.batch)
        for m in range(w.M):
            o.set_shard(m, w.X[m], w.y[m])
        scale = 1.0
        what = "fp64 oracle, full workload"
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
    return {"value": n / dt * scale, "unit": "iters/s", "cores": 1, "kind": "oracle",
            "sample": "%s, %d iterations after warm-up%s" % (
                what, n, "; iterations/s scaled by %g (cost is linear in p)" % scale if scale != 1.0 else "")}


def run_reference(args, w, name, rank):
    """--impl reference: the paper ships no code, so the reference arm is the CPU oracle (rank 0 only)."""
    if rank != 0:
        return
    t0 = time.time()
    base = cpu_baseline(w, name, steps=args.steps, warmup=args.warmup, budget_s=150.0)
    val = base["value"]
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "iters/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1000.0 / val, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": name, "M": w.M, "p": w.p, "b": w.b, "D": w.D, "tbar": w.tbar},
            "cpu_baseline": base,
            "e2e": {"value": val, "unit": "iters/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": time.time() - t0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="c4_b8")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w = make_workload(args.workload)

    if args.impl == "reference":
        run_reference(args, w, args.workload, rank)
        return

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
    ctx = laq.from_workload(w, trace_capacity=max(K, Wm), flags=w.flags, batch=w.batch)
    ctx.step(Wm)
    ctx.sync()
    s0 = ctx.get_state(big=False)

    # ---- timed region: K iterations, inputs resident, per-stage events on the library's stream ----------
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
        ctx.step(K)
        stage_ms, stage_n = ctx.kernel_times()
        ctx.set_profiling(False)
    clocks = sampler.stop()
    if not inline_events:
        s2 = ctx.get_state(big=False)
    ms = max_over_ranks(ms, world)
    u = (s2["uploads"] - s1["uploads"]) / float(K * w.M)       # of the iterations whose stages were timed

    # ---- end to end through the C ABI with host buffers ---------------------------------------------------
    Ke = K                                     # the same number of iterations as the device-timed region
    theta0_host = torch.zeros(w.p, dtype=torch.float32).pin_memory().numpy() if w.theta0 is None else w.theta0
    barrier()
    t0 = time.perf_counter()
    ctx2 = laq.from_workload(w, trace_capacity=1, theta0=theta0_host, flags=w.flags, batch=w.batch)     # theta0 and the shards cross PCIe here
    tr_bytes = 0
    for _ in range(Ke):
        tr = ctx2.step(1, trace=True)                                     # per-step report read back to the host
        tr_bytes = sum(v.nbytes for v in tr.values())
    theta_out = ctx2.get_state(big=False)["theta"]
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s, world)
    ctx2.close()
    shard_bytes = sum(x.nbytes + y.nbytes for x, y in zip(w.X, w.y))
    e2e = {"value": world * Ke / e2e_s, "unit": "iters/s", "steps": Ke,
           "h2d_bytes_per_step": (w.p * 4 + shard_bytes) / float(Ke),
           "d2h_bytes_per_step": tr_bytes + (theta_out.nbytes + 2 * w.p * 4) / float(Ke),
           "includes": "laq_init (theta0 H2D), laq_load_shards (H2D), laq_step(1, trace) per step, final laq_get_state"}

    # ---- roofline of the dominant kernel, per-stage table ---------------------------------------------------
    peak, peak_src = hbm_peak()
    abytes = algorithmic_bytes(w, u)
    stages = []
    iters_recorded = int(stage_n[3])          # one aggregate launch per iteration; at most 512 iterations are bracketed
    for i, name in enumerate(STAGES):
        if stage_n[i] == 0 or iters_recorded == 0:
            continue
        avg_ms = stage_ms[i] / iters_recorded  # per iteration (the gradient stage may be several launches)
        gbs = abytes[name] / (avg_ms * 1e-3) / 1e9 if avg_ms > 0 else 0.0
        if (w.flags & 1) and name == "radius":
            continue                            # quantizer off: radius and norm share one sweep (the next slot)
        kern = STAGE_KERNELS[name]
        if w.flags & 1:
            kern = {"quantize_kernel": "innovation_kernel", "aggregate_kernel": "aggregate_raw_kernel"}.get(kern, kern)
        stages.append({"stage": name, "kernel": kern, "ms": avg_ms, "bytes": abytes[name],
                       "GB/s": gbs, "frac": gbs / peak, "share": stage_ms[i] / max(stage_ms.sum(), 1e-12)})
    if w.model != 3 and w.M * ((w.p + 15) // 16 * 16) <= 8192:
        # small problems run steps 2-5 in one single-block kernel: its time sits in the last slot, the radius and
        # quantize slots are empty; it moves the bytes of all three sweeps
        last = stages[-1]
        last.update({"stage": "steps_2_to_5_single_block", "kernel": "small_iteration_kernel",
                     "bytes": abytes["radius"] + abytes["quantize_norms_trigger"] + abytes["aggregate_theta_step"]})
        last["GB/s"] = last["bytes"] / (last["ms"] * 1e-3) / 1e9 if last["ms"] > 0 else 0.0
        last["frac"] = last["GB/s"] / peak
        stages = [st for st in stages if st["stage"] not in ("radius", "quantize_norms_trigger")]
    dom = max(stages, key=lambda s: s["ms"])
    path_bytes = sum(s["bytes"] for s in stages)
    path_ms = sum(s["ms"] for s in stages)
    roofline = {"bound": "hbm", "kernel": dom["kernel"], "achieved": dom["GB/s"], "peak": peak, "unit": "GB/s",
                "frac": dom["frac"], "traffic": traffic_for(dom["stage"], w), "peak_source": peak_src,
                "bytes_per_launch": dom["bytes"], "ms_per_launch": dom["ms"], "upload_fraction": u,
                "stage_timing": ("CUDA events around every stage inside the timed region" if inline_events else
                                 "CUDA events around every stage over the %d iterations that follow the timed region" % K),
                "stages": stages,
                "whole_path": {"bytes_per_iter": path_bytes, "GB/s": path_bytes / (path_ms * 1e-3) / 1e9,
                               "frac": path_bytes / (path_ms * 1e-3) / 1e9 / peak}}

    if w.model == 2:
        # the network's gradient stage is two dense bf16 products (X W1^T and dH^T X): a tensor-core roofline
        g_stage = [st for st in stages if st["stage"] == "local_gradient"][0]
        flops = 4.0 * sum(w.N) * w.n_features * w.n_hidden
        tpeak, tsrc = tensor_peak()
        tf = flops / (g_stage["ms"] * 1e-3) / 1e12
        roofline.update({"bound": "tensor", "kernel": "umma_hidden_fused_kernel + umma_dw1_kernel (whole gradient stage)",
                         "achieved": tf, "peak": tpeak, "unit": "TFLOP/s", "frac": tf / tpeak, "traffic": None,
                         "peak_source": tsrc, "flops_per_launch": flops, "ms_per_launch": g_stage["ms"]})
    line = {"metric": METRIC, "value": replicas_throughput(world, K, ms), "unit": "iters/s", "n_gpus": world, "steps": K,
            "warmup": Wm, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "name": w.name, "M": w.M, "p": w.p, "b": w.b, "D": w.D,
                       "tbar": w.tbar, "alpha": w.alpha, "flags": w.flags, "batch": w.batch,
                       "parallelism": "replicas x%d" % world,
                       "l2": "no flush: the state swept every iteration (%.1f GB) exceeds the 126 MB L2"
                             % (ctx.workspace_bytes / 1e9) if ctx.workspace_bytes > 4e8 else
                             "no flush: working set is L2 resident by design of the workload"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, args.workload)
    elif rank == 0:
        line["cpu_baseline"] = None
    ctx.close()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the Orth-Dion optimizer step on B200.

    python bench.py --gpus N --steps K --warmup W            # the CUDA library (one JSON line)
    python bench.py --impl reference --steps K --warmup W    # the float64 CPU oracle, same metric

A step is one pass of the whole hot path (buffer, power-iteration product, left QR, right
factor, right QR or ColNorm, error feedback and weight update) over every weight matrix of the
8B Llama-style model (224 matrices, r = 512) with synthetic gradients.  `value` is parameter
elements per second with everything resident in HBM; `e2e` is the same with the gradients coming
from pinned host memory and the updated weights going back, copies inside the timed region.
For N > 1 (torchrun) every rank steps its own replica of the model (--scaling weak, the default)
or its share of the model's matrices (--scaling strong, whole matrices split by cost); either way
there is no collective on the data path, and the step time is the maximum over the ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2605_16341_b200 import sharding  # noqa: E402
from paper_2605_16341_b200 import workloads as wl  # noqa: E402

DEFAULT_LANES = 4      # the library's default number of internal streams of a grouped call
METRIC = "orthdion_step_param_elements_per_s"
UNIT = "param-elements/s"


# ------------------------------------------------------------------------------------------------
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def logical_flops(spec, mode_orth=True):
    """Logical flops of one step of one matrix: four m*n*r contractions and two CholeskyQR2
    (Gram 2kr^2 and apply kr^2, twice, plus the r^3/3 Cholesky); extra passes of the bf16 split
    are not counted."""
    m, n, r = spec.m, spec.n, spec.r
    gemm = 8.0 * m * n * r
    qr_left = 6.0 * m * r * r + 2.0 * r ** 3 / 3.0
    qr_right = (6.0 * n * r * r + 2.0 * r ** 3 / 3.0) if mode_orth else 3.0 * n * r
    return gemm, qr_left + qr_right


def stage_models(matrices, mode_orth=True):
    """Algorithmic flops and HBM bytes per step for each timed stage (bf16 X/G, fp32 M)."""
    out = {}
    def add(name, flops, byts):
        f, b = out.get(name, (0.0, 0.0))
        out[name] = (f + flops, b + byts)
    for s in matrices:
        m, n, r = s.m, s.n, s.r
        gb = 2 if s.g_dtype == torch.bfloat16 else 4
        xb = 2 if s.x_dtype == torch.bfloat16 else 4
        add("k1_buffer_times_q", 2.0 * m * n * r, (4 + gb) * m * n + 4.0 * (n + m) * r)
        add("k3_buffer_t_times_p", 2.0 * m * n * r, (4 + gb) * m * n + 4.0 * (n + m) * r)
        # the fused pass: M read and written, G read, X read and written (14 B per element with
        # bf16 X and G); the operand planes of P, R, Q it also reads are reported on their own
        add("k5_feedback_update", 4.0 * m * n * r, (8 + gb + 2 * xb) * m * n)
        qrs = [m] + ([n] if mode_orth else [])
        for k in qrs:
            add("gram", 2 * 2.0 * k * r * r, 2 * 4.0 * k * r)
            add("apply_inverse", 2 * 1.0 * k * r * r, 2 * 12.0 * k * r)
            add("cholesky_inverse", 2 * 2.0 * r ** 3 / 3.0, 2 * 8.0 * r * r)
    return out


def k5_factor_plane_bytes(matrices):
    """Bytes of the operand planes of P, R, Q that the fused pass reads once from HBM (fp16 planes
    for bf16 weights, two bf16 terms otherwise); not part of its 14 B per element."""
    return sum((2.0 if s.x_dtype == torch.bfloat16 else 4.0) * (2 * s.n + s.m) * s.r for s in matrices)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        self.lines, self.proc = [], None
        try:
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            gid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
            self.cmd = ["nvidia-smi", "-i", gid, f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                        "-lms", "100"]
        except Exception:
            self.cmd = None

    def start(self):
        if not self.cmd:
            return
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if not self.proc:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        for ts, line in self.lines:
            if ts < t0 or ts > t1 + 0.2:
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            try:
                pw.append(float(f[2]))
            except ValueError:
                pass
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                    power_w=(statistics.median(pw) if pw else None))


# ------------------------------------------------------------------------------------------------
def cpu_oracle_sample(w, steps=1, warmup=0):
    """Time the float64 oracle, as it stands, on one attention-projection matrix of the workload
    (inputs from the same seeded generators).  Returns (elements/s, seconds per step, description)."""
    from oracle import orthdion_oracle as orc
    # first square matrix of the model (q projection), else the first matrix
    idx = next((i for i, s in enumerate(w.matrices) if s.m == s.n), 0)
    spec = w.matrices[idx]
    X, M, Q = wl.initial_state(spec, 0, idx)
    basis = wl.grad_basis(w, spec, 0, idx)
    Xo, Mo, Qo = X.double().numpy(), M.double().numpy(), Q.double().numpy()
    times = []
    for t in range(warmup + steps):
        G = wl.gradient(w, spec, 0, idx, t, basis).double().numpy()
        t0 = time.perf_counter()
        out = orc.step(Xo, Mo, G, Qo, eta=w.eta, mu=w.mu, wd=w.wd, mode=orc.ORTH)
        dt = time.perf_counter() - t0
        Xo, Mo, Qo = out["X"], out["M"], out["Q"]
        if t >= warmup:
            times.append(dt)
    sec = sum(times) / len(times)
    desc = (f"{len(times)} step(s) of one {spec.m}x{spec.n} matrix (r={spec.r}) of {w.name}, "
            f"float64 numpy oracle; elements/s = m*n / seconds")
    return spec.numel / sec, sec, desc


def cpu_oracle_per_class(w, mode_orth=True):
    """One oracle step of the first matrix of every distinct shape of the workload, timed on the
    host cores, and the whole-model step extrapolated from the class counts:
    seconds(model) = sum over classes of (matrices in the class) x (seconds of its sample).
    Returns (elements/s, seconds, description, per-class list)."""
    from oracle import orthdion_oracle as orc
    classes = wl.shape_classes(w.matrices)
    per, total = [], 0.0
    for key, members in classes.items():
        idx = members[0]
        spec = w.matrices[idx]
        X, M, Q = wl.initial_state(spec, 0, idx)
        basis = wl.grad_basis(w, spec, 0, idx)
        G = wl.gradient(w, spec, 0, idx, 0, basis).double().numpy()
        Xo, Mo, Qo = X.double().numpy(), M.double().numpy(), Q.double().numpy()
        del X, M, Q, basis
        t0 = time.perf_counter()
        orc.step(Xo, Mo, G, Qo, eta=w.eta, mu=w.mu, wd=w.wd, mode=orc.ORTH if mode_orth else orc.COLNORM)
        dt = time.perf_counter() - t0
        del Xo, Mo, Qo, G
        per.append({"shape": f"{spec.m}x{spec.n}", "r": spec.r, "matrices": len(members), "seconds": dt})
        total += dt * len(members)
    desc = (f"extrapolated: one float64 numpy oracle step of one matrix per distinct shape of {w.name} "
            f"({', '.join(p['shape'] for p in per)}; {sum(p['seconds'] for p in per):.1f} s of CPU work), "
            f"model step = sum over shapes of count x seconds; elements/s = all elements / that")
    return w.numel / total, total, desc, per


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.workload(args.workload, layers=args.layers)
    steps = max(1, args.steps)
    val, sec, desc = cpu_oracle_sample(w, steps=steps, warmup=max(0, args.warmup))
    cores = blas_threads()
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": max(0, args.warmup), "ms_per_step": sec * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": w.name, "sample": desc},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
def run_ours(args):
    from paper_2605_16341_b200 import binding as od
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    w = wl.workload(args.workload, layers=args.layers, r=args.rank)
    if args.lanes:
        od.orthdion_set_concurrency(args.lanes)
    mode = od.MODE_ORTH if args.mode == "orth" else od.MODE_COLNORM
    seed = 1000 + rank
    all_matrices = w.matrices
    if args.scaling == "strong" and world > 1:
        mine = sharding.partition_matrices([(s.m, s.n, s.r) for s in all_matrices], world)[rank]
        w = wl.Workload(w.name, tuple(all_matrices[i] for i in mine), w.grad, w.mu, w.eta, w.wd, w.grad_params)
        seed = 1000
    hs, Xs, Ms, Qs, Gsets = [], [], [], [], [[] for _ in range(args.grad_sets)]
    plan_cache = {}
    for i, spec in enumerate(w.matrices):
        key = (spec.m, spec.n, spec.r, spec.x_dtype, spec.g_dtype)
        if key not in plan_cache:
            h = od.orthdion_create(spec.m, spec.n, spec.r, w.mu, w.eta, w.wd, mode)
            od.orthdion_set_dtypes(h, spec.x_dtype, spec.g_dtype)
            if args.engine == "simt":
                od.orthdion_set_engine(h, od.ENGINE_SIMT)
            if args.passes:
                for which, pv in enumerate(int(x) for x in args.passes.split(",")):
                    od.orthdion_set_passes(h, which, pv)
            if args.diagnostics:
                od.orthdion_set_diagnostics(h, args.diagnostics)
            plan_cache[key] = h
        hs.append(plan_cache[key])
        X, M, Q = wl.initial_state(spec, seed, i, device=dev)
        basis = wl.grad_basis(w, spec, seed, i, device=dev)
        Xs.append(X); Ms.append(M); Qs.append(Q)
        for k in range(args.grad_sets):
            Gsets[k].append(wl.gradient(w, spec, seed, i, k, basis, device=dev))
        del basis
    ws = od.alloc_workspace(od.orthdion_workspace_bytes_grouped(hs), device=dev)
    tables = [od.PointerTable(hs, Xs, Ms, Gsets[k], Qs) for k in range(args.grad_sets)]
    stream = torch.cuda.current_stream()

    graphs = None

    def step(k):
        if graphs is not None:
            graphs[k % args.grad_sets].replay()
        else:
            od.orthdion_step_grouped(tables[k % args.grad_sets], ws, stream)

    def barrier():
        if dist is not None:
            dist.barrier()

    for k in range(args.warmup):
        step(k)
    torch.cuda.synchronize()
    launches_per_step = 0
    if args.warmup > 0:
        launches_per_step = od.orthdion_launch_count() // args.warmup
    if args.graph:
        # one CUDA graph per gradient set: a step is then a single graph launch (pays on workloads
        # whose step is bound by kernel launches; the stage profile is taken without graphs)
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(stream)
        captured = []
        for k in range(args.grad_sets):
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=side):
                od.orthdion_step_grouped(tables[k], ws, torch.cuda.current_stream())
            captured.append(gr)
        stream.wait_stream(side)
        torch.cuda.synchronize()
        graphs = captured
        for k in range(2):
            step(k)
        torch.cuda.synchronize()

    sampler = ClockSampler(dev) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(); torch.cuda.synchronize()
    l0 = od.orthdion_launch_count()
    t_wall0 = time.time()
    ev0.record(stream)
    for k in range(args.steps):
        step(args.warmup + k)
    ev1.record(stream)
    torch.cuda.synchronize(); barrier()
    t_wall1 = time.time()
    launches = od.orthdion_launch_count() - l0
    if args.graph:
        launches = launches_per_step * args.steps      # replayed from the captured graphs, not re-enqueued
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    ms_total = sharding.max_over_ranks(ev0.elapsed_time(ev1), dist, dev)

    # Per-stage times: a second timed region of the same K steps with every launch bracketed by
    # CUDA events on its stream.  It runs on ONE stream (lanes = 1): event pairs taken on the
    # overlapping internal streams of the default configuration would not add up to the step.
    profile_on = not args.no_profile
    stage_ms, ms_step_one_stream = {}, None
    graphs = None
    if profile_on:
        od.orthdion_set_concurrency(1)
        step(args.warmup + args.steps)                       # settle into the one-stream order
        torch.cuda.synchronize()
        od.orthdion_profile_begin(max(1024, (launches_per_step + 16) * args.steps))
        pv0, pv1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pv0.record(stream)
        for k in range(args.steps):
            step(args.warmup + args.steps + 1 + k)
        pv1.record(stream)
        torch.cuda.synchronize()
        stage_ms = od.orthdion_profile_end()
        ms_step_one_stream = pv0.elapsed_time(pv1) / args.steps
        od.orthdion_set_concurrency(args.lanes or DEFAULT_LANES)
    ms_step = ms_total / args.steps
    flags = od.orthdion_last_status(hs, ws, stream)
    failed = sum(1 for f in flags if f & (od.STATUS_RANK_DEFICIENT | od.STATUS_NONFINITE | od.STATUS_WAIT_LIMIT))
    shifted = sum(1 for f in flags if f & (od.STATUS_SHIFTED_LEFT | od.STATUS_SHIFTED_RIGHT))
    diag_summary = None
    if args.diagnostics:
        ds = [d for d in od.orthdion_last_diagnostics(hs, ws, stream) if d["nu"] == d["nu"]]
        if ds:
            diag_summary = {"nu_min": min(d["nu"] for d in ds), "nu_max": max(d["nu"] for d in ds),
                            "erank_mean": sum(d["erank"] for d in ds) / len(ds),
                            "eig_products_max": max(d["iterations"] for d in ds),
                            "eig_products_mean": sum(d["iterations"] for d in ds) / len(ds)}

    # elements stepped by the whole job: N replicas (weak) or the one model split N ways (strong)
    elements = w.numel * world if args.scaling == "weak" else sum(s.numel for s in all_matrices)
    value = elements / (ms_step * 1e-3)

    # ---- end to end: gradients from pinned host memory, updated weights back to the host ----
    e2e = None
    if not args.no_e2e:
        try:
            e2e = run_e2e(args, od, w, dev, stream, tables, ws, Xs, Gsets, world, dist)
        except Exception as exc:  # allocation of pinned memory can fail on small hosts
            e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                   "error": repr(exc)[:200]}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    orth = mode == od.MODE_ORTH
    gemm_f = sum(logical_flops(s, orth)[0] for s in w.matrices)
    qr_f = sum(logical_flops(s, orth)[1] for s in w.matrices)
    bytes20 = sum((2 * (4 + (2 if s.g_dtype == torch.bfloat16 else 4)) + 4 +
                   2 * (2 if s.x_dtype == torch.bfloat16 else 4)) * s.numel for s in w.matrices)
    t_hbm = bytes20 / (peaks["hbm_gbs"] * 1e9) * 1e3
    t_tensor = (gemm_f + qr_f) / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3
    t_roof = max(t_hbm, t_tensor)

    models = stage_models(w.matrices, orth)
    stages = {}
    dominant, dom_ms = None, 0.0
    for name, (ms, cnt) in stage_ms.items():
        if cnt == 0:
            continue
        per_step = ms / args.steps
        entry = {"ms_per_step": per_step, "launches_per_step": cnt / args.steps}
        if name in models:
            f, b = models[name]
            entry["tflops"] = f / (per_step * 1e-3) / 1e12
            entry["gbs"] = b / (per_step * 1e-3) / 1e9
        stages[name] = entry
        if name in models and per_step > dom_ms:
            dominant, dom_ms = name, per_step
    roofline = None
    if dominant:
        f, b = models[dominant]
        t_f = f / (peaks["bf16_tflops_sustained"] * 1e12)
        t_b = b / (peaks["hbm_gbs"] * 1e9)
        if t_f >= t_b:
            ach = f / (dom_ms * 1e-3) / 1e12
            roofline = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"],
                        "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops_sustained"]}
        else:
            ach = b / (dom_ms * 1e-3) / 1e9
            roofline = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": ach / peaks["hbm_gbs"]}
        bpe = MEASURED_DRAM_BYTES_PER_ELEMENT.get((args.workload, dominant))
        roofline.update({"kernel": dominant, "launches_per_step": stages[dominant]["launches_per_step"],
                         "per": "step (sum over the launches of this kernel in one step)",
                         "algorithmic": (b if roofline["bound"] == "hbm" else f),
                         "algorithmic_per_element": ((b / w.numel) if roofline["bound"] == "hbm" else None),
                         "factor_plane_bytes": (k5_factor_plane_bytes(w.matrices)
                                                if dominant == "k5_feedback_update" else None),
                         "traffic": (bpe * w.numel if (bpe and args.mode == "orth" and not args.passes) else None),
                         "peak_source": peaks["source"] + (" (sustained bf16 figure: kernel timed inside a long step)"
                                                           if roofline["bound"] == "tensor" else "")})

    cpu = None
    if not args.no_cpu_baseline:
        val, sec, desc, per = cpu_oracle_per_class(w, orth)
        cpu = {"value": val, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc,
               "seconds_per_model_step_extrapolated": sec, "per_shape": per}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": args.scaling,
        "vs_baseline": None, "dtype": "bf16-split products, f32 accumulate and state",
        "data": "synthetic",
        "config": {"workload": f"{w.name}: {len(w.matrices)} matrices per rank, {elements / 1e6:.1f}M elements in the job, r={w.matrices[0].r}, "
                               f"bf16 X/G, fp32 M, mode {args.mode}",
                   "engine": args.engine, "l2": "inputs (tens of GB per step) far exceed the 126 MB L2",
                   "grad_sets": args.grad_sets, "replicas": world, "diagnostics": args.diagnostics,
                   "lanes": args.lanes or DEFAULT_LANES, "cuda_graph": bool(args.graph),
                   "diagnostics_summary": diag_summary,
                   "matrices_failed": failed, "matrices_shifted_qr": shifted},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "roofline": roofline,
        "step_roofline": {"t_hbm_ms": t_hbm, "t_tensor_ms": t_tensor, "t_roof_ms": t_roof,
                          "frac": t_roof / ms_step, "bytes_per_element": 20,
                          "logical_tflop": (gemm_f + qr_f) / 1e12,
                          "peaks": peaks},
        "stages": stages,
        "stages_region": ("second timed region of the same steps on one stream (lanes = 1), every launch between "
                          "two CUDA events on its stream" if stage_ms else None),
        "ms_per_step_one_stream": ms_step_one_stream,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# DRAM bytes per parameter element of a stage, measured with ncu (dram__bytes_read.sum +
# dram__bytes_write.sum of one launch) on a 4-layer case of the same kernel: 6.782 GB over
# 469.8 M elements.  Traffic grows in proportion to the elements, so a step's traffic is this
# figure x its elements.  Set to None whenever the kernel changes until the counters are retaken.
MEASURED_DRAM_BYTES_PER_ELEMENT = {("cfg4", "k5_feedback_update"): 14.44}


def run_e2e(args, od, w, dev, stream, tables, ws, Xs, Gsets, world, dist):
    """Same step, end to end: every step copies all gradients host->device from pinned memory and
    all updated weights device->host, inside the timed region.  The model is stepped in chunks of
    consecutive matrices (one orthdion_step_grouped call per chunk) so that the copies of one chunk
    overlap the kernels of another: an input stream, the compute stream and an output stream,
    ordered by events (a chunk's gradients are not overwritten before its step has read them, its
    weights not stepped again before they have been copied out)."""
    steps = max(1, min(args.steps, args.e2e_steps))
    g_host = [torch.empty(g.shape, dtype=g.dtype, pin_memory=True) for g in Gsets[0]]
    x_host = [torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for x in Xs]
    for gh, gd in zip(g_host, Gsets[0]):
        gh.copy_(gd)
    torch.cuda.synchronize()
    h2d = sum(g.numel() * g.element_size() for g in g_host)
    d2h = sum(x.numel() * x.element_size() for x in x_host)

    # chunks of consecutive matrices with about equal element counts
    n_mat = len(Xs)
    n_chunks = max(1, min(args.e2e_chunks, n_mat))
    total = sum(x.numel() for x in Xs)
    bounds, acc, nxt = [0], 0, 1
    for i, x in enumerate(Xs):
        acc += x.numel()
        if nxt < n_chunks and acc >= total * nxt / n_chunks and i + 1 < n_mat:
            bounds.append(i + 1)
            nxt += 1
    bounds.append(n_mat)
    chunks = [range(bounds[k], bounds[k + 1]) for k in range(len(bounds) - 1) if bounds[k + 1] > bounds[k]]
    t0 = tables[0]
    hs_all = [t0.hs[i] for i in range(n_mat)]
    Ms, Qs = t0._keep[1], t0._keep[3]
    sub = [od.PointerTable([hs_all[i] for i in ch], [Xs[i] for i in ch], [Ms[i] for i in ch],
                           [Gsets[0][i] for i in ch], [Qs[i] for i in ch]) for ch in chunks]
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    in_done = [torch.cuda.Event() for _ in chunks]
    comp_done = [torch.cuda.Event() for _ in chunks]
    out_done = [torch.cuda.Event() for _ in chunks]
    first = [True]

    def one():
        for c, ch in enumerate(chunks):
            with torch.cuda.stream(s_in):
                if not first[0]:
                    s_in.wait_event(comp_done[c])          # the previous step has read this chunk's G
                for i in ch:
                    Gsets[0][i].copy_(g_host[i], non_blocking=True)
                in_done[c].record(s_in)
            stream.wait_event(in_done[c])
            if not first[0]:
                stream.wait_event(out_done[c])             # the previous X of this chunk has left
            od.orthdion_step_grouped(sub[c], ws, stream)
            comp_done[c].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(comp_done[c])
                for i in ch:
                    x_host[i].copy_(Xs[i], non_blocking=True)
                out_done[c].record(s_out)
        first[0] = False

    def join():
        stream.wait_stream(s_in)
        stream.wait_stream(s_out)

    one()
    join()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    ev0.record(stream)
    s_in.wait_event(ev0)
    s_out.wait_event(ev0)
    for _ in range(steps):
        one()
    join()
    ev1.record(stream)
    torch.cuda.synchronize()
    ms = sharding.max_over_ranks(ev0.elapsed_time(ev1), dist, dev)
    ms_step = ms / steps
    job_elements = float(w.numel * world)
    if args.scaling == "strong" and dist is not None:
        t = torch.tensor([float(w.numel)], device=dev, dtype=torch.float64)
        dist.all_reduce(t)
        job_elements = float(t.item())
    return {"value": job_elements / (ms_step * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms_step, "steps": steps,
            "pipeline": f"{len(chunks)} chunks of consecutive matrices, copies on their own streams"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--layers", type=int, default=None, help="truncate the grouped models (experiments)")
    ap.add_argument("--rank", type=int, default=None, help="override r (cfg2 sweep)")
    ap.add_argument("--mode", default="orth", choices=["orth", "colnorm"])
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="N > 1: one model replica per rank (weak) or the model's matrices split over ranks (strong)")
    ap.add_argument("--engine", default="tensor", choices=["tensor", "simt"])
    ap.add_argument("--passes", default=None,
                    help="bf16 split passes of the four product groups, e.g. 3,3,3,1 (0 keeps the default)")
    ap.add_argument("--diagnostics", type=int, default=0, choices=[0, 1, 3],
                    help="on-device diagnostics inside the timed step (0 off, 1 factor diagnostics, 3 plus buffer norms)")
    ap.add_argument("--lanes", type=int, default=None,
                    help="internal streams a grouped call spreads its launch batches over (library default if unset)")
    ap.add_argument("--graph", action="store_true",
                    help="replay the step from a CUDA graph captured after the warm-up (one per gradient set)")
    ap.add_argument("--grad-sets", type=int, default=2)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--e2e-chunks", type=int, default=8,
                    help="grouped calls per end-to-end step (copies of one chunk overlap the kernels of another)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-profile", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    else:
        run_ours(args)


def spawn_ranks(n):
    """`python bench.py --gpus N` without a launcher: start N ranks of this same command line under
    torch.distributed.run on this node (one process per GPU, rendezvous on 127.0.0.1) and pass
    their output through.  NCCL's own initialisation lines go to stderr."""
    import socket
    have = torch.cuda.device_count()
    if have < n:
        print(f"bench.py: --gpus {n} asked for, {have} CUDA device(s) visible", file=sys.stderr)
        return 2
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd, env=env)


if __name__ == "__main__":
    main()

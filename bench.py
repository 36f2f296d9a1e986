#!/usr/bin/env python
"""Benchmark of the clustering hot path (reshape -> init -> Lloyd iterations -> finalize -> decode).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]
    python bench.py --kernel assign|update|decode|reshape|fit|linear --N .. --g .. --K .. [--reps R]

One "step" is one pass of the whole path over the synthetic weight matrices of the workload
(default: the 8192x28672, g=4, K=65536, 10-iteration configuration, the largest one).  Rank 0 prints
one JSON line; it also carries, under "workloads", a short run of every other configuration.
With N > 1 every rank clusters its own matrices (different seeds) and no data crosses ranks: the
paper's "clustering of different matrices is independent".

`--kernel` runs one entry point a few times on a synthetic case of the given size and prints the
mean device time per kernel class (the small cases the ncu summaries under profiles/ were taken on).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_13089_b200 import workloads as wl  # noqa: E402

DEFAULT_WORKLOAD = "cfg4_8192x28672_g4_k65536"
NOMINAL_SM, NOMINAL_LANES, NOMINAL_MHZ = 148, 128, 1965.0   # B200: SMs, FP32 lanes per SM, max SM clock
E_STEP_CLASSES = ("assign_main", "assign_prep", "assign_finish", "resolve", "objective")
M_STEP_CLASSES = ("update_accum", "update_delta", "update_finish")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while a timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()          # the exact process started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2])); pw.append(float(r[3]))
            except ValueError:
                continue
            for n, v in zip(names, r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        # "under load": samples drawing more than half of the largest power seen
        load = [s for s, p in zip(sm, pw) if pw and p >= 0.5 * max(pw)]
        return {"sm_mhz": statistics.median(load or sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def contraction_columns(g: int) -> int:
    """Length of the FP16 contraction the tensor-core scan runs for sub-vector dimension g (the
    library's choice of operand pieces: see TcCfg in csrc/cc_assign_tensor.cu)."""
    kd34, kd24, kd22 = ((3 * g + 4 + 15) // 16 * 16, (2 * g + 4 + 15) // 16 * 16, (2 * g + 2 + 15) // 16 * 16)
    return kd34 if (kd34 <= 48 and kd34 <= min(kd24, kd22)) else min(kd24, kd22)


def algorithmic_counts(N: int, g: int, K: int):
    return {
        "N": N,
        "dist_evals_per_assign": N * K,
        "flops_per_assign": 2 * g * N * K,
        "bytes_update": N * (2 * g + 2) + K * (4 * g + 4),
        "bytes_update_delta_min": N * 4,
        "bytes_decode": N * (2 + 2 * g),
        "bytes_reshape": N * 4 * g,
    }


def alu_ceiling(min_rate, sm_count):
    """Scores per second the ALU pipes can compare: every score of the N x K scan goes through one
    FP32 minimum; a two-input min.f32 retires one new score per lane-instruction, a three-input one
    two.  The measured lane-instruction rates per clock per SM give the per-SM ceiling; it is
    quoted at the GPU's maximum SM clock."""
    per_clk = max(min_rate["min2"], 2.0 * min_rate["min3"], min_rate["mixed"] * 1.5)
    return per_clk, per_clk * sm_count * NOMINAL_MHZ * 1e6


# ----------------------------------------------------------------------------------------------
# reference arm: the CPU oracle

def run_reference(args, w: wl.Workload):
    """The CPU oracle as it stands, timed on the host cores: each step is one Lloyd iteration
    (E-step + M-step) over a bounded sample of the workload's first matrix from its seeded start."""
    import oracle
    spec = w.matrices[0]
    cores = len(os.sched_getaffinity(0))
    W = wl.make_matrix(spec)
    X = oracle.reshape_subvectors(W, w.g)
    N = len(X)
    budget_evals = 2.0e10          # keeps one step near a few seconds of CPU work
    frac = min(1.0, budget_evals / (N * w.K))
    sel = None if frac >= 1.0 else wl.subset_positions(N, frac, 99)
    C = oracle.init_codebook(X, w.K, spec.init_seed)
    n_pts = N if sel is None else len(sel)
    times = []
    for s in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        idx, d1, _ = oracle.assign(X, C, sel)
        if sel is None:
            C, _ = oracle.update(X, idx, C)
        else:
            C, _ = oracle.update(X[sel], idx, C)
        dt = time.perf_counter() - t0
        if s >= args.warmup:
            times.append(dt)
    t = sum(times) / len(times)
    value = n_pts * w.K / t
    sample = ("one Lloyd iteration per step on %s of the %d sub-vectors against all %d centroids"
              % ("all" if sel is None else "a seeded %.5f share" % frac, N, w.K))
    line = {
        "impl": "reference", "metric": "distance_evals_per_s", "value": value, "unit": "distance evaluations/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "g": w.g, "K": w.K, "N": N, "iters_per_step": 1, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "distance evaluations/s", "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "distance evaluations/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# our arm

class Runner:
    """Holds the device buffers of one workload on one rank and runs / times / profiles its step."""

    def __init__(self, cc, torch, ctx, w, specs, layout):
        self.cc, self.torch, self.ctx, self.w, self.specs, self.layout = cc, torch, ctx, w, specs, layout
        g, K, iters = w.g, w.K, w.iters
        self.mats = []
        for spec in specs:
            Wn = wl.make_matrix(spec)
            Wh = torch.from_numpy(Wn.view(np.int16)).view(torch.float16).pin_memory()
            self.mats.append((spec, Wn, Wh))
        self.Ns = [w.n_subvectors(s) for s in specs]
        ctx.ensure_workspace(max(self.Ns), g, K)
        self.stream = torch.cuda.current_stream()
        self.bufs = {}
        for (spec, Wn, Wh), N in zip(self.mats, self.Ns):
            self.bufs[spec.name] = dict(
                W=Wh.cuda(), X=torch.empty((N, g), dtype=torch.float16, device="cuda"),
                C=torch.empty((K, g), dtype=torch.float32, device="cuda"),
                C16=torch.empty((K, g), dtype=torch.float16, device="cuda"),
                idx=torch.empty(N, dtype=torch.uint16, device="cuda"),
                dist=torch.empty(N, dtype=torch.float32, device="cuda"),
                counts=torch.empty(K, dtype=torch.int32, device="cuda"),
                trace=torch.empty(iters + 1, dtype=torch.float64, device="cuda"),
                What=torch.empty((spec.d_out, spec.d_in), dtype=torch.float16, device="cuda"))

    def step(self, on_phase=None):
        cc, ctx, w = self.cc, self.ctx, self.w
        g, K, iters = w.g, w.K, w.iters
        for (spec, Wn, Wh), N in zip(self.mats, self.Ns):
            b = self.bufs[spec.name]
            cc.cc_reshape_subvectors(ctx, b["W"], spec.d_out, spec.d_in, g, self.layout, b["X"])
            cc.cc_init_codebook(ctx, b["X"], N, g, K, spec.init_seed, b["C"])
            if on_phase:
                on_phase("setup")
            cc.cc_fit(ctx, b["X"], N, g, K, iters, b["C"], b["idx"], b["dist"], b["counts"], b["trace"])
            if on_phase:
                on_phase("fit")
            cc.cc_finalize(ctx, b["X"], N, g, b["C"], K, b["C16"], b["idx"], b["dist"], b["trace"][iters:])
            if on_phase:
                on_phase("finalize")
            cc.cc_decode(ctx, b["C16"], K, g, b["idx"], spec.d_out, spec.d_in, self.layout, b["What"])
            if on_phase:
                on_phase("decode")

    def timed(self, steps, flush, barrier):
        """`steps` steps, one CUDA-event pair each on the launching stream, the per-launch event
        pairs of the library switched off; L2 flushed before every step, outside its event pair."""
        torch = self.torch
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        launches0 = self.cc.cc_launch_count(self.ctx)
        barrier()
        for a, b in ev:
            flush.zero_()
            a.record(self.stream)
            self.step()
            b.record(self.stream)
        barrier()
        return [a.elapsed_time(b) for a, b in ev], self.cc.cc_launch_count(self.ctx) - launches0

    def profiled(self, steps, flush):
        """`steps` more steps with an event pair around every kernel launch; the record is read after
        each phase so that the Lloyd loop, the final E-step and the layout kernels are kept apart."""
        cc, ctx = self.cc, self.ctx
        phases = {}

        def on_phase(name):
            prof = cc.cc_profile_read(ctx)          # waits for the events recorded so far
            acc = phases.setdefault(name, {})
            for k, (ms, n) in prof.items():
                a = acc.setdefault(k, [0.0, 0])
                a[0] += ms
                a[1] += n

        cc.cc_profile_enable(ctx, True)
        cc.cc_profile_read(ctx)
        for _ in range(steps):
            flush.zero_()
            self.step(on_phase)
        cc.cc_profile_enable(ctx, False)
        return phases

    def near_ties(self):
        """Points the exact stage decides in one E-step against the fitted codebook (untimed call)."""
        torch, cc, w = self.torch, self.cc, self.w
        nres = torch.zeros(1, dtype=torch.int64, device="cuda")
        b0 = self.bufs[self.specs[0].name]
        cc.cc_assign(self.ctx, b0["X"], self.Ns[0], w.g, b0["C"], w.K, b0["idx"], b0["dist"], None, nres)
        return int(nres.item())

    def free_device(self):
        self.bufs = None
        self.torch.cuda.empty_cache()

    def e2e(self, steps, warm, flush, barrier):
        """The same step through cc_compress_host: pinned host buffers in and out every step (W up;
        FP16 codebook, codes, objective trace and the decoded matrix down)."""
        torch, cc, w = self.torch, self.cc, self.w
        g, K, iters = w.g, w.K, w.iters
        outs, h2d, d2h = [], 0, 0
        for (spec, Wn, Wh), N in zip(self.mats, self.Ns):
            outs.append((torch.empty((K, g), dtype=torch.float16).pin_memory(),
                         torch.empty(N, dtype=torch.uint16).pin_memory(),
                         torch.empty(iters + 1, dtype=torch.float64).pin_memory(),
                         torch.empty((spec.d_out, spec.d_in), dtype=torch.float16).pin_memory()))
            h2d += Wh.numel() * 2
            d2h += K * g * 2 + N * 2 + (iters + 1) * 8 + Wh.numel() * 2
        ms = []
        for s in range(warm + steps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            flush.zero_()
            barrier()
            a.record(self.stream)
            for (spec, Wn, Wh), (C16h, idxh, trh, Whath) in zip(self.mats, outs):
                cc.cc_compress_host(self.ctx, Wh, spec.d_out, spec.d_in, g, K, iters, spec.init_seed, self.layout,
                                    C16h, idxh, trh, Whath)
            b.record(self.stream)
            barrier()
            if s >= warm:
                ms.append(a.elapsed_time(b))
        return ms, h2d, d2h


def summarise(w, Ns, phases, prof_steps, peaks, ceiling_scores, path):
    """Per-kernel-class figures of one workload from the profiled steps."""
    g, K, iters = w.g, w.K, w.iters
    n_mat = len(Ns)
    fit = phases.get("fit", {})
    fin = phases.get("finalize", {})

    def ms_n(d, k):
        v = d.get(k, [0.0, 0])
        return v[0], v[1]

    evals_per_estep = sum(N * K for N in Ns) / n_mat               # mean over the matrices
    flops_per_estep = 2 * g * evals_per_estep
    scan_ms, scan_n = ms_n(fit, "assign_main")
    # a launch of the scan = one E-step of one matrix (the ragged rest rides in the same event pair)
    scan_avg = scan_ms / max(scan_n, 1)
    estep_ms = sum(ms_n(fit, k)[0] for k in E_STEP_CLASSES) / max(scan_n, 1)
    mstep_ms = sum(ms_n(fit, k)[0] for k in M_STEP_CLASSES) / max(scan_n, 1)
    fin_estep_ms = sum(ms_n(fin, k)[0] for k in E_STEP_CLASSES) / max(ms_n(fin, "assign_main")[1], 1)
    peak_tf = ceiling_scores * 2 * g / 1e12
    kd = contraction_columns(g)
    scan_tf = flops_per_estep / (scan_avg * 1e-3) / 1e12 if scan_avg > 0 else 0.0
    estep_tf = flops_per_estep / (estep_ms * 1e-3) / 1e12 if estep_ms > 0 else 0.0
    nominal_fp32 = NOMINAL_SM * NOMINAL_LANES * 2 * NOMINAL_MHZ * 1e6 / 1e12
    out = {
        "s_per_lloyd_iteration": (estep_ms + mstep_ms) * 1e-3,
        "e_step_ms": estep_ms, "m_step_ms": mstep_ms, "final_e_step_ms": fin_estep_ms,
        "scan": {"avg_launch_ms": scan_avg, "launches": scan_n, "scores_per_s": evals_per_estep / (scan_avg * 1e-3) if scan_avg else 0.0,
                 "achieved_tflops": scan_tf, "frac": scan_tf / peak_tf if peak_tf else None},
        "e_step": {"ms": estep_ms, "scores_per_s": evals_per_estep / (estep_ms * 1e-3) if estep_ms else 0.0,
                   "achieved_tflops": estep_tf, "frac": estep_tf / peak_tf if peak_tf else None,
                   "kernels": "scan + finish + staging + exact stage + objective sum, per E-step of the Lloyd loop"},
        "x_fp32_fma_peak": scan_tf / nominal_fp32,
    }
    if path != "ffma":
        out["contraction_columns"] = kd
        out["tensor_frac_algorithmic_of_measured_bf16"] = scan_tf / peaks["bf16_tflops"]
        out["tensor_frac_executed_of_measured_bf16"] = scan_tf * kd / g / peaks["bf16_tflops"]
    # HBM-bound kernels: algorithmic bytes of one launch over its mean duration
    hbm = {}
    cnt = [algorithmic_counts(N, g, K) for N in Ns]
    mean = lambda key: sum(c[key] for c in cnt) / len(cnt)   # noqa: E731
    for name, phase, cls, key in (("update_full", fit, "update_accum", "bytes_update"),
                                  ("update_delta", fit, "update_delta", "bytes_update_delta_min"),
                                  ("decode", phases.get("decode", {}), "decode", "bytes_decode"),
                                  ("reshape", phases.get("setup", {}), "reshape", "bytes_reshape")):
        ms, n = ms_n(phase, cls)
        if n:
            gbs = mean(key) / (ms / n * 1e-3) / 1e9
            hbm[name] = {"avg_launch_ms": ms / n, "launches": n, "algorithmic_GBs": gbs,
                         "frac_of_hbm": gbs / peaks["hbm_gbs"]}
    if "update_delta" in hbm:
        hbm["update_delta"]["note"] = "bytes counted: the two code arrays only (4 B per point); rows of moved points come on top"
    out["hbm_kernels"] = hbm
    total = sum(v[0] for ph in phases.values() for v in ph.values())
    shares = {}
    for ph in phases.values():
        for k, v in ph.items():
            if v[1]:
                s = shares.setdefault(k, {"ms_per_step": 0.0, "launches_per_step": 0.0})
                s["ms_per_step"] += v[0] / prof_steps
                s["launches_per_step"] += v[1] / prof_steps
    for k, s in shares.items():
        s["share"] = s["ms_per_step"] * prof_steps / max(total, 1e-9)
    out["kernel_classes"] = shares
    return out


def linear_rows(cc, torch, ctx, peaks):
    """Forward of the compressed linear layer (decode fused into the GEMM) on a 4096 x 4096 layer with the
    paper's g = 4 / 65536-entry codebook, for 1 to 4096 tokens: time per call, tensor and HBM fractions."""
    d_out = d_in = 4096
    g, K = 4, 65536
    N = d_in * d_out // g
    gen = torch.Generator(device="cuda").manual_seed(1)
    C16 = (torch.randn((K, g), device="cuda", generator=gen) * 0.02).to(torch.float16)
    idx = torch.randint(-32768, 32768, (N,), device="cuda", generator=gen, dtype=torch.int16).view(torch.uint16)   # all 65536 codes
    rows = []
    ctx.ensure_workspace(N, g, K)
    q4 = torch.empty((K * g + 1) // 2, dtype=torch.uint8, device="cuda")
    scale4 = torch.empty(1, dtype=torch.float32, device="cuda")
    cc.cc_quantize_codebook(ctx, C16, K, g, 4, q4, scale4, None)
    for M in (1, 16, 256, 4096):
        x = (torch.randn((M, d_in), device="cuda", generator=gen) * 0.5).to(torch.float16)
        y = torch.empty((M, d_out), dtype=torch.float32, device="cuda")
        ctx.ensure_workspace(N, g, K, at_least=cc.cc_linear_workspace_bytes(ctx, M, d_out, d_in))
        reps = 20

        def timed(call):
            for _ in range(3):
                call()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(torch.cuda.current_stream())
            for _ in range(reps):
                call()
            b.record(torch.cuda.current_stream())
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps

        ms = timed(lambda: cc.cc_linear_forward(ctx, x, M, C16, K, g, idx, d_out, d_in, None, y))
        # the same layer with the codebook quantised to 4 bits and held in shared memory (Section 5.3)
        ms_q4 = timed(lambda: cc.cc_linear_forward_q4(ctx, x, M, q4, scale4, K, g, idx, d_out, d_in, None, y))
        flops = 2.0 * M * d_in * d_out
        by = 2.0 * N + 2.0 * K * g + 2.0 * M * d_in + 4.0 * M * d_out          # codes, codebook, x, y
        rows.append({"M": M, "d_out": d_out, "d_in": d_in, "g": g, "K": K, "ms": ms, "ms_codebook_4bit": ms_q4,
                     "tflops": flops / (ms * 1e-3) / 1e12, "tensor_frac_of_measured_bf16": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                     "algorithmic_GBs": by / (ms * 1e-3) / 1e9, "frac_of_hbm": by / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     "bytes_fused": by, "bytes_decode_then_gemm": by + 2 * 2.0 * d_in * d_out,
                     "l2": "not flushed between the repetitions: codes (8 MB) and codebook (0.5 MB) stay in L2"})
    cc.cc_poll_status(ctx)
    return rows


def run_kernel_mode(a):
    """One entry point, a few repetitions, per-kernel-class device times (CUDA events on the stream)."""
    import torch
    from paper_2503_13089_b200 import binding as cc
    N, g, K = a.N, a.g, a.K
    ctx = cc.Context(0)
    d_out, d_in = g * 1024, N // 1024
    ctx.ensure_workspace(N, g, K, at_least=cc.cc_linear_workspace_bytes(ctx, a.M, d_out, max(d_in, 1)) if a.kernel in ("linear", "linear_q4") else 0)
    cc.cc_set_path(ctx, {"auto": 0, "ffma": 1, "tensor": 2}[a.path])
    Xn = wl.make_points(N, g, 1)
    X = torch.from_numpy(Xn.view(np.int16)).cuda().view(torch.float16)
    C = torch.empty((K, g), dtype=torch.float32, device="cuda")
    cc.cc_init_codebook(ctx, X, N, g, K, 7, C)
    idx = torch.empty(N, dtype=torch.uint16, device="cuda")
    dist = torch.empty(N, dtype=torch.float32, device="cuda")
    counts = torch.empty(K, dtype=torch.int32, device="cuda")
    obj = torch.zeros(1, dtype=torch.float64, device="cuda")
    nres = torch.zeros(1, dtype=torch.int64, device="cuda")
    C16 = torch.empty((K, g), dtype=torch.float16, device="cuda")
    if a.kernel in ("decode", "reshape", "linear", "linear_q4"):
        assert d_in * 1024 == N, "N must be a multiple of 1024 for the reshape / decode / linear cases"
    W = torch.empty((d_out, d_in), dtype=torch.float16, device="cuda")
    cc.cc_assign(ctx, X, N, g, C, K, idx, dist, obj, nres)      # warm-up; also valid codes for update / decode
    cc.cc_finalize(ctx, X, N, g, C, K, C16, idx, dist, obj)
    C2 = C.clone()
    X2 = torch.empty_like(X)
    if a.kernel in ("linear", "linear_q4"):
        q4 = torch.empty((K * g + 1) // 2, dtype=torch.uint8, device="cuda")
        scale4 = torch.empty(1, dtype=torch.float32, device="cuda")
        cc.cc_quantize_codebook(ctx, C16, K, g, 4, q4, scale4, None)
        xin = (torch.randn((a.M, d_in), device="cuda") * 0.5).to(torch.float16)
        y = torch.empty((a.M, d_out), dtype=torch.float32, device="cuda")

    def once():
        if a.kernel == "assign":
            cc.cc_assign(ctx, X, N, g, C, K, idx, dist, obj, nres)
        elif a.kernel == "update":
            cc.cc_update(ctx, X, N, g, idx, K, C2, counts)
        elif a.kernel == "decode":
            cc.cc_decode(ctx, C16, K, g, idx, d_out, d_in, cc.LAYOUT_PAPER_T, W)
        elif a.kernel == "reshape":
            cc.cc_reshape_subvectors(ctx, W, d_out, d_in, g, cc.LAYOUT_PAPER_T, X2)
        elif a.kernel == "linear":
            cc.cc_linear_forward(ctx, xin, a.M, C16, K, g, idx, d_out, d_in, None, y)
        elif a.kernel == "linear_q4":
            cc.cc_linear_forward_q4(ctx, xin, a.M, q4, scale4, K, g, idx, d_out, d_in, None, y)
        else:
            cc.cc_fit(ctx, X, N, g, K, a.iters, C, idx, dist, counts, None)

    once()                                   # untimed: the first launch of a kernel also loads it
    torch.cuda.synchronize()
    cc.cc_profile_enable(ctx, True)
    cc.cc_profile_read(ctx)
    for _ in range(a.reps):
        once()
    torch.cuda.synchronize()
    prof = cc.cc_profile_read(ctx)
    cc.cc_poll_status(ctx)
    out = {k: {"mean_ms": ms / n, "launches": n} for k, (ms, n) in prof.items() if n}
    print(json.dumps({"kernel": a.kernel, "N": N, "g": g, "K": K, "path": a.path,
                      "near_tie_points": int(nres.item()), "timing": out}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(wl.WORKLOADS))
    ap.add_argument("--path", default="auto", choices=["auto", "ffma", "tensor"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the short runs of the other workloads")
    ap.add_argument("--kernel", default=None, choices=["assign", "update", "decode", "reshape", "fit", "linear", "linear_q4"])
    ap.add_argument("--N", type=int, default=1 << 20)
    ap.add_argument("--g", type=int, default=4)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--M", type=int, default=256)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--iters", type=int, default=2)
    args = ap.parse_args()
    if args.kernel:
        return run_kernel_mode(args)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = wl.WORKLOADS[args.workload]

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2503_13089_b200 import binding as cc
    from paper_2503_13089_b200 import sharding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    ctx = cc.Context(local_rank)
    path = {"auto": cc.PATH_AUTO, "ffma": cc.PATH_FFMA, "tensor": cc.PATH_TENSOR}[args.path]
    cc.cc_set_path(ctx, path)
    layout = cc.LAYOUT_PAPER_T
    peaks = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # > L2 (126 MB)

    # instruction-rate probes: the ceilings the E-step is measured against
    ctx.ensure_workspace(1024, 4, 16)
    fp32_scalar, fp32_packed = cc.cc_measure_fp32_peak(ctx)
    min_rate, probe_mhz, probe_sms = cc.cc_measure_min_rate(ctx)
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    per_clk, ceiling_scores = alu_ceiling(min_rate, sm_count)
    nominal_fp32 = NOMINAL_SM * NOMINAL_LANES * 2 * NOMINAL_MHZ * 1e6 / 1e12
    if args.path == "ffma":
        ceiling_for = lambda g: nominal_fp32 * 1e12 / (2 * g)       # noqa: E731  scores/s at the FP32 FMA peak
    else:
        ceiling_for = lambda g: ceiling_scores                      # noqa: E731

    # ---------------- headline workload.  The job is `world` copies of the workload's matrices (copy r with
    # seeds shifted by r: weak scaling); the library's size-balanced scheduler says which of them this rank
    # clusters.  Nothing is exchanged between ranks.
    job = [m for r in range(world) for m in sharding.matrices_for_rank(w, r)]
    mine = cc.cc_schedule_matrices([w.n_subvectors(m) for m in job], world, rank)
    specs = tuple(job[i] for i in mine)
    run = Runner(cc, torch, ctx, w, specs, layout)
    for _ in range(args.warmup):
        flush.zero_()
        run.step()
    cc.cc_poll_status(ctx)
    sampler = ClockSampler(local_rank).start() if rank == 0 else None
    ms_steps, launches = run.timed(args.steps, flush, barrier)
    clocks = sampler.stop() if sampler else None
    cc.cc_poll_status(ctx)
    prof_steps = max(1, min(args.steps, 3))
    phases = run.profiled(prof_steps, flush)
    resolved = run.near_ties()
    cc.cc_poll_status(ctx)
    ms_local = sum(ms_steps) / len(ms_steps)
    run.free_device()
    e2e_ms, h2d, d2h = run.e2e(args.steps, 1, flush, barrier)
    e2e_local = sum(e2e_ms) / len(e2e_ms)

    # ---------------- max over ranks
    evals_step_local = sum(N * w.K * (w.iters + 1) for N in run.Ns)   # iters E-steps + the final one
    t = torch.tensor([ms_local, e2e_local], dtype=torch.float64, device="cuda")
    tot = torch.tensor([float(evals_step_local)], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    ms_step, e2e_step = float(t[0]), float(t[1])
    total_evals = float(tot[0])

    if rank == 0:
        g, K, iters = w.g, w.K, w.iters
        summ = summarise(w, run.Ns, phases, prof_steps, peaks, ceiling_for(g), args.path)
        scan = summ["scan"]
        flops_launch = 2 * g * sum(run.Ns) * K / len(run.Ns)
        n0 = run.Ns[0]
        if args.path == "ffma":
            roofline = {"bound": "alu", "kernel": "assign_ffma_kernel (E-step distance scan, FP32 FMA path)",
                        "achieved": scan["achieved_tflops"], "peak": nominal_fp32, "unit": "TFLOP/s",
                        "frac": scan["achieved_tflops"] / nominal_fp32,
                        "peak_kind": "nominal FP32 FMA: 148 SMs x 128 lanes x 2 x 1965 MHz",
                        "peak_measured_ffma_scalar": fp32_scalar, "peak_measured_ffma_packed": fp32_packed,
                        "traffic": None}
        else:
            # DRAM bytes of one launch of the scan kernel: one ncu capture of this kernel at g = 4 on
            # 1,048,576 points (8,947,712 bytes read, 0 written: X once, the staged codebook and the
            # per-point results stay in L2), scaled by the number of points; other g were not captured
            traffic = n0 * (8947712.0 / 1048576.0) if g == 4 else None
            roofline = {"bound": "alu",
                        "kernel": "assign_tensor_persistent_kernel (E-step scan: tcgen05 scores + min-reduction epilogue)",
                        "achieved": scan["achieved_tflops"], "peak": ceiling_scores * 2 * g / 1e12, "unit": "TFLOP/s",
                        "frac": scan["frac"],
                        "peak_kind": "ALU min-reduction, of measured: %.1f scores per clock per SM (probe: min.f32 %.1f, "
                                     "three-input min.f32 %.1f, alternating %.1f lane-instructions per clock per SM on %d SMs "
                                     "at %.0f MHz) x %d SMs x %.0f MHz x 2g flops per score"
                                     % (per_clk, min_rate["min2"], min_rate["min3"], min_rate["mixed"], probe_sms, probe_mhz,
                                        sm_count, NOMINAL_MHZ),
                        "scores_per_s": scan["scores_per_s"], "peak_scores_per_s": ceiling_scores,
                        "frac_at_sampled_clock": (scan["frac"] * NOMINAL_MHZ / clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None,
                        "e_step": summ["e_step"],
                        "x_fp32_fma_peak": summ["x_fp32_fma_peak"],
                        "frac_of_measured_fp32_fma": scan["achieved_tflops"] / fp32_scalar if fp32_scalar else None,
                        "tensor_frac_algorithmic_of_measured_bf16": summ["tensor_frac_algorithmic_of_measured_bf16"],
                        "tensor_frac_executed_of_measured_bf16": summ["tensor_frac_executed_of_measured_bf16"],
                        "contraction_columns": summ["contraction_columns"],
                        "peak_measured_ffma_scalar": fp32_scalar, "peak_measured_ffma_packed": fp32_packed,
                        "traffic": traffic}
        roofline.update({"avg_launch_ms": scan["avg_launch_ms"], "launches": scan["launches"],
                         "flops_per_launch": flops_launch,
                         "timed_in": "%d profiled steps run right after the timed region (an event pair around every "
                                     "launch, on the launching stream); the timed region itself runs without them" % prof_steps})

        # ---------------- the other configurations, briefly (one GPU only: all N GPUs would be held meanwhile)
        others = []
        Ns_head, W_head = list(run.Ns), run.mats[0][1]
        del run
        torch.cuda.empty_cache()
        if world == 1 and not args.no_secondary:
            for name in sorted(wl.WORKLOADS):
                if name == w.name:
                    continue
                w2 = wl.WORKLOADS[name]
                r2 = Runner(cc, torch, ctx, w2, w2.matrices, layout)
                flush.zero_()
                r2.step()
                cc.cc_poll_status(ctx)
                s2 = ClockSampler(local_rank).start()
                ms2, _ = r2.timed(2, flush, barrier)
                ph2 = r2.profiled(1, flush)
                c2 = s2.stop()
                nt2 = r2.near_ties()
                cc.cc_poll_status(ctx)
                sm2 = summarise(w2, r2.Ns, ph2, 1, peaks, ceiling_for(w2.g), args.path)
                ms2m = sum(ms2) / len(ms2)
                others.append({"workload": name, "g": w2.g, "K": w2.K, "iters": w2.iters, "N_per_matrix": r2.Ns,
                               "steps": 2, "warmup": 1, "ms_per_step": ms2m,
                               "value": sum(N * w2.K * (w2.iters + 1) for N in r2.Ns) / (ms2m * 1e-3),
                               "s_per_lloyd_iteration": sm2["s_per_lloyd_iteration"],
                               "scan": sm2["scan"], "e_step": sm2["e_step"],
                               "tensor_frac_executed_of_measured_bf16": sm2.get("tensor_frac_executed_of_measured_bf16"),
                               "contraction_columns": sm2.get("contraction_columns"),
                               "hbm_kernels": sm2["hbm_kernels"], "near_tie_points_per_assign": nt2, "clocks": c2})
                r2.free_device()
                del r2
                torch.cuda.empty_cache()

        linear = linear_rows(cc, torch, ctx, peaks) if (world == 1 and not args.no_secondary) else []

        cpu_baseline = None
        if not args.no_cpu_baseline and world == 1:
            import oracle
            spec0 = specs[0]
            X0 = oracle.reshape_subvectors(W_head, g)
            N0 = len(X0)
            frac = min(1.0, 6.0e10 / (N0 * K))
            sel = None if frac >= 1.0 else wl.subset_positions(N0, frac, 99)
            C0 = oracle.init_codebook(X0, K, spec0.init_seed)
            t0 = time.perf_counter()
            idx0, _, _ = oracle.assign(X0, C0, sel)
            C0, _ = oracle.update(X0 if sel is None else X0[sel], idx0, C0)
            dt = time.perf_counter() - t0
            n_pts = N0 if sel is None else len(sel)
            cpu_baseline = {"value": n_pts * K / dt, "unit": "distance evaluations/s",
                            "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                            "sample": "one Lloyd iteration on %s of the %d sub-vectors, all %d centroids, %.1f s"
                                      % ("all" if sel is None else "a seeded %.5f share" % frac, N0, K, dt)}

        line = {
            "metric": "distance_evals_per_s", "value": total_evals / (ms_step * 1e-3),
            "unit": "distance evaluations/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "matrices_per_rank": len(specs), "g": g, "K": K, "iters": iters,
                       "N_per_matrix": Ns_head,
                       "layout": "paper_transpose", "path": args.path,
                       "l2": "flushed between timed steps (256 MB write)",
                       "step": "reshape + init + %d x (assign + update) + finalize + decode per matrix" % iters},
            "s_per_lloyd_iteration": summ["s_per_lloyd_iteration"],
            "e_step_ms": summ["e_step_ms"], "m_step_ms": summ["m_step_ms"], "final_e_step_ms": summ["final_e_step_ms"],
            "near_tie_points_per_assign": resolved,
            "ms_steps": ms_steps,
            "e2e": {"value": total_evals / (e2e_step * 1e-3), "unit": "distance evaluations/s",
                    "ms_per_step": e2e_step, "steps": len(e2e_ms), "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "api": "cc_compress_host: pinned host W in; FP16 codebook, codes, objective trace and the decoded "
                           "matrix out (the same work as the device-resident step plus the copies); its device buffer "
                           "is allocated by one untimed call"},
            "gpu_launches": launches,
            "roofline": roofline,
            "hbm_kernels": summ["hbm_kernels"],
            "kernels": summ["kernel_classes"],
            "workloads": others,
            "linear_forward": linear,
            "peaks": peaks,
            "probes": {"min_rate_lane_instr_per_clk_per_sm": min_rate, "probe_sm_mhz": probe_mhz,
                       "probe_distinct_sms": probe_sms, "fp32_fma_tflops_scalar": fp32_scalar,
                       "fp32_fma_tflops_packed": fp32_packed},
            "clocks": clocks,
            "cpu_baseline": cpu_baseline,
            "context": {"paper_70B_clustering_hours_1gpu": 25.6},
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

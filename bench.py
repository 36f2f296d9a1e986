#!/usr/bin/env python
"""Benchmark of the clustering hot path (reshape -> init -> Lloyd iterations -> finalize -> decode).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one pass of the whole path over one synthetic weight matrix of the workload
(default: the 4096x4096, g=4, K=4096, 20-iteration configuration).  Rank 0 prints one JSON line.
With N > 1 every rank clusters its own matrix (different seed) and no data crosses ranks: the
paper's "clustering of different matrices is independent".
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

DEFAULT_WORKLOAD = "cfg2_4096x4096_g4_k4096"
NOMINAL_SM, NOMINAL_LANES, NOMINAL_MHZ = 148, 128, 1965.0   # B200: SMs, FP32 lanes per SM, max SM clock


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
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

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()          # the exact process started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def algorithmic_counts(w: wl.Workload, spec: wl.MatrixSpec):
    N = w.n_subvectors(spec)
    g, K = w.g, w.K
    return {
        "N": N,
        "dist_evals_per_assign": N * K,
        "flops_per_assign": 2 * g * N * K,
        "bytes_update": N * (2 * g + 2) + K * (4 * g + 4),
        "bytes_decode": N * (2 + 2 * g),
        "bytes_reshape": N * 4 * g,
    }


def run_reference(args, w: wl.Workload):
    """The CPU oracle as it stands, timed on the host cores: each step is one Lloyd iteration
    (E-step + M-step) over the workload's first matrix from its seeded start."""
    import oracle
    spec = w.matrices[0]
    cores = len(os.sched_getaffinity(0))
    W = wl.make_matrix(spec)
    X = oracle.reshape_subvectors(W, w.g)
    N = len(X)
    # bounded sample: keep one step near a few seconds of CPU work
    budget_evals = 2.0e10
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
              % ("all" if sel is None else "a seeded %.4f share" % frac, N, w.K))
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(wl.WORKLOADS))
    ap.add_argument("--path", default="auto", choices=["auto", "ffma", "tensor"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
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

    # every rank clusters its own matrices: rank r takes the workload's matrices with seeds shifted by r
    specs = sharding.matrices_for_rank(w, rank)
    ctx = cc.Context(local_rank)
    path = {"auto": cc.PATH_AUTO, "ffma": cc.PATH_FFMA, "tensor": cc.PATH_TENSOR}[args.path]
    cc.cc_set_path(ctx, path)
    g, K, iters = w.g, w.K, w.iters
    layout = cc.LAYOUT_PAPER_T

    mats = []
    for spec in specs:
        Wn = wl.make_matrix(spec)
        Wh = torch.from_numpy(Wn.view(np.int16)).view(torch.float16).pin_memory()
        mats.append((spec, Wn, Wh))
    maxN = max(w.n_subvectors(s) for s in specs)
    ctx.ensure_workspace(maxN, g, K)
    stream = torch.cuda.current_stream()

    bufs = {}
    for spec, Wn, Wh in mats:
        N = w.n_subvectors(spec)
        bufs[spec.name] = dict(
            W=Wh.cuda(), X=torch.empty((N, g), dtype=torch.float16, device="cuda"),
            C=torch.empty((K, g), dtype=torch.float32, device="cuda"),
            C16=torch.empty((K, g), dtype=torch.float16, device="cuda"),
            idx=torch.empty(N, dtype=torch.uint16, device="cuda"),
            dist=torch.empty(N, dtype=torch.float32, device="cuda"),
            counts=torch.empty(K, dtype=torch.int32, device="cuda"),
            trace=torch.empty(iters + 1, dtype=torch.float64, device="cuda"),
            What=torch.empty((spec.d_out, spec.d_in), dtype=torch.float16, device="cuda"))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # > L2 (126 MB)

    def step():
        for spec, Wn, Wh in mats:
            b = bufs[spec.name]
            N = w.n_subvectors(spec)
            cc.cc_reshape_subvectors(ctx, b["W"], spec.d_out, spec.d_in, g, layout, b["X"])
            cc.cc_init_codebook(ctx, b["X"], N, g, K, spec.init_seed, b["C"])
            cc.cc_fit(ctx, b["X"], N, g, K, iters, b["C"], b["idx"], b["dist"], b["counts"], b["trace"])
            cc.cc_finalize(ctx, b["X"], N, g, b["C"], K, b["C16"], b["idx"], b["dist"], b["trace"][iters:])
            cc.cc_decode(ctx, b["C16"], K, g, b["idx"], spec.d_out, spec.d_in, layout, b["What"])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    fp32_scalar, fp32_packed = cc.cc_measure_fp32_peak(ctx)
    nres = torch.zeros(1, dtype=torch.int64, device="cuda")
    for _ in range(args.warmup):
        flush.zero_()
        step()
    cc.cc_poll_status(ctx)

    # ---------------- timed region: device-resident inputs
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    cc.cc_profile_enable(ctx, True)
    cc.cc_profile_read(ctx)
    launches0 = cc.cc_launch_count(ctx)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for a, b in ev:
        flush.zero_()            # L2 flush between timed steps (outside the step's event pair)
        a.record(stream)
        step()
        b.record(stream)
    barrier()
    launches = cc.cc_launch_count(ctx) - launches0
    prof = cc.cc_profile_read(ctx)
    cc.cc_profile_enable(ctx, False)
    clocks = sampler.stop() if rank == 0 else None
    cc.cc_poll_status(ctx)
    # how many points the last E-step state sends to the exact stage (one extra, untimed call)
    b0 = bufs[specs[0].name]
    cc.cc_assign(ctx, b0["X"], w.n_subvectors(specs[0]), g, b0["C"], K, b0["idx"], b0["dist"], None, nres)
    resolved = int(nres.item())
    ms_steps = [a.elapsed_time(b) for a, b in ev]
    ms_local = sum(ms_steps) / len(ms_steps)

    # ---------------- end to end: host buffers in, host buffers out, through cc_compress_host
    e2e_ms = []
    h2d = d2h = 0
    outs = []
    for spec, Wn, Wh in mats:
        N = w.n_subvectors(spec)
        outs.append((torch.empty((K, g), dtype=torch.float16).pin_memory(), torch.empty(N, dtype=torch.uint16).pin_memory(),
                     torch.empty(iters + 1, dtype=torch.float64).pin_memory()))
        h2d += Wh.numel() * 2
        d2h += K * g * 2 + N * 2 + (iters + 1) * 8
    del bufs
    torch.cuda.empty_cache()
    for s in range(1 + max(1, min(args.steps, 2))):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        flush.zero_()
        barrier()
        a.record(stream)
        for (spec, Wn, Wh), (C16h, idxh, trh) in zip(mats, outs):
            cc.cc_compress_host(ctx, Wh, spec.d_out, spec.d_in, g, K, iters, spec.init_seed, layout, C16h, idxh, trh)
        b.record(stream)
        barrier()
        if s > 0:
            e2e_ms.append(a.elapsed_time(b))
    e2e_local = sum(e2e_ms) / len(e2e_ms)

    # ---------------- max over ranks
    evals_step_local = sum(w.n_subvectors(s) * K * (iters + 1) for s in specs)   # iters E-steps + the final one
    t = torch.tensor([ms_local, e2e_local], dtype=torch.float64, device="cuda")
    tot = torch.tensor([float(evals_step_local)], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    ms_step, e2e_step = float(t[0]), float(t[1])
    total_evals = float(tot[0])

    if rank == 0:
        peaks = measured_peaks()
        counts = [algorithmic_counts(w, s) for s in specs]
        ms_assign, n_assign = prof["assign_main"]
        flops_launch = sum(c["flops_per_assign"] for c in counts) / len(counts)
        avg_ms = ms_assign / max(n_assign, 1)
        achieved_tf = flops_launch / (avg_ms * 1e-3) / 1e12 if avg_ms > 0 else 0.0
        nominal_fp32 = NOMINAL_SM * NOMINAL_LANES * 2 * NOMINAL_MHZ * 1e6 / 1e12
        if args.path == "ffma":
            # FP32 FMA scan: 2g flops per distance evaluation against the FP32 FMA pipes
            roofline = {"bound": "alu", "kernel": "assign_ffma_kernel (E-step distance scan, FP32 FMA path)",
                        "achieved": achieved_tf, "peak": nominal_fp32, "unit": "TFLOP/s",
                        "frac": achieved_tf / nominal_fp32,
                        "peak_kind": "nominal FP32 FMA: 148 SMs x 128 lanes x 2 x 1965 MHz",
                        "peak_measured_ffma_scalar": fp32_scalar, "peak_measured_ffma_packed": fp32_packed,
                        "avg_launch_ms": avg_ms, "launches": n_assign, "flops_per_launch": flops_launch,
                        "traffic": None}
        else:
            # tensor-core scan: the contraction is cheap (1-3 MMA steps per 128 x 256 tile); the kernel
            # is bound by the min-reduction of the scores on the ALU pipes, one lane-operation per score
            # (a 3-input min retires two scores in two pipe cycles).  Peak: 148 SMs x 128 lanes x 1965 MHz
            # scores/s, expressed in the same 2g flops per distance evaluation as `achieved`.
            evals_launch = flops_launch / (2 * g)
            peak_scores = NOMINAL_SM * NOMINAL_LANES * NOMINAL_MHZ * 1e6
            peak_tf = peak_scores * 2 * g / 1e12
            kd34, kd24, kd22 = ((3 * g + 4 + 15) // 16 * 16, (2 * g + 4 + 15) // 16 * 16, (2 * g + 2 + 15) // 16 * 16)
            kd = kd34 if (kd34 <= 48 and kd34 <= min(kd24, kd22)) else min(kd24, kd22)   # the library's choice of operand pieces
            executed_tf = achieved_tf * kd / g
            # DRAM bytes of one launch of the scan kernel: one ncu capture of this kernel at g = 4 on
            # 1,048,576 points (8,947,712 bytes read, 0 written: X once, the staged codebook and the
            # per-point results stay in L2), scaled by the number of points; other g were not captured
            traffic = counts[0]["N"] * (8947712.0 / 1048576.0) if g == 4 else None
            roofline = {"bound": "alu", "kernel": "assign_tensor_kernel (E-step: tcgen05 scores + min-reduction epilogue)",
                        "achieved": achieved_tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved_tf / peak_tf,
                        "peak_kind": "ALU min-reduction: 148 SMs x 128 lanes x 1965 MHz scores/s x 2g flops per score",
                        "scores_per_s": evals_launch / (avg_ms * 1e-3) if avg_ms > 0 else 0.0,
                        "x_fp32_fma_peak": achieved_tf / nominal_fp32,
                        "tensor_frac_algorithmic_of_measured_bf16": achieved_tf / peaks["bf16_tflops"],
                        "tensor_frac_executed_of_measured_bf16": executed_tf / peaks["bf16_tflops"],
                        "contraction_columns": kd,
                        "peak_measured_ffma_scalar": fp32_scalar,
                        "avg_launch_ms": avg_ms, "launches": n_assign, "flops_per_launch": flops_launch,
                        "traffic": traffic}
        kern = {}
        for k, (ms, n) in prof.items():
            if n:
                kern[k] = {"ms_total": ms, "launches": n, "share": ms / max(sum(v[0] for v in prof.values()), 1e-9)}
        ms_upd, n_upd = prof["update_accum"]
        if n_upd:
            by = sum(c["bytes_update"] for c in counts) / len(counts)
            gbs = by / (ms_upd / n_upd * 1e-3) / 1e9
            kern["update_accum"].update({"algorithmic_GBs": gbs, "frac_of_hbm": gbs / peaks["hbm_gbs"]})
        ms_dec, n_dec = prof["decode"]
        if n_dec:
            by = sum(c["bytes_decode"] for c in counts) / len(counts)
            gbs = by / (ms_dec / n_dec * 1e-3) / 1e9
            kern["decode"].update({"algorithmic_GBs": gbs, "frac_of_hbm": gbs / peaks["hbm_gbs"]})
        ms_rs, n_rs = prof["reshape"]
        if n_rs:
            by = sum(c["bytes_reshape"] for c in counts) / len(counts)
            gbs = by / (ms_rs / n_rs * 1e-3) / 1e9
            kern["reshape"].update({"algorithmic_GBs": gbs, "frac_of_hbm": gbs / peaks["hbm_gbs"]})
        n_mat = len(specs)
        lloyd_ms = (prof["assign_main"][0] + prof["assign_prep"][0] + prof["assign_finish"][0] + prof["resolve"][0]
                    + prof["objective"][0] + prof["update_accum"][0] + prof["update_finish"][0]) / max(args.steps, 1)
        s_per_iter = lloyd_ms * 1e-3 / (n_mat * (iters + 1))

        cpu_baseline = None
        if not args.no_cpu_baseline:
            import oracle
            spec0, W0, _ = mats[0]
            X0 = oracle.reshape_subvectors(W0, g)
            N0 = len(X0)
            frac = min(1.0, 6.0e10 / (N0 * K))
            sel = None if frac >= 1.0 else wl.subset_positions(N0, frac, 99)
            C0 = oracle.init_codebook(X0, K, spec0.init_seed)
            t0 = time.perf_counter()
            reps = 3 if sel is None and N0 * K < 2.5e10 else 1
            for _ in range(reps):
                idx0, _, _ = oracle.assign(X0, C0, sel)
                C0, _ = oracle.update(X0 if sel is None else X0[sel], idx0, C0)
            dt = time.perf_counter() - t0
            n_pts = N0 if sel is None else len(sel)
            cpu_baseline = {"value": reps * n_pts * K / dt, "unit": "distance evaluations/s",
                            "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                            "sample": "%d Lloyd iteration(s) on %s of the %d sub-vectors, all %d centroids, %.1f s"
                                      % (reps, "all" if sel is None else "a seeded %.4f share" % frac, N0, K, dt)}

        line = {
            "metric": "distance_evals_per_s", "value": total_evals / (ms_step * 1e-3),
            "unit": "distance evaluations/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "matrices_per_rank": n_mat, "g": g, "K": K, "iters": iters,
                       "N_per_matrix": [w.n_subvectors(s) for s in specs], "layout": "paper_transpose",
                       "path": args.path, "l2": "flushed between timed steps (256 MB write)",
                       "step": "reshape + init + %d x (assign + update) + finalize + decode per matrix" % iters},
            "s_per_lloyd_iteration": s_per_iter,
            "near_tie_points_per_assign": resolved,
            "ms_steps": ms_steps,
            "e2e": {"value": total_evals / (e2e_step * 1e-3), "unit": "distance evaluations/s",
                    "ms_per_step": e2e_step, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "api": "cc_compress_host (pinned host buffers in and out; its device buffer is allocated by the untimed first call)"},
            "gpu_launches": launches,
            "roofline": roofline,
            "kernels": kern,
            "peaks": peaks,
            "clocks": clocks,
            "cpu_baseline": cpu_baseline,
            "context": {"paper_70B_clustering_hours_1gpu": 25.6},
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

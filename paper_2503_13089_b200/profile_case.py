"""Runs one kernel of the path a few times on a synthetic case (for ncu captures and quick timing).

    python -m paper_2503_13089_b200.profile_case --kernel assign --N 1048576 --g 4 --K 4096 [--path ffma]

Prints the mean device time of each kernel class over the repetitions.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as cc
from . import workloads as wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", default="assign", choices=["assign", "update", "decode", "reshape", "fit"])
    ap.add_argument("--N", type=int, default=1 << 20)
    ap.add_argument("--g", type=int, default=4)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--iters", type=int, default=2)
    ap.add_argument("--path", default="auto", choices=["auto", "ffma", "tensor"])
    a = ap.parse_args()
    N, g, K = a.N, a.g, a.K
    ctx = cc.Context(0)
    ctx.ensure_workspace(N, g, K)
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
    d_out, d_in = g * 1024, N // 1024
    if a.kernel in ("decode", "reshape"):
        assert d_in * 1024 == N, "N must be a multiple of 1024 for the reshape / decode cases"
    W = torch.empty((d_out, d_in), dtype=torch.float16, device="cuda")
    cc.cc_assign(ctx, X, N, g, C, K, idx, dist, obj, nres)      # warm-up; also valid codes for update / decode
    cc.cc_finalize(ctx, X, N, g, C, K, C16, idx, dist, obj)
    def once():
        if a.kernel == "assign":
            cc.cc_assign(ctx, X, N, g, C, K, idx, dist, obj, nres)
        elif a.kernel == "update":
            cc.cc_update(ctx, X, N, g, idx, K, C2, counts)
        elif a.kernel == "decode":
            cc.cc_decode(ctx, C16, K, g, idx, d_out, d_in, cc.LAYOUT_PAPER_T, W)
        elif a.kernel == "reshape":
            cc.cc_reshape_subvectors(ctx, W, d_out, d_in, g, cc.LAYOUT_PAPER_T, X2)
        else:
            cc.cc_fit(ctx, X, N, g, K, a.iters, C, idx, dist, counts, None)

    C2 = C.clone()
    X2 = torch.empty_like(X)
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


if __name__ == "__main__":
    main()

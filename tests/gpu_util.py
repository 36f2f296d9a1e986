"""Helpers for the GPU parity tests: numpy in, numpy out, everything through the C ABI."""
import numpy as np
import torch

import oracle
from paper_2503_13089_b200 import binding as cc

REL_TIE = 1e-6      # mismatches are tolerated only where the oracle's own distances nearly tie
REL_CENTROID = 1e-4
REL_OBJECTIVE = 1e-5

_ctx = None


def ctx():
    global _ctx
    if _ctx is None:
        _ctx = cc.Context(0)
    return _ctx


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype)
    return t.cuda()


def half_dev(a):
    assert a.dtype == np.float16
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.float16)


def u16_np(t):
    return t.cpu().view(torch.int16).numpy().view(np.uint16)


def gpu_assign(X, C, path=cc.PATH_AUTO, want_dist=True, want_flagged=False):
    c = ctx()
    N, g = X.shape
    K = C.shape[0]
    c.ensure_workspace(N, g, K)
    cc.cc_set_path(c, path)
    Xd, Cd = half_dev(X), dev(C.astype(np.float32))
    idx = torch.empty(max(N, 1), dtype=torch.uint16, device="cuda")
    dist = torch.empty(max(N, 1), dtype=torch.float32, device="cuda") if want_dist else None
    obj = torch.zeros(1, dtype=torch.float64, device="cuda")
    nres = torch.zeros(1, dtype=torch.int64, device="cuda")
    cc.cc_assign(c, Xd, N, g, Cd, K, idx, dist, obj, nres)
    cc.cc_poll_status(c)
    cc.cc_set_path(c, cc.PATH_AUTO)
    out = (u16_np(idx)[:N].astype(np.int32), None if dist is None else dist.cpu().numpy()[:N],
           float(obj.item()), int(nres.item()))
    if want_flagged:
        out = out + (last_flagged(N, g, K, out[3]),)
    return out


def last_flagged(N, g, K, count):
    """Point numbers the last E-step on the shared context sent to the exact FP64 stage."""
    pts = torch.empty(max(count, 1), dtype=torch.int32, device="cuda")
    cc.cc_last_flagged(ctx(), N, g, K, pts, count)
    torch.cuda.synchronize()
    return pts.cpu().numpy()[:count].astype(np.int64)


def gpu_update(X, idx, C_prev):
    c = ctx()
    N, g = X.shape
    K = C_prev.shape[0]
    c.ensure_workspace(N, g, K)
    Xd = half_dev(X)
    Cd = dev(C_prev.astype(np.float32))
    idxd = torch.from_numpy(idx.astype(np.uint16).view(np.int16)).cuda().view(torch.uint16)
    counts = torch.empty(K, dtype=torch.int32, device="cuda")
    cc.cc_update(c, Xd, N, g, idxd, K, Cd, counts)
    cc.cc_poll_status(c)
    return Cd.cpu().numpy(), counts.cpu().numpy()


def check_assign_against_oracle(X, C, idx_gpu, dist_gpu, sel=None, flagged=None):
    """Bit-exact indices except near-ties of the oracle's float64 distances; returns (#tolerated, o_idx, d1).
    `flagged`: the points the GPU decided in its exact FP64 stage, which uses the oracle's own
    arithmetic -- there even a near-tie must come out as the oracle's index."""
    o_idx, d1, d2 = oracle.assign(X, C, sel)
    gi = idx_gpu if sel is None else idx_gpu[sel]
    bad = np.flatnonzero(gi != o_idx)
    tolerated = 0
    rows = np.arange(len(X)) if sel is None else sel
    if flagged is not None and len(bad):
        wrong = np.intersect1d(rows[bad], flagged)
        assert len(wrong) == 0, "points decided by the exact stage differ from the oracle: %r" % wrong[:10]
    for r in bad:
        d_g = oracle.point_dist(X, int(rows[r]), C, int(gi[r]))
        rel = 0.0 if d_g == 0 else (d_g - d1[r]) / d_g
        assert rel < REL_TIE, "point %d: gpu %d (d=%r) vs oracle %d (d=%r)" % (rows[r], gi[r], d_g, o_idx[r], d1[r])
        tolerated += 1
    if dist_gpu is not None:
        dg = dist_gpu if sel is None else dist_gpu[sel]
        ok = gi == o_idx
        assert np.allclose(dg[ok], d1[ok], rtol=2e-7, atol=1e-44), np.abs(dg[ok] - d1[ok]).max()
    return tolerated, o_idx, d1


def centroid_rel_err(C_gpu, C_or, X):
    """max_j ||c_gpu - c_or||_inf / max(||c_or||_inf, 1e-3 rms(X))."""
    rms = float(np.sqrt(np.mean(X.astype(np.float64) ** 2)))
    den = np.maximum(np.abs(C_or).max(axis=1), 1e-3 * rms)
    return float((np.abs(C_gpu.astype(np.float64) - C_or.astype(np.float64)).max(axis=1) / den).max())

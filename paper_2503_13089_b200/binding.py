"""ctypes binding of libcluscomp.so: argument marshalling only.

Every function has the name and the argument order of its C entry point (see
include/cluscomp.h, which states meaning, layout and ownership).  Device arguments are
torch CUDA tensors (PyTorch supplies device memory and streams, nothing else); FP16 data
is a torch.float16 tensor, codes are torch.uint16.  A non-OK status raises CCError.
"""
from __future__ import annotations

import ctypes as ct
import os
from typing import Optional

import torch

from . import build as _build

CC_OK = 0
LAYOUT_PAPER_T = 0
LAYOUT_ROWS = 1
PATH_AUTO, PATH_FFMA, PATH_TENSOR = 0, 1, 2
EMPTY_KEEP, EMPTY_SPLIT_LARGEST = 0, 1

STATUS_NAMES = {
    0: "CC_OK", 1: "CC_ERR_NULL", 2: "CC_ERR_SHAPE", 3: "CC_ERR_UNSUPPORTED_G", 4: "CC_ERR_K_RANGE",
    5: "CC_ERR_N_LT_K", 6: "CC_ERR_ALIGN", 7: "CC_ERR_WORKSPACE", 8: "CC_ERR_NONFINITE",
    9: "CC_ERR_DEVICE_TIMEOUT", 10: "CC_ERR_CUDA", 11: "CC_ERR_LAYOUT", 12: "CC_ERR_STATIC_CAPACITY",
}
UPDATE_STATIC_MAX_KG = 262144

# name -> (restype, argtypes); mirrors include/cluscomp.h one to one
_vp, _i64, _i32, _u64, _sz, _dbl = ct.c_void_p, ct.c_int64, ct.c_int, ct.c_uint64, ct.c_size_t, ct.c_double
SIGNATURES = {
    "cc_create": (_i32, [ct.POINTER(_vp), _i32]),
    "cc_destroy": (_i32, [_vp]),
    "cc_status_string": (ct.c_char_p, [_i32]),
    "cc_workspace_bytes": (_sz, [_i64, _i32, _i32]),
    "cc_set_workspace": (_i32, [_vp, _vp, _sz]),
    "cc_set_path": (_i32, [_vp, _i32]),
    "cc_launch_count": (_i64, [_vp]),
    "cc_profile_enable": (_i32, [_vp, _i32]),
    "cc_profile_read": (_i32, [_vp, _vp, _vp]),
    "cc_measure_fp32_peak": (_i32, [_vp, _vp, _vp, _vp]),
    "cc_measure_min_rate": (_i32, [_vp, _vp, _vp, _vp, _vp]),
    "cc_num_subvectors": (_i64, [_i64, _i64, _i32, _i32]),
    "cc_bits_per_param": (_dbl, [_i64, _i64, _i32, _i32]),
    "cc_reshape_subvectors": (_i32, [_vp, _vp, _i64, _i64, _i32, _i32, _vp, _vp]),
    "cc_init_positions": (_i32, [_i64, _i32, _u64, _vp]),
    "cc_init_codebook": (_i32, [_vp, _vp, _i64, _i32, _i32, _u64, _vp, _vp]),
    "cc_set_codebook": (_i32, [_vp, _vp, _i32, _i32, _vp, _vp]),
    "cc_assign": (_i32, [_vp, _vp, _i64, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _vp]),
    "cc_last_flagged": (_i32, [_vp, _i64, _i32, _i32, _vp, _i64, _vp]),
    "cc_tensor_scores_ld": (_i64, [_i32]),
    "cc_tensor_scores": (_i32, [_vp, _vp, _i64, _i32, _vp, _i32, _vp, _vp]),
    "cc_tensor_finish_only": (_i32, [_vp, _vp, _i64, _i32, _vp, _i32, _vp, _vp, _vp, _vp]),
    "cc_selftest_bounded_wait": (_i32, [_vp, _i64, _vp, _vp]),
    "cc_update": (_i32, [_vp, _vp, _i64, _i32, _vp, _i32, _vp, _vp, _vp]),
    "cc_update_static": (_i32, [_i32, _vp, _i64, _i32, _vp, _i32, _vp, _vp, _vp]),
    "cc_codebook_grad": (_i32, [_vp, _vp, _i64, _i32, _vp, _i32, _vp, _vp]),
    "cc_fit": (_i32, [_vp, _vp, _i64, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "cc_set_empty_rule": (_i32, [_vp, _i32]),
    "cc_train_points": (_i64, [_i64, _i32, _i32]),
    "cc_sample_positions": (_i32, [_i64, _i64, _u64, _vp]),
    "cc_fit_sampled": (_i32, [_vp, _vp, _i64, _i32, _i32, _i32, _i32, _u64, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "cc_quantize_codebook": (_i32, [_vp, _vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp]),
    "cc_schedule_matrices": (_i32, [_i32, _vp, _i32, _i32, _vp, _vp]),
    "cc_compress_many": (_i32, [_vp, _i32, _vp, _vp, _vp, _i32, _i32, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _vp]),
    "cc_finalize": (_i32, [_vp, _vp, _i64, _i32, _vp, _i32, _vp, _vp, _vp, _vp, _vp]),
    "cc_decode": (_i32, [_vp, _vp, _i32, _i32, _vp, _i64, _i64, _i32, _vp, _vp]),
    "cc_linear_workspace_bytes": (_sz, [_vp, _i64, _i64, _i64]),
    "cc_linear_forward": (_i32, [_vp, _vp, _i64, _vp, _i32, _i32, _vp, _i64, _i64, _vp, _vp, _vp]),
    "cc_linear_forward_q4": (_i32, [_vp, _vp, _i64, _vp, _vp, _i32, _i32, _vp, _i64, _i64, _vp, _vp, _vp]),
    "cc_poll_status": (_i32, [_vp, _vp]),
    "cc_compress_host": (_i32, [_vp, _vp, _i64, _i64, _i32, _i32, _i32, _u64, _i32, _vp, _vp, _vp, _vp, _vp]),
}

_lib = None


class CCError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s returned %s" % (where, STATUS_NAMES.get(status, status)))


def library_path() -> str:
    return _build.LIB


def load() -> ct.CDLL:
    """Load libcluscomp.so (building it when the sources are newer); raises if that fails."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if os.environ.get("CLUSCOMP_NO_BUILD") != "1":
            path = _build.build()
        lib = ct.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)          # AttributeError if the library lacks a declared symbol
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _check(status: int, where: str) -> None:
    if status != CC_OK:
        raise CCError(status, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors must be contiguous"
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    return stream.cuda_stream or None


class Context:
    """Owns a cc_ctx and (optionally) a torch-allocated workspace."""

    def __init__(self, device: int = 0):
        self._h = _vp()
        _check(load().cc_create(ct.byref(self._h), device), "cc_create")
        self.device = device
        self._ws = None

    def close(self):
        if self._h:
            load().cc_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def ensure_workspace(self, N: int, g: int, K: int, at_least: int = 0) -> None:
        need = max(cc_workspace_bytes(N, g, K), at_least)
        if need == 0:
            raise CCError(2, "cc_workspace_bytes")
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device="cuda:%d" % self.device)
            cc_set_workspace(self, self._ws, self._ws.numel())


def cc_status_string(status: int) -> str:
    return load().cc_status_string(status).decode()


def cc_workspace_bytes(N: int, g: int, K: int) -> int:
    return int(load().cc_workspace_bytes(N, g, K))


def cc_set_workspace(ctx: Context, workspace: Optional[torch.Tensor], nbytes: int) -> None:
    _check(load().cc_set_workspace(ctx._h, _ptr(workspace), nbytes), "cc_set_workspace")


def cc_set_path(ctx: Context, path: int) -> None:
    _check(load().cc_set_path(ctx._h, path), "cc_set_path")


def cc_launch_count(ctx: Context) -> int:
    return int(load().cc_launch_count(ctx._h))


KERNEL_CLASSES = ("assign_main", "assign_prep", "resolve", "objective", "update_accum", "update_finish",
                  "reshape", "decode", "other", "assign_finish", "update_delta", "linear", "linear_reduce")


def cc_profile_enable(ctx: Context, on: bool) -> None:
    _check(load().cc_profile_enable(ctx._h, 1 if on else 0), "cc_profile_enable")


def cc_profile_read(ctx: Context):
    """Returns {kernel class: (total device ms, launches)} since the last read."""
    ms = (_dbl * len(KERNEL_CLASSES))()
    n = (_i64 * len(KERNEL_CLASSES))()
    _check(load().cc_profile_read(ctx._h, ms, n), "cc_profile_read")
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_CLASSES)}


def cc_measure_fp32_peak(ctx: Context, stream=None):
    """Returns (scalar FMA TFLOP/s, packed f32x2 FMA TFLOP/s) measured on the device."""
    a, b = _dbl(0.0), _dbl(0.0)
    _check(load().cc_measure_fp32_peak(ctx._h, ct.byref(a), ct.byref(b), _stream(stream)), "cc_measure_fp32_peak")
    return a.value, b.value


def cc_measure_min_rate(ctx: Context, stream=None):
    """Returns ({"min2", "min3", "mixed"}: lane-instructions per clock per SM, SM MHz, distinct SMs)."""
    r = (_dbl * 3)()
    mhz, sms = _dbl(0.0), ct.c_int32(0)
    _check(load().cc_measure_min_rate(ctx._h, r, ct.byref(mhz), ct.byref(sms), _stream(stream)),
           "cc_measure_min_rate")
    return {"min2": r[0], "min3": r[1], "mixed": r[2]}, mhz.value, sms.value


def cc_num_subvectors(d_out: int, d_in: int, g: int, layout: int = LAYOUT_PAPER_T) -> int:
    return int(load().cc_num_subvectors(d_out, d_in, g, layout))


def cc_bits_per_param(d_out: int, d_in: int, g: int, K: int) -> float:
    return float(load().cc_bits_per_param(d_out, d_in, g, K))


def cc_reshape_subvectors(ctx, W, d_out, d_in, g, layout, X, stream=None) -> None:
    _check(load().cc_reshape_subvectors(ctx._h, _ptr(W), d_out, d_in, g, layout, _ptr(X), _stream(stream)),
           "cc_reshape_subvectors")


def cc_init_positions(N: int, K: int, seed: int):
    import numpy as np
    pos = np.empty(max(K, 1), dtype=np.int64)
    _check(load().cc_init_positions(N, K, seed, pos.ctypes.data_as(_vp)), "cc_init_positions")
    return pos[:K]


def cc_init_codebook(ctx, X, N, g, K, seed, C, stream=None) -> None:
    _check(load().cc_init_codebook(ctx._h, _ptr(X), N, g, K, seed, _ptr(C), _stream(stream)), "cc_init_codebook")


def cc_set_codebook(ctx, C0, K, g, C, stream=None) -> None:
    """C0: a torch tensor on the host or on the device, or a contiguous float32 numpy array."""
    if hasattr(C0, "ctypes"):
        assert C0.dtype.name == "float32" and C0.flags["C_CONTIGUOUS"]
        src = C0.ctypes.data
    else:
        src = _ptr(C0)
    _check(load().cc_set_codebook(ctx._h, src, K, g, _ptr(C), _stream(stream)), "cc_set_codebook")


def cc_assign(ctx, X, N, g, C, K, idx, dist=None, objective=None, n_resolved=None, stream=None) -> None:
    _check(load().cc_assign(ctx._h, _ptr(X), N, g, _ptr(C), K, _ptr(idx), _ptr(dist), _ptr(objective),
                            _ptr(n_resolved), _stream(stream)), "cc_assign")


def cc_selftest_bounded_wait(ctx, limit_cycles: int):
    """Returns (results[4], cycles[2]) of the bounded-wait self-test (see cluscomp.h)."""
    res = (ct.c_int32 * 4)()
    cyc = (ct.c_int64 * 2)()
    _check(load().cc_selftest_bounded_wait(ctx._h, limit_cycles, ct.cast(res, ct.c_void_p), ct.cast(cyc, ct.c_void_p)),
           "cc_selftest_bounded_wait")
    return list(res), list(cyc)


def cc_last_flagged(ctx, N, g, K, points, count, stream=None) -> None:
    _check(load().cc_last_flagged(ctx._h, N, g, K, _ptr(points), count, _stream(stream)), "cc_last_flagged")


def cc_tensor_scores_ld(K: int) -> int:
    return int(load().cc_tensor_scores_ld(K))


def cc_tensor_scores(ctx, X, N, g, C, K, scores, stream=None) -> None:
    _check(load().cc_tensor_scores(ctx._h, _ptr(X), N, g, _ptr(C), K, _ptr(scores), _stream(stream)),
           "cc_tensor_scores")


def cc_tensor_finish_only(ctx, X, N, g, C, K, scan, idx, dist, stream=None) -> None:
    _check(load().cc_tensor_finish_only(ctx._h, _ptr(X), N, g, _ptr(C), K, _ptr(scan), _ptr(idx), _ptr(dist),
                                        _stream(stream)), "cc_tensor_finish_only")


def cc_update(ctx, X, N, g, idx, K, C, counts, stream=None) -> None:
    _check(load().cc_update(ctx._h, _ptr(X), N, g, _ptr(idx), K, _ptr(C), _ptr(counts), _stream(stream)),
           "cc_update")


def cc_update_static(device, X, N, g, idx, K, C, counts, stream=None) -> None:
    """cc_update for callers that may not allocate device memory: no context, no workspace; the
    accumulators are a fixed array inside the library (K * g <= UPDATE_STATIC_MAX_KG)."""
    _check(load().cc_update_static(device, _ptr(X), N, g, _ptr(idx), K, _ptr(C), _ptr(counts), _stream(stream)),
           "cc_update_static")


def cc_codebook_grad(ctx, dX, N, g, idx, K, dC, stream=None) -> None:
    _check(load().cc_codebook_grad(ctx._h, _ptr(dX), N, g, _ptr(idx), K, _ptr(dC), _stream(stream)),
           "cc_codebook_grad")


def cc_fit(ctx, X, N, g, K, iters, C, idx, dist, counts, objective_trace=None, stream=None) -> None:
    _check(load().cc_fit(ctx._h, _ptr(X), N, g, K, iters, _ptr(C), _ptr(idx), _ptr(dist), _ptr(counts),
                         _ptr(objective_trace), _stream(stream)), "cc_fit")


def cc_set_empty_rule(ctx, rule: int) -> None:
    _check(load().cc_set_empty_rule(ctx._h, rule), "cc_set_empty_rule")


def cc_train_points(N: int, K: int, max_points_per_centroid: int) -> int:
    return int(load().cc_train_points(N, K, max_points_per_centroid))


def cc_sample_positions(N: int, n: int, seed: int):
    import numpy as np
    pos = np.empty(max(n, 1), dtype=np.uint32)
    _check(load().cc_sample_positions(N, n, seed, pos.ctypes.data_as(_vp)), "cc_sample_positions")
    return pos[:n]


def cc_fit_sampled(ctx, X, N, g, K, iters, max_points_per_centroid, seed, X_train, C, idx, dist, counts,
                   objective_trace=None, stream=None) -> None:
    _check(load().cc_fit_sampled(ctx._h, _ptr(X), N, g, K, iters, max_points_per_centroid, seed, _ptr(X_train), _ptr(C),
                                 _ptr(idx), _ptr(dist), _ptr(counts), _ptr(objective_trace), _stream(stream)),
           "cc_fit_sampled")


def cc_quantize_codebook(ctx, C16, K, g, bits, q, scale, C16_dequantized=None, stream=None) -> None:
    _check(load().cc_quantize_codebook(ctx._h, _ptr(C16), K, g, bits, _ptr(q), _ptr(scale), _ptr(C16_dequantized),
                                       _stream(stream)), "cc_quantize_codebook")


def cc_schedule_matrices(sizes, world: int, rank: int):
    """Indices (increasing) of the matrices that fall to `rank` in the size-balanced split."""
    n = len(sizes)
    arr = (_i64 * max(n, 1))(*[int(v) for v in sizes])
    mine = (ct.c_int32 * max(n, 1))()
    cnt = ct.c_int32(0)
    _check(load().cc_schedule_matrices(n, arr, world, rank, mine, ct.byref(cnt)), "cc_schedule_matrices")
    return [int(mine[i]) for i in range(cnt.value)]


def cc_compress_many(ctx, W_hosts, d_outs, d_ins, g, K, iters, seeds, layout, C16_hosts, idx_hosts,
                     objective_trace_hosts=None, W_hat_hosts=None, stream=None) -> None:
    """Lists of HOST tensors, one entry per matrix (entries of the two optional lists may be None)."""
    n = len(W_hosts)

    def ptrs(lst):
        if lst is None:
            return None
        assert len(lst) == n and all(t is None or not t.is_cuda for t in lst)
        return (_vp * max(n, 1))(*[_ptr(t) for t in lst])

    _check(load().cc_compress_many(ctx._h, n, ptrs(W_hosts), (_i64 * max(n, 1))(*d_outs), (_i64 * max(n, 1))(*d_ins), g, K,
                                   iters, (_u64 * max(n, 1))(*seeds), layout, ptrs(C16_hosts), ptrs(idx_hosts),
                                   ptrs(objective_trace_hosts), ptrs(W_hat_hosts), _stream(stream)), "cc_compress_many")


def cc_finalize(ctx, X, N, g, C, K, C16, idx, dist=None, objective=None, stream=None) -> None:
    _check(load().cc_finalize(ctx._h, _ptr(X), N, g, _ptr(C), K, _ptr(C16), _ptr(idx), _ptr(dist),
                              _ptr(objective), _stream(stream)), "cc_finalize")


def cc_decode(ctx, C16, K, g, idx, d_out, d_in, layout, W_hat, stream=None) -> None:
    _check(load().cc_decode(ctx._h, _ptr(C16), K, g, _ptr(idx), d_out, d_in, layout, _ptr(W_hat),
                            _stream(stream)), "cc_decode")


def cc_linear_workspace_bytes(ctx, M: int, d_out: int, d_in: int) -> int:
    return int(load().cc_linear_workspace_bytes(ctx._h, M, d_out, d_in))


def cc_linear_forward(ctx, x, M, C16, K, g, idx, d_out, d_in, bias, y, stream=None) -> None:
    _check(load().cc_linear_forward(ctx._h, _ptr(x), M, _ptr(C16), K, g, _ptr(idx), d_out, d_in, _ptr(bias), _ptr(y),
                                    _stream(stream)), "cc_linear_forward")


def cc_linear_forward_q4(ctx, x, M, q, scale, K, g, idx, d_out, d_in, bias, y, stream=None) -> None:
    _check(load().cc_linear_forward_q4(ctx._h, _ptr(x), M, _ptr(q), _ptr(scale), K, g, _ptr(idx), d_out, d_in, _ptr(bias),
                                       _ptr(y), _stream(stream)), "cc_linear_forward_q4")


def cc_poll_status(ctx, stream=None) -> None:
    _check(load().cc_poll_status(ctx._h, _stream(stream)), "cc_poll_status")


def cc_compress_host(ctx, W_host, d_out, d_in, g, K, iters, seed, layout, C16_host, idx_host,
                     objective_trace_host=None, W_hat_host=None, stream=None) -> None:
    """All tensor arguments are HOST tensors here (pinned memory makes the copies asynchronous)."""
    for t in (W_host, C16_host, idx_host, objective_trace_host, W_hat_host):
        assert t is None or not t.is_cuda
    _check(load().cc_compress_host(ctx._h, _ptr(W_host), d_out, d_in, g, K, iters, seed, layout, _ptr(C16_host),
                                   _ptr(idx_host), _ptr(objective_trace_host), _ptr(W_hat_host),
                                   _stream(stream)), "cc_compress_host")

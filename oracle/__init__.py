"""CPU oracle (float64, plain C) for the ClusComp clustering path.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg, never by the product package.  This wrapper only
marshals numpy arrays into `cluscomp_oracle.c`; all arithmetic lives there.
"""
from __future__ import annotations

import ctypes as ct
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

LAYOUT_PAPER_T = 0
LAYOUT_ROWS = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cluscomp_oracle.c")
_LIB = os.path.join(_HERE, "libcluscomp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ct.CDLL(build())
        i64, i32, u64, dbl, vp = ct.c_int64, ct.c_int, ct.c_uint64, ct.c_double, ct.c_void_p
        lib.oc_num_subvectors.restype = i64
        lib.oc_num_subvectors.argtypes = [i64, i64, i32, i32]
        lib.oc_bits_per_param.restype = dbl
        lib.oc_bits_per_param.argtypes = [i64, i64, i32, i32]
        lib.oc_reshape.argtypes = [vp, i64, i64, i32, i32, vp]
        lib.oc_decode.argtypes = [vp, i32, i32, vp, i64, i64, i32, vp]
        lib.oc_init_positions.argtypes = [i64, i32, u64, vp]
        lib.oc_init_codebook.argtypes = [vp, i64, i32, i32, u64, vp]
        lib.oc_assign.argtypes = [vp, i64, i32, vp, i32, vp, i64, vp, vp, vp]
        lib.oc_point_dist.restype = dbl
        lib.oc_point_dist.argtypes = [vp, i64, i32, vp, i32]
        lib.oc_update.argtypes = [vp, i64, i32, vp, i32, vp, vp]
        lib.oc_codebook_grad.argtypes = [vp, i64, i32, vp, i32, vp]
        lib.oc_fit.argtypes = [vp, i64, i32, i32, i32, vp, vp, vp, vp, vp]
        lib.oc_linear_forward.argtypes = [vp, i64, vp, i32, vp, i64, i64, vp, vp]
        lib.oc_quantize_codebook.argtypes = [vp, i64, i32, vp, vp, vp]
        lib.oc_split_empty.argtypes = [vp, i32, i32, vp]
        lib.oc_float_to_half.argtypes = [vp, i64, vp]
        lib.oc_half_to_double.argtypes = [vp, i64, vp]
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ct.c_void_p)


def _half(a: np.ndarray) -> np.ndarray:
    assert a.dtype == np.float16, a.dtype
    return np.ascontiguousarray(a)


def num_subvectors(d_out: int, d_in: int, g: int, layout: int = LAYOUT_PAPER_T) -> int:
    return int(_load().oc_num_subvectors(d_out, d_in, g, layout))


def bits_per_param(d_out: int, d_in: int, g: int, K: int) -> float:
    return float(_load().oc_bits_per_param(d_out, d_in, g, K))


def reshape_subvectors(W: np.ndarray, g: int, layout: int = LAYOUT_PAPER_T) -> np.ndarray:
    W = _half(W)
    d_out, d_in = W.shape
    N = num_subvectors(d_out, d_in, g, layout)
    X = np.empty((N, g), dtype=np.float16)
    _load().oc_reshape(_p(W), d_out, d_in, g, layout, _p(X))
    return X


def decode(C16: np.ndarray, idx: np.ndarray, d_out: int, d_in: int,
           layout: int = LAYOUT_PAPER_T) -> np.ndarray:
    C16 = _half(C16)
    K, g = C16.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    assert idx.size == num_subvectors(d_out, d_in, g, layout)
    assert idx.min() >= 0 and idx.max() < K
    W_hat = np.empty((d_out, d_in), dtype=np.float16)
    _load().oc_decode(_p(C16), K, g, _p(idx), d_out, d_in, layout, _p(W_hat))
    return W_hat


def init_positions(N: int, K: int, seed: int) -> np.ndarray:
    pos = np.empty(K, dtype=np.int64)
    assert 1 <= K <= N
    rc = _load().oc_init_positions(N, K, seed, _p(pos))
    assert rc == 0
    return pos


def init_codebook(X: np.ndarray, K: int, seed: int) -> np.ndarray:
    X = _half(X)
    N, g = X.shape
    assert 1 <= K <= N
    C = np.empty((K, g), dtype=np.float32)
    rc = _load().oc_init_codebook(_p(X), N, g, K, seed, _p(C))
    assert rc == 0
    return C


def assign(X: np.ndarray, C: np.ndarray, sel: Optional[np.ndarray] = None
           ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """E-step.  Returns (idx int32, best distance, second-best distance) in float64."""
    X = _half(X)
    C = np.ascontiguousarray(C, dtype=np.float32)
    N, g = X.shape
    K = C.shape[0]
    assert C.shape[1] == g and g <= 64
    if sel is not None:
        sel = np.ascontiguousarray(sel, dtype=np.int64)
        assert sel.size == 0 or (sel.min() >= 0 and sel.max() < N)
    n = N if sel is None else sel.size
    idx = np.empty(n, dtype=np.int32)
    d1 = np.empty(n, dtype=np.float64)
    d2 = np.empty(n, dtype=np.float64)
    _load().oc_assign(_p(X), N, g, _p(C), K, _p(sel), 0 if sel is None else sel.size,
                      _p(idx), _p(d1), _p(d2))
    return idx, d1, d2


def point_dist(X: np.ndarray, i: int, C: np.ndarray, j: int) -> float:
    X = _half(X)
    C = np.ascontiguousarray(C, dtype=np.float32)
    return float(_load().oc_point_dist(_p(X), int(i), X.shape[1], _p(C), int(j)))


def update(X: np.ndarray, idx: np.ndarray, C_prev: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """M-step.  Returns (new centroids float32, counts int64); empty clusters keep C_prev."""
    X = _half(X)
    N, g = X.shape
    C = np.array(C_prev, dtype=np.float32, order="C", copy=True)
    K = C.shape[0]
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    assert idx.shape == (N,) and (N == 0 or (idx.min() >= 0 and idx.max() < K))
    counts = np.empty(K, dtype=np.int64)
    _load().oc_update(_p(X), N, g, _p(idx), K, _p(C), _p(counts))
    return C, counts


def codebook_grad(dX: np.ndarray, idx: np.ndarray, K: int) -> np.ndarray:
    """dC[j] = sum of dX[i] over the sub-vectors coded j (K x g float32)."""
    dX = _half(dX)
    N, g = dX.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    assert idx.shape == (N,) and (N == 0 or (idx.min() >= 0 and idx.max() < K))
    dC = np.empty((K, g), dtype=np.float32)
    _load().oc_codebook_grad(_p(dX), N, g, _p(idx), K, _p(dC))
    return dC


def fit(X: np.ndarray, C0: np.ndarray, iters: int):
    """iters x (E-step, M-step).  Returns (C, idx of the last E-step, d1, counts, objective[iters])."""
    X = _half(X)
    N, g = X.shape
    C = np.array(C0, dtype=np.float32, order="C", copy=True)
    K = C.shape[0]
    idx = np.empty(N, dtype=np.int32)
    d1 = np.empty(N, dtype=np.float64)
    counts = np.empty(K, dtype=np.int64)
    obj = np.empty(iters, dtype=np.float64)
    _load().oc_fit(_p(X), N, g, K, iters, _p(C), _p(idx), _p(d1), _p(counts), _p(obj))
    return C, idx, d1, counts, obj


def to_half(C: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> FP16 (the stored codebook)."""
    C = np.ascontiguousarray(C, dtype=np.float32)
    out = np.empty(C.shape, dtype=np.float16)
    _load().oc_float_to_half(_p(C), C.size, _p(out))
    return out


def half_to_double(a: np.ndarray) -> np.ndarray:
    a = _half(a)
    out = np.empty(a.shape, dtype=np.float64)
    _load().oc_half_to_double(_p(a), a.size, _p(out))
    return out


def finalize(X: np.ndarray, C: np.ndarray):
    """Stored codebook and codes: C16 = FP16(C); codes = E-step against C16.

    Returns (C16, idx, d1, objective)."""
    C16 = to_half(C)
    idx, d1, _ = assign(X, C16.astype(np.float32))
    return C16, idx, d1, float(np.sum(d1))


def linear_forward(x: np.ndarray, C16: np.ndarray, idx: np.ndarray, d_out: int, d_in: int,
                   bias: Optional[np.ndarray] = None) -> np.ndarray:
    """Forward of the compressed linear layer: y = x . codebook[code].view(in, -1)[:, :d_out] (+ bias).

    x: M x d_in FP16.  Returns M x d_out float64."""
    x = _half(x)
    C16 = _half(C16)
    M = x.shape[0]
    K, g = C16.shape
    assert x.shape[1] == d_in
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    assert idx.size == num_subvectors(d_out, d_in, g) and idx.min() >= 0 and idx.max() < K
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
        assert bias.shape == (d_out,)
    y = np.empty((M, d_out), dtype=np.float64)
    _load().oc_linear_forward(_p(x), M, _p(C16), g, _p(idx), d_out, d_in, _p(bias), _p(y))
    return y


def quantize_codebook(C16: np.ndarray, bits: int):
    """Uniform symmetric quantisation of the stored codebook to `bits` (8 or 4) bits.

    Returns (q int8 of C16's shape, scale float32, dequantised FP16 codebook)."""
    C16 = _half(C16)
    assert bits in (8, 4)
    q = np.empty(C16.shape, dtype=np.int8)
    scale = np.empty(1, dtype=np.float32)
    deq = np.empty(C16.shape, dtype=np.float16)
    _load().oc_quantize_codebook(_p(C16), C16.size, bits, _p(q), _p(scale), _p(deq))
    return q, float(scale[0]), deq


def pack_nibbles(q: np.ndarray) -> np.ndarray:
    """Storage format of a 4-bit codebook: element 2k in the low nibble of byte k, element 2k+1 in the
    high nibble (two's complement nibbles); an odd element count leaves the last high nibble 0."""
    flat = q.reshape(-1).astype(np.int16) & 0xF
    if flat.size % 2:
        flat = np.concatenate([flat, np.zeros(1, np.int16)])
    return (flat[0::2] | (flat[1::2] << 4)).astype(np.uint8)


def split_empty(C: np.ndarray, counts: np.ndarray) -> np.ndarray:
    """Second empty-cluster rule applied to the centroids of one M-step; returns the new centroids."""
    C = np.array(C, dtype=np.float32, order="C", copy=True)
    counts = np.ascontiguousarray(counts, dtype=np.int64)
    K, g = C.shape
    assert counts.shape == (K,)
    _load().oc_split_empty(_p(C), K, g, _p(counts))
    return C


EMPTY_KEEP, EMPTY_SPLIT = 0, 1


def fit_ex(X: np.ndarray, C0: np.ndarray, iters: int, empty_rule: int = EMPTY_KEEP):
    """Lloyd loop with a choice of empty-cluster rule, written with the one-step primitives.

    Returns (C, idx of the last E-step, d1, counts, objective[iters])."""
    C = np.array(C0, dtype=np.float32, order="C", copy=True)
    obj = np.empty(iters, dtype=np.float64)
    idx = d1 = counts = None
    for it in range(iters):
        idx, d1, _ = assign(X, C)
        obj[it] = float(np.sum(d1))
        C, counts = update(X, idx, C)
        if empty_rule == EMPTY_SPLIT:
            C = split_empty(C, counts)
    return C, idx, d1, counts, obj


def train_positions(N: int, K: int, max_points_per_centroid: int, seed: int) -> Optional[np.ndarray]:
    """Training-set subsampling: when N exceeds max_points_per_centroid * K, the Lloyd loop runs on
    that many points, drawn as distinct positions by the same seeded partial shuffle that draws the
    initial centroids; None when all points are used."""
    n = max_points_per_centroid * K
    if n >= N:
        return None
    return init_positions(N, n, seed)


def fit_sampled(X: np.ndarray, C0: np.ndarray, iters: int, max_points_per_centroid: int, seed: int):
    """Lloyd loop on the subsampled training set, then one E-step over ALL points against the fitted
    codebook.  Returns (C, idx over all points, d1 over all points, training counts, objective[iters])."""
    pos = train_positions(len(X), C0.shape[0], max_points_per_centroid, seed)
    Xt = X if pos is None else np.ascontiguousarray(X[pos])
    C, _, _, counts, obj = fit(Xt, C0, iters)
    idx, d1, _ = assign(X, C)
    return C, idx, d1, counts, obj

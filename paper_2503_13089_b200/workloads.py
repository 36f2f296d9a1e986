"""Seeded synthetic inputs: weight matrices, blobs and point subsets.

This module only *draws numbers*.  It holds none of the clustering method's
arithmetic (no distances, no means, no reshaping rule), so that the CUDA path
and the CPU oracle can both be fed the very same bytes without sharing any
code that could hide a common mistake.  It imports neither of them.

The matrices stand in for the Llama weight matrices the paper clusters
(Section 3.1 and the pilot study on heavy-tailed weights): same shapes,
FP16 storage, heavy-tailed entries with sparse large outliers.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

_CHUNK = 1 << 22  # elements drawn per call; part of the recipe (fixes the stream)


@dataclass(frozen=True)
class MatrixSpec:
    """One weight matrix of a workload (stored d_out x d_in, row-major FP16)."""
    name: str
    d_out: int
    d_in: int
    dist: str            # "normal" | "student_t3"
    scale: float
    outlier_frac: float  # fraction of entries overwritten by +-U(0.2, 1.0)
    data_seed: int
    init_seed: int


@dataclass(frozen=True)
class Workload:
    """A benchmark / parity configuration: matrices plus clustering settings."""
    name: str
    g: int
    K: int
    iters: int
    matrices: Tuple[MatrixSpec, ...]
    subset_frac: float = 1.0   # share of points the oracle checks per iteration
    notes: str = ""

    def n_subvectors(self, m: MatrixSpec) -> int:
        # out_features are padded up to a multiple of g (only the paper-grid workloads need it)
        return m.d_in * ((m.d_out + self.g - 1) // self.g)


def _layer7b(prefix_seed: int, init_seed: int) -> Tuple[MatrixSpec, ...]:
    shapes = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
              ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]
    return tuple(MatrixSpec(n, o, i, "student_t3", 0.02, 0.0, prefix_seed + k, init_seed + k)
                 for k, (n, o, i) in enumerate(shapes))


WORKLOADS = {
    # small correctness case: the oracle finishes a full fit in seconds
    "cfg1_256x512_g4_k256": Workload(
        "cfg1_256x512_g4_k256", 4, 256, 10,
        (MatrixSpec("w", 256, 512, "normal", 0.02, 0.001, 0, 2001),)),
    # a 7B attention-projection shape with a small codebook (3 bits per weight of index)
    "cfg2_4096x4096_g4_k4096": Workload(
        "cfg2_4096x4096_g4_k4096", 4, 4096, 20,
        (MatrixSpec("w", 4096, 4096, "student_t3", 0.02, 0.0, 1002, 2002),)),
    "cfg3_4096x11008_g8_k65536": Workload(
        "cfg3_4096x11008_g8_k65536", 8, 65536, 20,
        (MatrixSpec("w", 4096, 11008, "student_t3", 0.02, 0.0005, 1003, 2003),),
        subset_frac=0.01),
    "cfg4_8192x28672_g4_k65536": Workload(
        "cfg4_8192x28672_g4_k65536", 4, 65536, 10,
        (MatrixSpec("w", 8192, 28672, "student_t3", 0.015, 0.0, 1004, 2004),),
        subset_frac=0.01),
    "cfg5_layer7b_g16_k65536": Workload(
        "cfg5_layer7b_g16_k65536", 16, 65536, 15, _layer7b(1050, 2050),
        subset_frac=0.01),
    # the paper's own settings for a 4096 x 4096 matrix (bits table): odd g with real padding and
    # codebook sizes that are not powers of two
    "grid_g6_n65500": Workload(
        "grid_g6_n65500", 6, 65500, 20,
        (MatrixSpec("w", 4096, 4096, "student_t3", 0.02, 0.0, 1106, 2106),), subset_frac=0.01),
    "grid_g9_n65500": Workload(
        "grid_g9_n65500", 9, 65500, 20,
        (MatrixSpec("w", 4096, 4096, "student_t3", 0.02, 0.0, 1109, 2109),), subset_frac=0.01),
    "grid_g5_n50000": Workload(
        "grid_g5_n50000", 5, 50000, 20,
        (MatrixSpec("w", 4096, 4096, "student_t3", 0.02, 0.0, 1105, 2105),), subset_frac=0.01),
    "grid_g7_n35000": Workload(
        "grid_g7_n35000", 7, 35000, 20,
        (MatrixSpec("w", 4096, 4096, "student_t3", 0.02, 0.0, 1107, 2107),), subset_frac=0.01),
}


def make_matrix(spec: MatrixSpec) -> np.ndarray:
    """Draw the d_out x d_in FP16 matrix of `spec` (C-contiguous).

    Recipe: one PCG64 stream per matrix; entries are drawn in row-major order
    in calls of 2**22 elements, scaled in float64 and rounded to FP16
    (round-to-nearest-even, numpy's cast).  Outliers: round(frac * numel)
    distinct flat positions (choice without replacement from a second stream,
    seed + 7919), each overwritten by sign * U(0.2, 1.0).
    """
    rng = np.random.Generator(np.random.PCG64(spec.data_seed))
    numel = spec.d_out * spec.d_in
    out = np.empty(numel, dtype=np.float16)
    for lo in range(0, numel, _CHUNK):
        n = min(_CHUNK, numel - lo)
        if spec.dist == "normal":
            v = rng.standard_normal(n)
        elif spec.dist == "student_t3":
            v = rng.standard_t(3.0, n)
        else:
            raise ValueError(spec.dist)
        v *= spec.scale
        np.clip(v, -65504.0, 65504.0, out=v)
        out[lo:lo + n] = v.astype(np.float16)
    n_out = int(round(spec.outlier_frac * numel))
    if n_out > 0:
        rng2 = np.random.Generator(np.random.PCG64(spec.data_seed + 7919))
        pos = rng2.choice(numel, size=n_out, replace=False)
        mag = rng2.uniform(0.2, 1.0, size=n_out)
        sgn = np.where(rng2.random(n_out) < 0.5, -1.0, 1.0)
        out[pos] = (sgn * mag).astype(np.float16)
    return out.reshape(spec.d_out, spec.d_in)


def make_points(N: int, g: int, seed: int, dist: str = "student_t3", scale: float = 0.02) -> np.ndarray:
    """N x g FP16 points drawn directly (for per-call parity cases)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    v = rng.standard_t(3.0, (N, g)) if dist == "student_t3" else rng.standard_normal((N, g))
    return np.clip(v * scale, -65504, 65504).astype(np.float16)


def make_codebook(K: int, g: int, seed: int, scale: float = 0.02) -> np.ndarray:
    """K x g FP32 centroids with the same heavy-tailed law as the points."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return (rng.standard_t(3.0, (K, g)) * scale).astype(np.float32)


def make_blobs(n_blobs: int, per_blob: int, g: int, seed: int, sep: float = 1.0,
               sigma: float = 0.01) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Well-separated Gaussian blobs.

    Returns (points FP16 [n_blobs*per_blob, g] in shuffled order, labels int64,
    blob centres float64).  Centres sit on a lattice with spacing `sep`, far
    more than `sigma`, so the true partition is the only sensible one.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    side = int(np.ceil(n_blobs ** (1.0 / g)))
    grid = np.stack(np.meshgrid(*[np.arange(side)] * g, indexing="ij"), -1).reshape(-1, g)
    centres = grid[rng.permutation(len(grid))[:n_blobs]].astype(np.float64) * sep
    labels = np.repeat(np.arange(n_blobs), per_blob)
    pts = centres[labels] + rng.standard_normal((len(labels), g)) * sigma
    perm = rng.permutation(len(labels))
    return pts[perm].astype(np.float16), labels[perm], centres


def subset_positions(N: int, frac: float, seed: int) -> np.ndarray:
    """Sorted, distinct point positions: ceil(frac*N) of them (a seeded sample)."""
    n = int(np.ceil(frac * N))
    rng = np.random.Generator(np.random.PCG64(seed))
    return np.sort(rng.choice(N, size=n, replace=False)).astype(np.int64)

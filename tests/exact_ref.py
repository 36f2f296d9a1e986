"""Exact-rational k-means steps for tiny inputs (test helper, not the oracle).

FP16 and FP32 values are dyadic rationals, so distances and means can be
computed with `fractions.Fraction` without any rounding.  The oracle is pinned
against these, and against exhaustive enumeration of all labelings.
"""
from fractions import Fraction
from itertools import product

import numpy as np


def frac_rows(a):
    return [[Fraction(float(v)) for v in row] for row in np.asarray(a)]


def exact_dist(x, c):
    return sum((a - b) ** 2 for a, b in zip(x, c))


def exact_assign(X, C):
    """Lowest index among exact minimisers, with best / second-best distances."""
    Xf, Cf = frac_rows(X), frac_rows(C)
    idx, d1, d2 = [], [], []
    for x in Xf:
        ds = [exact_dist(x, c) for c in Cf]
        j = min(range(len(ds)), key=lambda k: (ds[k], k))
        rest = sorted(ds[:j] + ds[j + 1:])
        idx.append(j)
        d1.append(ds[j])
        d2.append(rest[0] if rest else None)
    return idx, d1, d2


def exact_means(X, idx, K):
    Xf = frac_rows(X)
    g = len(Xf[0])
    sums = [[Fraction(0)] * g for _ in range(K)]
    counts = [0] * K
    for x, j in zip(Xf, idx):
        counts[j] += 1
        sums[j] = [s + v for s, v in zip(sums[j], x)]
    means = [[s / counts[j] for s in sums[j]] if counts[j] else None for j in range(K)]
    return means, counts


def exact_objective_of_labeling(X, labels, K):
    """Sum of squared distances to the exact per-cluster means."""
    Xf = frac_rows(X)
    means, counts = exact_means(X, labels, K)
    return sum(exact_dist(x, means[j]) for x, j in zip(Xf, labels))


def global_optimum(X, K):
    """Minimum of the k-means objective over all K**N labelings (tiny N only)."""
    N = len(X)
    best = None
    for labels in product(range(K), repeat=N):
        J = exact_objective_of_labeling(X, labels, K)
        if best is None or J < best:
            best = J
    return best

"""Pins for the CPU oracle: things the paper and the mathematics fix.

Each test is chosen so that a plausible slip in the oracle (a dropped term, a
wrong sign or index, a transposed operand, an off-by-one in padding) fails it.
None of them touches the CUDA library.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2503_13089_b200 import workloads as wl
from tests import exact_ref as ex

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------- sizes, Eq. 1

def test_bits_table_printed_values():
    for row in _golden_lines("bits_per_param_table.txt"):
        if row[0] == "example":
            g, n = int(row[1]), int(row[2])
            assert abs(16.0 / g - float(row[3])) < 1e-12
            assert round(16.0 * g * n / 4096 ** 2, 2) == float(row[4])
            assert round(oracle.bits_per_param(4096, 4096, g, n), 2) == float(row[5])
        elif row[0] == "layer7b":
            g, n = int(row[1]), int(row[2])
            shapes = [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]
            bits = sum(oracle.bits_per_param(o, i, g, n) * o * i for o, i in shapes)
            assert round(bits / sum(o * i for o, i in shapes), 2) == float(row[3])
        else:
            g, n = int(row[0]), int(row[1])
            # the table counts k = d_in*d_out/g codes (Section 3.1), i.e. before padding: for
            # g = 9 that is 1.864M -> "1.86M", while the listing stores 1,867,776 padded codes
            assert round(4096 * 4096 / g / 1e6, 2) == float(row[2])
            codes = oracle.num_subvectors(4096, 4096, g)
            assert 0 <= codes - 4096 * 4096 / g < 4096
            assert round(g * n / 1e6, 2) == float(row[3])
            # the printed percentage is the rounded codebook size over the caption's 16.78M
            assert round(100.0 * float(row[3]) / 16.78, 2) == float(row[4])
            assert round(oracle.bits_per_param(4096, 4096, g, n), 2) == float(row[5])


def test_num_subvectors_padding_rule():
    # the listing: deficiency = g - out % g when out % g > 0; codes = in*(out+deficiency)/g
    assert oracle.num_subvectors(4096, 4096, 6) == 4096 * 4098 // 6 == 2797568
    assert oracle.num_subvectors(4096, 4096, 9) == 4096 * 4104 // 9 == 1867776
    assert oracle.num_subvectors(10, 7, 4) == 7 * 3            # pads out_features 10 -> 12
    assert oracle.num_subvectors(10, 7, 4, oracle.LAYOUT_ROWS) == 10 * 2   # pads in_features 7 -> 8


# ---------------------------------------------------------------- FP16 conversions

def test_half_to_double_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    h = bits.view(np.float16)
    got = oracle.half_to_double(h)
    want = h.astype(np.float64)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok])
    assert np.array_equal(np.signbit(got[ok]), np.signbit(want[ok]))


def test_float_to_half_matches_numpy_rne():
    rng = np.random.default_rng(5)
    f = np.concatenate([
        (rng.standard_normal(200000) * 10.0 ** rng.integers(-9, 6, 200000)).astype(np.float32),
        np.array([0.0, -0.0, 65504.0, 65519.99, 65520.0, 65536.0, 1e9, -1e9, np.inf, -np.inf,
                  2.0 ** -24, 2.0 ** -25, 1.5 * 2.0 ** -25, 2.0 ** -14, 2.0 ** -14 - 2.0 ** -26],
                 dtype=np.float32)])
    # exact midpoints between neighbouring halves: the ties-to-even cases
    h = np.arange(0, 0x7bff, 7, dtype=np.uint16).view(np.float16).astype(np.float64)
    h2 = np.arange(1, 0x7c00, 7, dtype=np.uint16).view(np.float16).astype(np.float64)
    mid = ((h + h2) / 2).astype(np.float32)
    f = np.concatenate([f, mid, -mid])
    with np.errstate(over="ignore"):
        want = f.astype(np.float16)
    got = oracle.to_half(f)
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))


# ---------------------------------------------------------------- reshape / decode

@pytest.mark.parametrize("d_out,d_in,g", [(8, 6, 4), (10, 7, 4), (9, 5, 3), (16, 16, 8), (7, 3, 5)])
def test_reshape_is_transpose_pad_view(d_out, d_in, g):
    rng = np.random.default_rng(d_out * 100 + d_in)
    W = rng.standard_normal((d_out, d_in)).astype(np.float16)
    # Section 3.1 footnote: W' = W.transpose(1, 0).view(-1, g) after zero-padding (the listing
    # pads out_features)
    pad = (-d_out) % g
    want = np.concatenate([W.T, np.zeros((d_in, pad), np.float16)], axis=1).reshape(-1, g)
    got = oracle.reshape_subvectors(W, g)
    assert got.shape == want.shape and np.array_equal(got, want)
    pad_r = (-d_in) % g
    want_r = np.concatenate([W, np.zeros((d_out, pad_r), np.float16)], axis=1).reshape(-1, g)
    assert np.array_equal(oracle.reshape_subvectors(W, g, oracle.LAYOUT_ROWS), want_r)


@pytest.mark.parametrize("layout", [oracle.LAYOUT_PAPER_T, oracle.LAYOUT_ROWS])
@pytest.mark.parametrize("d_out,d_in,g", [(10, 7, 4), (12, 8, 4), (9, 5, 3)])
def test_decode_inverts_reshape_when_every_point_is_a_centroid(d_out, d_in, g, layout):
    rng = np.random.default_rng(3)
    W = rng.standard_normal((d_out, d_in)).astype(np.float16)
    X = oracle.reshape_subvectors(W, g, layout)
    perm = rng.permutation(len(X))
    C16 = X[perm]                                   # codebook = the points, shuffled
    idx = np.argsort(perm).astype(np.int32)         # code of point i = where it went
    assert np.array_equal(oracle.decode(C16, idx, d_out, d_in, layout), W)


def test_decode_matches_listing_semantics():
    # codebook[code].view(in_features, -1)[:, :-deficiency], used as x @ weight
    rng = np.random.default_rng(11)
    d_out, d_in, g, K = 10, 6, 4, 17
    C16 = rng.standard_normal((K, g)).astype(np.float16)
    idx = rng.integers(0, K, oracle.num_subvectors(d_out, d_in, g)).astype(np.int32)
    weight = C16[idx].reshape(d_in, -1)[:, :d_out]          # (in, out)
    assert np.array_equal(oracle.decode(C16, idx, d_out, d_in), weight.T)


# ---------------------------------------------------------------- initialisation

def test_init_positions_follow_published_generator_vector():
    outs = [int(r[0]) for r in _golden_lines("splitmix64_seed1234567.txt")]
    N, K = 1000003, 5
    a = {}
    want = []
    for i in range(K):                      # partial Fisher-Yates driven by the published outputs
        j = i + outs[i] % (N - i)
        ai, aj = a.get(i, i), a.get(j, j)
        a[i], a[j] = aj, ai
        want.append(a[i])
    assert oracle.init_positions(N, K, 1234567).tolist() == want


def test_init_positions_distinct_and_full_permutation():
    pos = oracle.init_positions(5000, 700, 42)
    assert len(set(pos.tolist())) == 700 and pos.min() >= 0 and pos.max() < 5000
    full = oracle.init_positions(257, 257, 9)
    assert sorted(full.tolist()) == list(range(257))
    assert not np.array_equal(oracle.init_positions(5000, 700, 43), pos)
    X = wl.make_points(5000, 4, 1)
    assert np.array_equal(oracle.init_codebook(X, 700, 42), X[pos].astype(np.float32))


# ---------------------------------------------------------------- E-step

@pytest.mark.parametrize("g,N,K,seed", [(1, 40, 5, 0), (3, 60, 7, 1), (4, 80, 16, 2), (8, 50, 9, 3)])
def test_assign_against_exact_rationals(g, N, K, seed):
    X = wl.make_points(N, g, seed)
    C = wl.make_codebook(K, g, seed + 100)
    C[K // 2] = C[1]                                   # a duplicated centroid: lowest index must win
    X[3] = C[1].astype(np.float16)
    idx, d1, d2 = oracle.assign(X, C)
    eidx, ed1, ed2 = ex.exact_assign(X, C)
    assert idx.tolist() == eidx
    assert np.allclose(d1, [float(v) for v in ed1], rtol=1e-13, atol=0)
    assert np.allclose(d2, [float(v) for v in ed2], rtol=1e-13, atol=0)
    assert np.all(idx != K // 2)


def test_assign_exact_tie_takes_lowest_index_and_reports_zero_gap():
    X = np.array([[0.0, 0.0]], dtype=np.float16)
    C = np.array([[1, 0], [0, 1], [-1, 0], [0.5, 0.5]], dtype=np.float32)
    idx, d1, d2 = oracle.assign(X, C)
    assert idx[0] == 3 and d1[0] == 0.5 and d2[0] == 1.0
    idx, d1, d2 = oracle.assign(X, C[:3])
    assert idx[0] == 0 and d1[0] == 1.0 and d2[0] == 1.0


def test_assign_matches_scipy_vq():
    from scipy.cluster.vq import vq
    X = wl.make_points(3000, 4, 7)
    C = wl.make_codebook(64, 4, 8)
    idx, d1, _ = oracle.assign(X, C)
    code, dist = vq(X.astype(np.float64), C.astype(np.float64))
    assert np.array_equal(idx, code)
    assert np.allclose(np.sqrt(d1), dist, rtol=1e-12)


def test_assign_special_cases_and_metamorphic():
    X = wl.make_points(500, 4, 21)
    C = wl.make_codebook(33, 4, 22)
    idx, d1, d2 = oracle.assign(X, C)
    assert np.all(oracle.assign(X, C[:1])[0] == 0)                       # K = 1
    own = oracle.assign(X[:200], X[:200].astype(np.float32))             # centroids = the points
    first = [np.flatnonzero((X[:200] == X[i]).all(1))[0] for i in range(200)]
    assert own[0].tolist() == first and np.all(own[1] == 0)
    # scaling by a power of two changes no index and scales distances by its square
    Xs = (X.astype(np.float32) * 4).astype(np.float16)
    idx_s, d1_s, _ = oracle.assign(Xs, C * 4)
    assert np.array_equal(idx_s, idx) and np.array_equal(d1_s, d1 * 16)
    # permuting the centroids permutes the indices
    perm = np.random.default_rng(0).permutation(33)
    idx_p, d1_p, d2_p = oracle.assign(X, C[perm])
    assert np.array_equal(perm[idx_p], idx) and np.array_equal(d1_p, d1) and np.array_equal(d2_p, d2)
    # subset selection returns the same rows
    sel = np.array([499, 0, 17, 17, 250])
    s = oracle.assign(X, C, sel)
    assert np.array_equal(s[0], idx[sel]) and np.array_equal(s[1], d1[sel])
    assert oracle.point_dist(X, 17, C, int(idx[17])) == d1[17]


# ---------------------------------------------------------------- M-step

def test_update_against_exact_means_and_empty_rule():
    X = wl.make_points(90, 4, 31)
    K = 8
    rng = np.random.default_rng(0)
    idx = rng.integers(0, K - 2, 90).astype(np.int32)        # clusters K-2, K-1 stay empty
    C_prev = wl.make_codebook(K, 4, 32)
    C, counts = oracle.update(X, idx, C_prev)
    means, ecounts = ex.exact_means(X, idx.tolist(), K)
    assert counts.tolist() == ecounts and counts.sum() == 90
    assert np.array_equal(counts, np.bincount(idx, minlength=K))
    for j in range(K):
        if ecounts[j]:
            want = np.array([float(v) for v in means[j]]).astype(np.float32)
            assert np.array_equal(C[j], want)
        else:
            assert np.array_equal(C[j].view(np.uint32), C_prev[j].view(np.uint32))
    # order of the points does not matter (sums of FP16 values are exact in double here)
    p = rng.permutation(90)
    C2, counts2 = oracle.update(X[p], idx[p], C_prev)
    assert np.array_equal(C2, C) and np.array_equal(counts2, counts)


def test_k1_closed_form_mean_and_variance():
    X = wl.make_points(4000, 3, 33)
    Xd = X.astype(np.float64)
    C0 = np.zeros((1, 3), np.float32)
    C, idx, d1, counts, obj = oracle.fit(X, C0, 2)
    assert counts[0] == 4000 and np.all(idx == 0)
    assert np.array_equal(C[0], Xd.mean(0).astype(np.float32))
    assert obj[0] == pytest.approx((Xd ** 2).sum(), rel=1e-12)         # distances to the origin
    mean32 = Xd.mean(0).astype(np.float32).astype(np.float64)
    assert obj[1] == pytest.approx(((Xd - mean32) ** 2).sum(), rel=1e-12)
    assert obj[1] == pytest.approx(4000 * Xd.var(0).sum(), rel=1e-6)   # N * total variance


# ---------------------------------------------------------------- Lloyd loop

def test_objective_never_increases():
    for seed, (N, g, K) in enumerate([(3000, 4, 50), (2000, 8, 300), (1500, 2, 17)]):
        X = wl.make_points(N, g, 40 + seed)
        C0 = oracle.init_codebook(X, K, 50 + seed)
        _, _, _, _, obj = oracle.fit(X, C0, 12)
        assert np.all(np.diff(obj) <= 1e-6 * obj[:-1]), obj
        assert obj[-1] < obj[0]


def test_lloyd_versus_brute_force_over_all_labelings():
    hits = 0
    for seed in range(6):
        N, K, g = 8, 3, 2
        X = wl.make_points(N, g, 60 + seed, dist="normal", scale=1.0)
        opt = ex.global_optimum(X, K)
        best_seen = None
        for init_seed in range(8):
            C0 = oracle.init_codebook(X, K, init_seed)
            C, idx, d1, counts, obj = oracle.fit(X, C0, 20)
            # fixed point: one more E-step changes nothing; centroids are the exact means
            idx2, d1b, _ = oracle.assign(X, C)
            assert np.array_equal(idx2, idx)
            means, cnt = ex.exact_means(X, idx.tolist(), K)
            for j in range(K):
                if cnt[j]:
                    assert np.array_equal(C[j], np.array([float(v) for v in means[j]], np.float32))
            J = ex.exact_objective_of_labeling(X, idx.tolist(), K)
            assert J >= opt                                    # Lloyd never beats the optimum
            assert float(J) == pytest.approx(d1b.sum(), rel=1e-5)
            best_seen = J if best_seen is None else min(best_seen, J)
        hits += best_seen == opt
    assert hits >= 4          # over eight starts Lloyd reaches the certified optimum most times


def test_one_dimensional_optimum_by_dynamic_programming():
    # g = 1: optimal clusters are contiguous runs of the sorted points (textbook DP)
    X = wl.make_points(14, 1, 70, dist="normal", scale=1.0)
    xs = sorted(Fraction(float(v)) for v in X[:, 0])
    K, n = 3, len(xs)

    def cost(a, b):                         # points a..b-1 as one cluster
        seg = xs[a:b]
        m = sum(seg) / len(seg)
        return sum((v - m) ** 2 for v in seg)

    INF = Fraction(10 ** 9)
    dp = [[INF] * (n + 1) for _ in range(K + 1)]
    dp[0][0] = Fraction(0)
    for k in range(1, K + 1):
        for b in range(k, n + 1):
            dp[k][b] = min(dp[k - 1][a] + cost(a, b) for a in range(k - 1, b))
    opt = dp[K][n]
    best = min(ex.exact_objective_of_labeling(X, oracle.fit(X, oracle.init_codebook(X, K, s), 25)[1].tolist(), K)
               for s in range(12))
    assert best >= opt and best == opt


def test_k_equals_n_gives_zero_error():
    X = np.unique(wl.make_points(300, 4, 80), axis=0)
    N = len(X)
    C0 = oracle.init_codebook(X, N, 5)
    C, idx, d1, counts, obj = oracle.fit(X, C0, 3)
    assert np.all(obj == 0) and np.all(counts == 1)
    assert np.array_equal(C[idx], X.astype(np.float32))


def test_separated_blobs_are_recovered():
    X, labels, centres = wl.make_blobs(12, 40, 3, seed=90, sep=1.0, sigma=0.01)
    # one starting centroid per blob (a member of it)
    first = np.array([np.flatnonzero(labels == b)[0] for b in range(12)])
    C, idx, d1, counts, obj = oracle.fit(X, X[first].astype(np.float32), 5)
    assert np.array_equal(idx, labels) and np.all(counts == 40)
    Xd = X.astype(np.float64)
    for b in range(12):
        assert np.array_equal(C[b], Xd[labels == b].mean(0).astype(np.float32))
        assert np.allclose(C[b], centres[b], atol=0.01)
    # seeded starts: whenever the start has one point per blob the partition is exact
    X, labels, centres = wl.make_blobs(3, 50, 2, seed=91, sep=1.0, sigma=0.01)
    ok = 0
    for seed in range(40):
        pos = oracle.init_positions(len(X), 3, seed)
        if len(set(labels[pos].tolist())) == 3:
            _, idx_s, _, counts_s, _ = oracle.fit(X, X[pos].astype(np.float32), 4)
            assert np.array_equal(labels[pos][idx_s], labels) and np.all(counts_s == 50)
            ok += 1
    assert ok >= 3


def test_fit_matches_scipy_kmeans2_with_given_start():
    from scipy.cluster.vq import kmeans2
    X = wl.make_points(2500, 4, 95, dist="normal", scale=1.0)
    C0 = oracle.init_codebook(X, 12, 96)
    C, idx, d1, counts, obj = oracle.fit(X, C0, 6)
    C_sp, lab_sp = kmeans2(X.astype(np.float64), C0.astype(np.float64), iter=6, minit="matrix",
                           missing="raise")
    # scipy returns labels against the centroids before its last update
    assert np.mean(lab_sp == idx) > 0.999
    assert np.allclose(C, C_sp, rtol=0, atol=2e-3 * np.abs(C_sp).max())


def test_decode_error_equals_objective():
    spec = wl.WORKLOADS["cfg1_256x512_g4_k256"].matrices[0]
    W = wl.make_matrix(spec)[:64, :96]
    W = np.ascontiguousarray(W)
    for layout in (oracle.LAYOUT_PAPER_T, oracle.LAYOUT_ROWS):
        X = oracle.reshape_subvectors(W, 4, layout)
        C0 = oracle.init_codebook(X, 32, 1)
        C = oracle.fit(X, C0, 5)[0]
        C16, idx, d1, J = oracle.finalize(X, C)
        W_hat = oracle.decode(C16, idx, 64, 96, layout)
        err = ((W.astype(np.float64) - W_hat.astype(np.float64)) ** 2).sum()
        assert err == pytest.approx(J, rel=1e-12)


def test_workload_generators_are_seeded_and_shaped():
    spec = wl.WORKLOADS["cfg1_256x512_g4_k256"].matrices[0]
    W1, W2 = wl.make_matrix(spec), wl.make_matrix(spec)
    assert W1.shape == (256, 512) and W1.dtype == np.float16 and np.array_equal(W1, W2)
    big = np.abs(W1.astype(np.float32)) >= 0.19
    assert 100 <= big.sum() <= 140          # 0.1 % of 131072 entries are outliers
    assert np.isfinite(W1.astype(np.float32)).all()
    sel = wl.subset_positions(1000, 0.01, 3)
    assert len(sel) == 10 and len(set(sel.tolist())) == 10


# ------------------------------------------------------------------ codebook gradient

def test_codebook_grad_against_exact_rationals_autograd_and_the_m_step():
    """dC[j] = sum of dX[i] over idx[i] = j: exact rational sums on a small case, torch autograd
    of the gather codebook[code] in float64, linearity in dX, and counts x mean of the M-step."""
    from fractions import Fraction
    import torch
    rng = np.random.default_rng(17)
    N, g, K = 300, 5, 11
    dX = (rng.standard_normal((N, g)) * rng.choice([1e-3, 1.0, 300.0], (N, 1))).astype(np.float16)
    idx = rng.integers(0, K - 2, N).astype(np.int32)              # two clusters get no gradient
    got = oracle.codebook_grad(dX, idx, K)
    want = np.zeros((K, g), dtype=np.float32)
    for j in range(K):
        for t in range(g):
            sacc = sum((Fraction(float(v)) for v in dX[idx == j, t]), Fraction(0))
            want[j, t] = np.float32(float(sacc))                  # Fraction -> double -> float: sums fit a double here
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert np.all(got[K - 2:] == 0)
    # autograd of the gather: loss = sum(codebook[code] * dX) has gradient index_add(dX)
    Cb = torch.zeros((K, g), dtype=torch.float64, requires_grad=True)
    (Cb[torch.from_numpy(idx.astype(np.int64))] * torch.from_numpy(dX.astype(np.float64))).sum().backward()
    assert np.array_equal(got, Cb.grad.numpy().astype(np.float32))
    # linearity where the sum of the two gradients is itself FP16-exact
    a = (rng.integers(-8, 9, (N, g)) * 0.25).astype(np.float16)
    b = (rng.integers(-8, 9, (N, g)) * 0.5).astype(np.float16)
    assert np.array_equal(oracle.codebook_grad((a + b).astype(np.float16), idx, K),
                          oracle.codebook_grad(a, idx, K) + oracle.codebook_grad(b, idx, K))
    # the M-step's mean times its count is the same sum (values chosen so that every step is exact)
    C_new, counts = oracle.update(a, idx, np.zeros((K, g), np.float32))
    nz = counts > 0
    assert np.allclose(oracle.codebook_grad(a, idx, K)[nz], C_new[nz] * counts[nz, None], rtol=1e-6, atol=0)
    # K = 1: the column sums
    assert np.array_equal(oracle.codebook_grad(a, np.zeros(N, np.int32), 1)[0],
                          a.astype(np.float64).sum(0).astype(np.float32))


# ---------------------------------------------------------------- compressed linear layer (appendix listing)

def _layer_case(M, d_out, d_in, g, K, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, d_in)).astype(np.float16)
    C16 = (rng.standard_normal((K, g)) * 0.1).astype(np.float16)
    idx = rng.integers(0, K, oracle.num_subvectors(d_out, d_in, g)).astype(np.int32)
    return x, C16, idx


@pytest.mark.parametrize("M,d_out,d_in,g,K", [(3, 8, 5, 4, 7), (2, 10, 7, 4, 9), (5, 9, 16, 6, 33), (1, 64, 48, 16, 5),
                                               (4, 7, 3, 9, 4)])
def test_linear_forward_is_the_listing(M, d_out, d_in, g, K):
    """codebook[code].view(in_features, -1) with the padded columns dropped, then x @ weight + bias:
    written here with numpy indexing and a library matmul in float64."""
    x, C16, idx = _layer_case(M, d_out, d_in, g, K, M + d_out + d_in)
    bias = np.random.default_rng(1).standard_normal(d_out).astype(np.float32)
    weight = C16[idx].reshape(d_in, -1)[:, :d_out].astype(np.float64)
    want = x.astype(np.float64) @ weight
    assert np.allclose(oracle.linear_forward(x, C16, idx, d_out, d_in), want, rtol=1e-13, atol=1e-13)
    assert np.allclose(oracle.linear_forward(x, C16, idx, d_out, d_in, bias), want + bias.astype(np.float64),
                       rtol=1e-13, atol=1e-13)
    # the same weight is what decode lays out as a (d_out, d_in) matrix
    W_hat = oracle.decode(C16, idx, d_out, d_in).astype(np.float64)
    assert np.allclose(oracle.linear_forward(x, C16, idx, d_out, d_in), x.astype(np.float64) @ W_hat.T,
                       rtol=1e-13, atol=1e-13)


def test_linear_forward_exact_rationals_and_unit_inputs():
    x, C16, idx = _layer_case(2, 6, 5, 4, 5, 3)
    d_out, d_in, g = 6, 5, 4
    got = oracle.linear_forward(x, C16, idx, d_out, d_in)
    out_pad = 8
    for m in range(2):
        for o in range(d_out):
            s = Fraction(0)
            for i in range(d_in):
                flat = i * out_pad + o
                s += Fraction(float(x[m, i])) * Fraction(float(C16[idx[flat // g], flat % g]))
            assert got[m, o] == pytest.approx(float(s), rel=1e-14, abs=1e-300)
    # unit vectors as inputs read the weight's rows: row i of the (in, out) weight = column i of decode
    eye = np.eye(d_in, dtype=np.float16)
    assert np.array_equal(oracle.linear_forward(eye, C16, idx, d_out, d_in),
                          oracle.decode(C16, idx, d_out, d_in).astype(np.float64).T)
    # zero input leaves the bias
    b = np.arange(d_out, dtype=np.float32)
    assert np.array_equal(oracle.linear_forward(np.zeros((1, d_in), np.float16), C16, idx, d_out, d_in, b)[0], b)


# ---------------------------------------------------------------- uniform codebook quantisation (Section 5.3)

@pytest.mark.parametrize("bits", [8, 4])
def test_quantize_codebook_grid_range_and_error_bound(bits):
    rng = np.random.default_rng(bits)
    C16 = (rng.standard_t(3.0, (500, 6)) * 0.02).astype(np.float16)
    q, s, deq = oracle.quantize_codebook(C16, bits)
    L = 2 ** (bits - 1) - 1
    c = C16.astype(np.float64)
    assert s == np.float32(np.float32(np.abs(c).max()) / np.float32(L))
    assert q.max() == L or q.min() == -L                       # the largest magnitude sits on the last level
    assert q.min() >= -L and q.max() <= L                      # -2^(b-1) is never needed on a symmetric grid
    assert np.all(np.abs(c - q.astype(np.float64) * s) <= 0.5 * s * (1 + 1e-6))   # round to NEAREST
    assert len(np.unique(q)) <= 2 ** bits
    q2, s2, _ = oracle.quantize_codebook((-C16).astype(np.float16), bits)
    assert s2 == s and np.array_equal(q2, -q)                  # symmetric grid, ties to even
    assert np.allclose(deq.astype(np.float64), q * np.float64(s), rtol=2.0 ** -11, atol=2.0 ** -25)


def test_quantize_codebook_worked_examples():
    # values that already sit on a power-of-two grid come back as themselves
    C16 = np.array([[-1.75, 0.0, 0.25, 1.5], [1.75, -0.5, 0.75, -1.25]], dtype=np.float16)   # max 1.75 = 7 * 0.25
    q, s, deq = oracle.quantize_codebook(C16, 4)
    assert s == 0.25 and np.array_equal(q, (C16.astype(np.float64) / 0.25).astype(np.int8))
    assert np.array_equal(deq, C16)
    # exact halves round to the even level: with s = 1/4, 0.125 -> 0.5 -> 0, 0.375 -> 1.5 -> 2, 0.625 -> 2.5 -> 2
    C16 = np.array([[1.75, 0.125, 0.375, 0.625, -0.125, -0.375]], dtype=np.float16)
    q, s, _ = oracle.quantize_codebook(C16, 4)
    assert s == 0.25 and q.tolist() == [[7, 0, 2, 2, 0, -2]]
    # 8 bits: 127 levels each side
    C16 = np.array([[127.0, -64.0, 0.5, 1.5, 2.5, -126.6]], dtype=np.float16)
    q, s, _ = oracle.quantize_codebook(C16, 8)
    assert s == 1.0 and q.tolist() == [[127, -64, 0, 2, 2, -127]]      # FP16(-126.6) = -126.625
    # an all-zero codebook
    q, s, deq = oracle.quantize_codebook(np.zeros((3, 4), np.float16), 8)
    assert s == 1.0 and not q.any() and not deq.any()
    # nibble packing: low nibble first, two's complement
    assert oracle.pack_nibbles(np.array([7, -7, 0, -1, 3], np.int8)).tolist() == [0x97, 0xF0, 0x03]


# ---------------------------------------------------------------- second empty-cluster rule

def test_split_empty_worked_example():
    """K = 4, g = 2, counts (5, 0, 3, 0): cluster 1 takes half of cluster 0; then the working counts are
    (3, 2, 3, 0), clusters 0 and 2 tie and the lower index donates again.  Centroid 0 = (1024, 2048) so
    that every product with 1 +- 2^-10 is exact."""
    C = np.array([[1024.0, 2048.0], [5.0, 5.0], [-3.0, 7.0], [9.0, 9.0]], dtype=np.float32)
    out = oracle.split_empty(C, np.array([5, 0, 3, 0]))
    assert out[1].tolist() == [1025.0, 2046.0]
    assert out[3].tolist() == [1023.0 + 1023.0 / 1024.0, 2050.0 - 2050.0 / 1024.0]
    assert out[0].tolist() == [1023.0 - 1023.0 / 1024.0, 2050.0 + 2050.0 / 1024.0]
    assert out[2].tolist() == [-3.0, 7.0]
    # nobody can donate: every cluster has at most one point
    C2 = np.arange(8, dtype=np.float32).reshape(4, 2)
    assert np.array_equal(oracle.split_empty(C2, np.array([1, 0, 1, 0])), C2)
    # no empty cluster: nothing moves
    assert np.array_equal(oracle.split_empty(C2, np.array([4, 2, 1, 9])), C2)


def test_split_rule_fills_empty_clusters_and_lowers_the_objective():
    X, labels, centres = wl.make_blobs(6, 200, 4, seed=4, sep=1.0, sigma=0.02)
    first = np.array([np.flatnonzero(labels == b)[0] for b in range(6)])
    C0 = X[first].astype(np.float32)
    C0[5] = 50.0                                        # one start far from every point: its cluster stays empty
    C_keep, idx_k, _, counts_k, obj_k = oracle.fit_ex(X, C0, 6, oracle.EMPTY_KEEP)
    C_ref, idx_r, _, counts_r, obj_r = oracle.fit(X, C0, 6)
    assert np.array_equal(C_keep, C_ref) and np.allclose(obj_k, obj_r, rtol=1e-13)   # rule 0 is the plain loop
    assert counts_k[5] == 0 and np.array_equal(C_keep[5], C0[5])
    C_split, idx_s, _, counts_s, obj_s = oracle.fit_ex(X, C0, 6, oracle.EMPTY_SPLIT)
    assert counts_s.min() > 0 and counts_s.sum() == len(X)
    assert obj_s[-1] < obj_k[-1]


# ---------------------------------------------------------------- training-set subsampling

def test_fit_sampled_reduces_to_the_plain_loop_and_uses_the_drawn_rows():
    X = wl.make_points(3000, 4, 21)
    C0 = oracle.init_codebook(X, 10, 3)
    # enough room for every point: the plain loop followed by one E-step
    C, idx, d1, counts, obj = oracle.fit_sampled(X, C0, 3, 300, 9)
    C_ref, _, _, counts_ref, obj_ref = oracle.fit(X, C0, 3)
    assert np.array_equal(C, C_ref) and np.array_equal(obj, obj_ref) and np.array_equal(counts, counts_ref)
    assert np.array_equal(idx, oracle.assign(X, C_ref)[0])
    # 50 points per centroid: 500 distinct seeded positions are the training set
    pos = oracle.train_positions(3000, 10, 50, 9)
    assert len(pos) == 500 and len(set(pos.tolist())) == 500 and np.array_equal(pos, oracle.init_positions(3000, 500, 9))
    C, idx, d1, counts, obj = oracle.fit_sampled(X, C0, 3, 50, 9)
    C_t, _, _, counts_t, obj_t = oracle.fit(np.ascontiguousarray(X[pos]), C0, 3)
    assert np.array_equal(C, C_t) and counts.sum() == 500 and np.array_equal(obj, obj_t)
    assert len(idx) == 3000 and np.array_equal(idx, oracle.assign(X, C)[0])
    assert oracle.train_positions(3000, 10, 300, 9) is None

"""GPU parity: the CUDA library against the CPU oracle, element by element, through the C ABI.

Bars: indices / counts bit-exact (a differing index is tolerated only where the oracle's two
distances differ by < 1e-6 relative, and is counted); centroids within 1e-4 relative max error;
objective within 1e-5 relative.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_13089_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _cc():
    from paper_2503_13089_b200 import binding
    return binding


def _u():
    from tests import gpu_util
    return gpu_util


# ------------------------------------------------------------------ reshape / decode / init

@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("d_out,d_in,g", [(8, 8, 4), (10, 7, 4), (130, 67, 4), (129, 200, 6), (64, 64, 16),
                                          (100, 33, 9), (257, 300, 5), (1, 1, 1), (136, 200, 4), (200, 72, 8),
                                          (144, 328, 16), (130, 72, 4), (250, 136, 8), (512, 256, 4)])
def test_reshape_and_decode_match_oracle(d_out, d_in, g, layout):
    cc, u = _cc(), _u()
    rng = np.random.default_rng(d_out + d_in + g)
    W = rng.standard_normal((d_out, d_in)).astype(np.float16)
    N = cc.cc_num_subvectors(d_out, d_in, g, layout)
    assert N == oracle.num_subvectors(d_out, d_in, g, layout)
    Wd = u.half_dev(W)
    X = torch.full((N, g), 7.0, dtype=torch.float16, device="cuda")
    cc.cc_reshape_subvectors(u.ctx(), Wd, d_out, d_in, g, layout, X)
    Xo = oracle.reshape_subvectors(W, g, layout)
    assert np.array_equal(u.u16_np(X.view(torch.uint16)).reshape(N, g), Xo.view(np.uint16))
    K = 37
    C16 = rng.standard_normal((K, g)).astype(np.float16)
    idx = rng.integers(0, K, N).astype(np.uint16)
    What = torch.zeros((d_out, d_in), dtype=torch.float16, device="cuda")
    cc.cc_decode(u.ctx(), u.half_dev(C16), K, g, u.dev(idx.view(np.int16)).view(torch.uint16), d_out, d_in,
                 layout, What)
    want = oracle.decode(C16, idx.astype(np.int32), d_out, d_in, layout)
    assert np.array_equal(u.u16_np(What.view(torch.uint16)).reshape(d_out, d_in), want.view(np.uint16))


def test_decode_accepts_codes_that_are_only_two_byte_aligned():
    """The vector kernels read two codes as one 32-bit word; a code array that starts at an odd
    element must take the scalar kernel instead of faulting."""
    cc, u = _cc(), _u()
    d_out, d_in, g, K = 136, 200, 4, 50
    rng = np.random.default_rng(5)
    N = cc.cc_num_subvectors(d_out, d_in, g, 0)
    C16 = rng.standard_normal((K, g)).astype(np.float16)
    idx = rng.integers(0, K, N).astype(np.uint16)
    buf = torch.zeros(N + 1, dtype=torch.int16, device="cuda")
    buf[1:] = u.dev(idx.view(np.int16))
    What = torch.zeros((d_out, d_in), dtype=torch.float16, device="cuda")
    cc.cc_decode(u.ctx(), u.half_dev(C16), K, g, buf[1:].view(torch.uint16), d_out, d_in, 0, What)
    want = oracle.decode(C16, idx.astype(np.int32), d_out, d_in, 0)
    assert np.array_equal(u.u16_np(What.view(torch.uint16)).reshape(d_out, d_in), want.view(np.uint16))


@pytest.mark.parametrize("g,K", [(4, 3000), (8, 2900), (16, 1400), (4, 1), (8, 6400), (16, 3000), (4, 65536),
                                 (8, 65536), (4, 40000), (8, 20001), (8, 9000), (16, 65536), (4, 16385)])
def test_decode_of_a_large_matrix_matches_oracle(g, K):
    """Matrices with at least 8 tiles per SM: g = 8 and 16 with a codebook of at most 128 KB take the
    persistent kernel (codebooks of at most 46 KB staged in shared memory), the others -- among them
    codebooks of 320 KB, 512 KB, 1 MB and 2 MB -- the plain tiled kernel.  Ragged tiles on both edges."""
    cc, u = _cc(), _u()
    d_out, d_in = 2056, 2568
    rng = np.random.default_rng(g * 100003 + K)
    N = cc.cc_num_subvectors(d_out, d_in, g, 0)
    C16 = rng.standard_normal((K, g)).astype(np.float16)
    idx = rng.integers(0, K, N).astype(np.uint16)
    What = torch.zeros((d_out, d_in), dtype=torch.float16, device="cuda")
    cc.cc_decode(u.ctx(), u.half_dev(C16), K, g, u.dev(idx.view(np.int16)).view(torch.uint16), d_out, d_in, 0, What)
    want = oracle.decode(C16, idx.astype(np.int32), d_out, d_in, 0)
    assert np.array_equal(u.u16_np(What.view(torch.uint16)).reshape(d_out, d_in), want.view(np.uint16))


@pytest.mark.parametrize("g,d_out,K", [
    (4, 2078, 1), (4, 2078, 3000), (4, 2078, 16385), (4, 2078, 19841), (4, 2078, 40000), (4, 2078, 65536),
    (8, 2107, 2900), (8, 2107, 9000), (8, 2107, 10945), (8, 2107, 20001), (8, 2107, 65536),
    (16, 2170, 1400), (16, 2170, 5000), (16, 2170, 5729), (16, 2170, 65536),
])
def test_decode_with_whole_sixteen_byte_code_rows_matches_oracle(g, d_out, K):
    """Padded out_features a multiple of 8 g (every in_feature's code row is a whole number of 16-byte
    pieces), codebooks from one row to 2 MB with every row used, ragged tiles on both edges, padded
    out_features dropped."""
    cc, u = _cc(), _u()
    d_in = 2568
    rng = np.random.default_rng(g * 7919 + K)
    N = cc.cc_num_subvectors(d_out, d_in, g, 0)
    C16 = rng.standard_normal((K, g)).astype(np.float16)
    idx = rng.integers(0, K, N).astype(np.uint16)
    idx[:K] = np.arange(K)[::-1].astype(np.uint16)     # every row is used
    What = torch.zeros((d_out, d_in), dtype=torch.float16, device="cuda")
    cc.cc_decode(u.ctx(), u.half_dev(C16), K, g, u.dev(idx.view(np.int16)).view(torch.uint16), d_out, d_in, 0, What)
    want = oracle.decode(C16, idx.astype(np.int32), d_out, d_in, 0)
    assert np.array_equal(u.u16_np(What.view(torch.uint16)).reshape(d_out, d_in), want.view(np.uint16))


@pytest.mark.parametrize("N,g,K,seed", [(5000, 4, 700, 42), (257, 3, 257, 9), (100000, 8, 4096, 1)])
def test_init_codebook_matches_oracle(N, g, K, seed):
    cc, u = _cc(), _u()
    X = wl.make_points(N, g, seed)
    assert np.array_equal(cc.cc_init_positions(N, K, seed), oracle.init_positions(N, K, seed))
    u.ctx().ensure_workspace(N, g, K)
    C = torch.empty((K, g), dtype=torch.float32, device="cuda")
    cc.cc_init_codebook(u.ctx(), u.half_dev(X), N, g, K, seed, C)
    assert np.array_equal(C.cpu().numpy(), oracle.init_codebook(X, K, seed))


# ------------------------------------------------------------------ E-step

ASSIGN_CASES = [
    # N, g, K   (tile = 2048 points x 128..512 centroids: several tiles and ragged tails)
    (1, 4, 1), (31, 4, 2), (2049, 4, 33), (5000, 4, 255), (5000, 4, 257), (70001, 4, 1000),
    (16384, 4, 64), (16385, 1, 130), (20011, 5, 1000), (33000, 8, 700), (18000, 12, 200), (17000, 16, 2100),
    (40000, 3, 65), (25000, 7, 4097),
    (20000, 4, 4096), (3000, 4, 5000), (9000, 8, 300), (4097, 8, 2049), (6000, 16, 129),
    (2500, 16, 1500), (3001, 1, 17), (3001, 2, 64), (3001, 3, 100), (3001, 5, 600), (3001, 6, 90),
    (3001, 7, 1025), (3001, 9, 513), (1500, 12, 77), (1500, 13, 300), (1500, 15, 64),
]


@pytest.mark.parametrize("N,g,K", ASSIGN_CASES)
def test_assign_matches_oracle(N, g, K):
    u = _u()
    X = wl.make_points(N, g, 1000 + N + g)
    C = wl.make_codebook(K, g, 2000 + K + g)
    idx, dist, obj, nres, flagged = u.gpu_assign(X, C, want_flagged=True)
    tol, o_idx, d1 = u.check_assign_against_oracle(X, C, idx, dist, flagged=flagged)
    print("N=%d g=%d K=%d: %d tolerated near-ties, %d points sent to the exact stage" % (N, g, K, tol, nres))
    assert tol <= max(1, N // 1000)
    assert obj == pytest.approx(float(np.sum(dist.astype(np.float64))), rel=1e-12)
    assert obj == pytest.approx(d1.sum(), rel=1e-6)
    assert 0 <= nres <= N


@pytest.mark.parametrize("N,g,K", [(1, 4, 1), (2049, 4, 33), (70001, 4, 1000), (20000, 4, 4096), (9000, 8, 300),
                                   (4097, 8, 2049), (6000, 16, 129), (2500, 16, 1500), (1100, 4, 65536),
                                   (3001, 1, 17), (3001, 2, 64), (3001, 3, 100), (3001, 5, 600), (3001, 6, 90),
                                   (3001, 7, 1025), (3001, 9, 513), (1500, 12, 77), (1500, 13, 300), (1500, 15, 64),
                                   (150000, 4, 300), (40000, 9, 700),
                                   # enough full groups for the persistent scan, plus a ragged rest for the generic one
                                   (400001, 4, 300), (310000, 9, 129), (305000, 16, 70), (320001, 6, 200), (310000, 12, 129),
                                   (306000, 14, 75)])
def test_assign_fp32_and_tensor_paths_agree_with_oracle_and_each_other(N, g, K):
    cc, u = _cc(), _u()
    X = wl.make_points(N, g, 1000 + N + g)
    C = wl.make_codebook(K, g, 2000 + K + g)
    res = {}
    for path in (cc.PATH_FFMA, cc.PATH_TENSOR):
        idx, dist, obj, nres, flagged = u.gpu_assign(X, C, path=path, want_flagged=True)
        tol, o_idx, d1 = u.check_assign_against_oracle(X, C, idx, dist, flagged=flagged)
        assert tol <= max(1, N // 1000)
        res[path] = (idx, dist, obj)
    a, b = res[cc.PATH_FFMA], res[cc.PATH_TENSOR]
    differ = np.flatnonzero(a[0] != b[0])
    assert len(differ) <= max(1, N // 1000)          # only oracle near-ties may differ between the paths
    same = a[0] == b[0]
    assert np.array_equal(a[1][same], b[1][same])


def _tensor_units(g):
    """Rounding model of the tensor-core scan as the library documents it: contraction length,
    number of FP16 pieces per centroid value, allowed error in units of 2^-24 (2||c||^2 + ||x||^2):
    19 per 16-column step (17 addends aligned to the largest and cut 24 bits below it, plus the
    rounding of the sum), 4 for a value cut into two pieces instead of three, 4 for two norm pieces."""
    kd34, kd24, kd22 = (3 * g + 4 + 15) // 16 * 16, (2 * g + 4 + 15) // 16 * 16, (2 * g + 2 + 15) // 16 * 16
    full = kd34 <= 48 and kd34 <= kd24 and kd34 <= kd22
    split = 3 if full else 2                 # two pieces of a value where that shortens the contraction
    nq = 4 if (full or kd24 <= kd22) else 2  # ... and two pieces of the norm (g = 7, 15)
    kd = (split * g + nq + 15) // 16 * 16
    return split, kd, 19 * (kd // 16) + (4 if split == 2 else 0) + (4 if nq == 2 else 0), nq


def _score_case(kind, g, rng):
    """(X FP16, C FP32) of one family of inputs for the rounding-model test."""
    N, K = 2048, 5000                       # 1.0e7 scores per call; K is not a multiple of the 256-centroid tile
    if kind == "weights":
        return wl.make_points(N, g, 50 + g), wl.make_codebook(K, g, 60 + g)
    if kind == "wide_range":
        X = (rng.standard_normal((N, g)) * np.exp2(rng.uniform(-20, 6, (N, g)))).astype(np.float16)
        return X, (rng.standard_normal((K, g)) * np.exp2(rng.uniform(-24, 6, (K, g)))).astype(np.float32)
    if kind == "on_centroids":
        C = wl.make_codebook(K, g, 61 + g)
        return C[rng.integers(0, K, N)].astype(np.float16), C
    if kind == "huge":
        X = (rng.standard_normal((N, g)) * 2e4).clip(-65000, 65000).astype(np.float16)
        return X, (rng.standard_normal((K, g)) * 1e4).astype(np.float32)
    if kind == "on_centroids_large":         # points equal to centroids at large magnitude
        C = (rng.standard_normal((K, g)) * 3000).astype(np.float16).astype(np.float32)
        return C[rng.integers(0, K, N)].astype(np.float16), C
    if kind == "one_huge_norm":              # one centroid sets the scale, all the others are tiny beside it
        C = wl.make_codebook(K, g, 62 + g)
        C[K // 3] = 900.0
        return wl.make_points(N, g, 51 + g), C
    if kind == "cancellation":               # x = c / 2: x.c = ||c||^2 / 2, the score cancels to (almost) zero
        C = wl.make_codebook(K, g, 63 + g, scale=0.5)
        X = (C[rng.integers(0, K, N)] * 0.5).astype(np.float16)
        return X, C
    if kind == "subnormal_points":           # every coordinate of x below 2^-14
        X = (rng.uniform(-1, 1, (N, g)) * 6e-5).astype(np.float16)
        assert np.all(np.abs(X.astype(np.float64)) < 2.0 ** -14)
        return X, wl.make_codebook(K, g, 64 + g)
    if kind == "k65536_from_points":         # the benchmark's shape: 65536 centroids drawn from the points
        Xall = wl.make_points(70000, g, 52 + g)
        return Xall[:160], Xall[4000:4000 + 65536].astype(np.float32)
    raise ValueError(kind)


SCORE_KINDS = ["weights", "wide_range", "on_centroids", "huge", "on_centroids_large", "one_huge_norm", "cancellation",
               "subnormal_points", "k65536_from_points"]


@pytest.mark.parametrize("kind", SCORE_KINDS)
@pytest.mark.parametrize("g", [1, 3, 4, 5, 6, 7, 8, 9, 10, 12, 14, 15, 16])
def test_tensor_scores_obey_the_rounding_model(g, kind):
    """Every raw score of the tensor-core scan against float64 (10^7 scores per case): the error must
    stay inside the bound that decides which points are sent to the exact stage -- here inside a
    third of it, so that the bound keeps a margin over everything seen."""
    cc, u = _cc(), _u()
    rng = np.random.default_rng(100 * g + len(kind))
    X, C = _score_case(kind, g, rng)
    N, K = len(X), len(C)
    c = u.ctx()
    c.ensure_workspace(N, g, K)
    ld = cc.cc_tensor_scores_ld(K)
    assert ld % 256 == 0 and ld >= K
    out = torch.full((N, ld), float("nan"), dtype=torch.float32, device="cuda")
    cc.cc_tensor_scores(c, u.half_dev(X), N, g, u.dev(C), K, out)
    cc.cc_poll_status(c)
    got = out.cpu().numpy().astype(np.float64)[:, :K]
    del out
    assert np.isfinite(got).all()
    Xd, Cd = X.astype(np.float64), C.astype(np.float64)
    csq = (Cd ** 2).sum(1)
    exact = csq[None, :] - 2.0 * Xd @ Cd.T
    # the library's scale: largest power of two with S * 2 max|c| < 2^15 and S * max||c||^2 < 2^30
    k = min(14 - (int(np.floor(np.log2(np.abs(C).max()))) + 1), 29 - int(np.floor(np.log2(csq.max() * (1 + 1e-7)))), 40)
    inv_s = 2.0 ** -k
    split, kd, units, nq = _tensor_units(g)
    # two norm pieces multiply 2^e and 2^(e-11), e fitted to the largest scaled norm; a piece written
    # as zero loses at most 2^(e-25) (four pieces: 2^-26)
    e_norm = min(max(k + int(np.floor(np.log2(csq.max() * (1 + 1e-7)))) - 14, -3), 15)
    norm_abs = 2.0 ** (e_norm - 25) if nq == 2 else 2.0 ** -26
    xsq = (np.maximum(np.abs(Xd), 2.0 ** -14) ** 2).sum(1)      # subnormal coordinates count as 2^-14
    rel = 2.0 ** -24 * (2 * csq[None, :] + xsq[:, None])
    absolute = inv_s * (2.0 ** -14 * np.abs(Xd).sum(1)[:, None] + norm_abs)
    err = np.abs(got - exact)
    worst = float(((err - absolute).clip(0) / rel).max())
    print("g=%d %s: worst error %.2f units (bound %d), scale 2^%d, %d scores" % (g, kind, worst, units, k, N * K))
    assert worst <= units / 3


@pytest.mark.parametrize("g,K", [(4, 1000), (8, 300), (16, 65536), (5, 64)])
def test_finish_kernel_alone_is_right_on_good_scan_results_and_safe_on_garbage(g, K):
    """The second kernel of the tensor-core E-step reads the winning chunk of every point from the scan's
    output.  A scan CTA that gave up on a bounded wait writes nothing, so that word can be anything: run
    the kernel alone on (a) the oracle's chunks -- it must find the oracle's centroid up to FP32
    near-ties -- and (b) arbitrary bit patterns -- it must stay inside its tables and return codes < K."""
    cc, u = _cc(), _u()
    N = 20000
    X = wl.make_points(N, g, 800 + g)
    C = wl.make_codebook(K, g, 900 + g)
    o_idx, d1, _ = oracle.assign(X, C)
    c = u.ctx()
    c.ensure_workspace(N, g, K)
    Xd, Cd = u.half_dev(X), u.dev(C)
    idx = torch.empty(N, dtype=torch.uint16, device="cuda")
    dist = torch.empty(N, dtype=torch.float32, device="cuda")
    scan = np.zeros((N, 2), dtype=np.float32)
    scan[:, 0] = np.inf
    scan[:, 1] = (o_idx // 64).astype(np.int32).view(np.float32)
    cc.cc_tensor_finish_only(c, Xd, N, g, Cd, K, u.dev(scan), idx, dist)
    cc.cc_poll_status(c)
    got = u.u16_np(idx).astype(np.int32)
    assert np.array_equal(got // 64, o_idx // 64)
    d_got = dist.cpu().numpy().astype(np.float64)
    slack = 1e-6 * ((X.astype(np.float64) ** 2).sum(1) + (C.astype(np.float64)[o_idx] ** 2).sum(1))
    assert np.all(d_got <= d1 + slack)                              # the chunk's best up to FP32 rounding
    assert np.mean(got == o_idx) > 0.999
    rng = np.random.default_rng(g)
    junk = rng.integers(-2 ** 31, 2 ** 31, (N, 2), dtype=np.int64).astype(np.int32)
    junk[::7, 1] = -1
    junk[::11, 1] = 2 ** 31 - 1
    junk[::13, 1] = (K + 63) // 64                                  # one past the last chunk
    cc.cc_tensor_finish_only(c, Xd, N, g, Cd, K, u.dev(junk.view(np.float32)), idx, dist)
    cc.cc_poll_status(c)                                            # no fault, no status bit
    got = u.u16_np(idx).astype(np.int32)
    assert got.min() >= 0 and got.max() < K
    assert np.isfinite(dist.cpu().numpy()).all()


def test_assign_exact_ties_and_duplicates_take_lowest_index():
    u = _u()
    g, K, N = 4, 600, 4000
    X = wl.make_points(N, g, 5)
    C = wl.make_codebook(K, g, 6)
    X[:K] = C.astype(np.float16)                  # points sitting (almost) on centroids
    C[:64] = X[:64].astype(np.float32)            # ... and exactly on them
    C[300:400] = C[100:200]                       # duplicated centroids
    C[450] = C[3]
    idx, dist, obj, nres = u.gpu_assign(X, C)
    o_idx, d1, d2 = oracle.assign(X, C)
    assert np.array_equal(idx, o_idx)             # exact ties included: no tolerance here
    assert not np.any((idx >= 300) & (idx < 400)) and not np.any(idx == 450)
    assert np.all(dist[:64] == 0)
    assert nres >= 100


def test_assign_lattice_points_with_many_exact_ties():
    u = _u()
    rng = np.random.default_rng(0)
    X = (rng.integers(-3, 4, (6000, 4)) * 0.25).astype(np.float16)      # exactly representable grid
    C = (rng.integers(-3, 4, (300, 4)) * 0.25 + 0.125).astype(np.float32)
    idx, dist, obj, nres = u.gpu_assign(X, C)
    o_idx, d1, _ = oracle.assign(X, C)
    assert np.array_equal(idx, o_idx) and np.array_equal(dist, d1.astype(np.float32))


def test_assign_empty_input_and_null_dist():
    cc, u = _cc(), _u()
    C = wl.make_codebook(10, 4, 1)
    idx, dist, obj, nres = u.gpu_assign(np.zeros((0, 4), np.float16), C)
    assert len(idx) == 0 and obj == 0.0 and nres == 0
    X = wl.make_points(3000, 4, 2)
    a = u.gpu_assign(X, C, want_dist=False)
    b = u.gpu_assign(X, C)
    assert np.array_equal(a[0], b[0]) and a[2] == b[2]


def test_assign_metamorphic_scaling_and_determinism():
    u = _u()
    X = wl.make_points(30000, 4, 11)
    C = wl.make_codebook(777, 4, 12)
    a = u.gpu_assign(X, C)
    b = u.gpu_assign(X, C)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) and a[2] == b[2] and a[3] == b[3]
    Xs = (X.astype(np.float32) * 4).astype(np.float16)
    s = u.gpu_assign(Xs, C * 4)
    assert np.array_equal(s[0], a[0]) and np.array_equal(s[1], a[1] * 16)


def test_assign_reports_nonfinite_input():
    cc, u = _cc(), _u()
    X = wl.make_points(5000, 4, 13)
    X[1234, 2] = np.inf
    with pytest.raises(cc.CCError) as e:
        u.gpu_assign(X, wl.make_codebook(50, 4, 14))
    assert e.value.status == 8
    u.gpu_assign(wl.make_points(100, 4, 1), wl.make_codebook(5, 4, 1))   # status was cleared


# ------------------------------------------------------------------ M-step

@pytest.mark.parametrize("N,g,K", [(1, 4, 3), (5000, 4, 64), (70001, 4, 1000), (9000, 8, 5000), (6000, 16, 129),
                                   (3001, 5, 17), (3001, 9, 200), (4000, 1, 7),
                                   # large inputs with accumulators that fit one SM: the shared-memory kernel
                                   (400001, 4, 300), (1500000, 16, 1400), (2000000, 4, 4096), (900000, 7, 2000),
                                   # ... and with accumulators that do not: L2 reductions
                                   (3000003, 4, 65536), (2000000, 9, 65500)])
def test_update_matches_oracle_bit_for_bit(N, g, K):
    u = _u()
    X = wl.make_points(N, g, 3000 + N)
    rng = np.random.default_rng(N)
    idx = rng.integers(0, max(1, K - 2), N).astype(np.int32)      # the last clusters stay empty
    C_prev = wl.make_codebook(K, g, 4000 + K)
    C_or, counts_or = oracle.update(X, idx, C_prev)
    C_gpu, counts_gpu = u.gpu_update(X, idx, C_prev)
    assert np.array_equal(counts_gpu.astype(np.int64), counts_or)
    assert u.centroid_rel_err(C_gpu, C_or, X) <= u.REL_CENTROID
    assert np.array_equal(C_gpu.view(np.uint32), C_or.view(np.uint32))     # exact integer sums: same bits
    assert np.array_equal(C_gpu[counts_or == 0].view(np.uint32), C_prev[counts_or == 0].view(np.uint32))


@pytest.mark.parametrize("N", [20000, 200000])
def test_update_large_and_tiny_values_and_point_order(N):
    """Values on the coarse accumulator (|x| >= 8), subnormals, a fixed point order and a shuffled one;
    the larger size takes the shared-memory kernel."""
    u = _u()
    rng = np.random.default_rng(3)
    X = wl.make_points(N, 4, 77)
    X[::7] = (rng.standard_normal((len(X[::7]), 4)) * 300).astype(np.float16)       # |x| >= 8 accumulator
    X[::11] = (rng.standard_normal((len(X[::11]), 4)) * 1e-6).astype(np.float16)    # subnormals
    idx = rng.integers(0, 50, len(X)).astype(np.int32)
    C_prev = np.zeros((50, 4), np.float32)
    C_or, counts_or = oracle.update(X, idx, C_prev)
    C_gpu, counts_gpu = u.gpu_update(X, idx, C_prev)
    assert np.array_equal(counts_gpu, counts_or)
    assert u.centroid_rel_err(C_gpu, C_or, X) <= u.REL_CENTROID
    assert np.array_equal(C_gpu.view(np.uint32), C_or.view(np.uint32))
    p = rng.permutation(len(X))
    C_perm, _ = u.gpu_update(X[p], idx[p], C_prev)
    assert np.array_equal(C_perm.view(np.uint32), C_gpu.view(np.uint32))


@pytest.mark.parametrize("N,g,K", [(1, 4, 3), (70001, 4, 1000), (9000, 8, 5000), (6000, 16, 129), (3001, 9, 200),
                                   (200000, 6, 65500)])
def test_codebook_grad_matches_oracle_bit_for_bit(N, g, K):
    """Gradient of the decoded weights pushed back to the codebook: exact integer sums on the GPU,
    float64 sums in the oracle, both rounded once, so the bits must agree; empty clusters get 0."""
    cc, u = _cc(), _u()
    rng = np.random.default_rng(N + K)
    dX = (rng.standard_normal((N, g)) * rng.choice([1e-4, 0.05, 40.0], (N, 1))).astype(np.float16)
    idx = rng.integers(0, max(1, K - 2), N).astype(np.int32)
    want = oracle.codebook_grad(dX, idx, K)
    c = u.ctx()
    c.ensure_workspace(N, g, K)
    dC = torch.full((K, g), 7.0, dtype=torch.float32, device="cuda")
    idxd = torch.from_numpy(idx.astype(np.uint16).view(np.int16)).cuda().view(torch.uint16)
    cc.cc_codebook_grad(c, u.half_dev(dX), N, g, idxd, K, dC)
    cc.cc_poll_status(c)
    got = dC.cpu().numpy()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    p = rng.permutation(N)                                   # order of the sub-vectors must not matter
    idxp = torch.from_numpy(idx[p].astype(np.uint16).view(np.int16)).cuda().view(torch.uint16)
    cc.cc_codebook_grad(c, u.half_dev(dX[p]), N, g, idxp, K, dC)
    assert np.array_equal(dC.cpu().numpy().view(np.uint32), want.view(np.uint32))


# ------------------------------------------------------------------ Lloyd loop

def _lockstep(X, C0, iters, full_oracle=True, sel=None):
    """Drive assign/update from the host; at every iteration the oracle gets the GPU's centroids."""
    u = _u()
    C = C0.copy()
    tolerated, trace = 0, []
    for it in range(iters):
        idx, dist, obj, nres = u.gpu_assign(X, C)
        t, o_idx, d1 = u.check_assign_against_oracle(X, C, idx, dist, sel)
        tolerated += t
        if sel is None:
            assert obj == pytest.approx(d1.sum(), rel=u.REL_OBJECTIVE)
        C_or, counts_or = oracle.update(X, idx, C)          # oracle M-step on the GPU's own indices
        C_gpu, counts_gpu = u.gpu_update(X, idx, C)
        assert np.array_equal(counts_gpu, counts_or)
        assert u.centroid_rel_err(C_gpu, C_or, X) <= u.REL_CENTROID
        trace.append(obj)
        C = C_gpu
    return C, trace, tolerated


def _gpu_fit(X, C0, iters, path=0):
    cc, u = _cc(), _u()
    N, g = X.shape
    K = C0.shape[0]
    c = u.ctx()
    c.ensure_workspace(N, g, K)
    cc.cc_set_path(c, path)
    Xd, C = u.half_dev(X), u.dev(C0)
    idx = torch.empty(N, dtype=torch.uint16, device="cuda")
    dist = torch.empty(N, dtype=torch.float32, device="cuda")
    counts = torch.empty(K, dtype=torch.int32, device="cuda")
    trace = torch.empty(max(iters, 1), dtype=torch.float64, device="cuda")
    cc.cc_fit(c, Xd, N, g, K, iters, C, idx, dist, counts, trace)
    cc.cc_poll_status(c)
    cc.cc_set_path(c, 0)
    return C.cpu().numpy(), u.u16_np(idx).astype(np.int32), dist.cpu().numpy(), counts.cpu().numpy(), \
        trace.cpu().numpy()[:iters]


def test_cfg1_lockstep_fit_and_free_run():
    u = _u()
    w = wl.WORKLOADS["cfg1_256x512_g4_k256"]
    W = wl.make_matrix(w.matrices[0])
    X = oracle.reshape_subvectors(W, w.g)
    C0 = oracle.init_codebook(X, w.K, w.matrices[0].init_seed)
    C_lock, trace_lock, tol = _lockstep(X, C0, w.iters)
    print("cfg1 tolerated near-ties:", tol)
    C_fit, idx_fit, dist_fit, counts_fit, trace_fit = _gpu_fit(X, C0, w.iters)
    assert np.array_equal(C_fit.view(np.uint32), C_lock.view(np.uint32))      # cc_fit == the driven loop
    assert np.array_equal(trace_fit, np.array(trace_lock))
    assert np.all(np.diff(trace_fit) <= 1e-6 * trace_fit[:-1])                # objective never increases
    C_or, idx_or, d1_or, counts_or, obj_or = oracle.fit(X, C0, w.iters)        # free-running oracle
    assert trace_fit[-1] == pytest.approx(obj_or[-1], rel=u.REL_OBJECTIVE)
    assert np.allclose(trace_fit, obj_or, rtol=u.REL_OBJECTIVE)
    assert counts_fit.sum() == len(X)


@pytest.mark.parametrize("N,g,K,iters", [(30000, 4, 300, 6), (9000, 8, 5000, 4), (5000, 16, 40, 5), (7000, 5, 129, 4)])
def test_fit_moves_only_changed_points_yet_matches_the_driven_loop(N, g, K, iters):
    """cc_fit sums all points in its first M-step and afterwards only moves the points whose code
    changed; with exact integer sums that must give the same bits as a full M-step every time,
    including for values on the coarse accumulator (|x| >= 8), subnormals and emptied clusters."""
    u = _u()
    rng = np.random.default_rng(N + g)
    X = wl.make_points(N, g, 7000 + N)
    X[::5] = (rng.standard_normal((len(X[::5]), g)) * 200).astype(np.float16)
    X[::9] = (rng.standard_normal((len(X[::9]), g)) * 1e-6).astype(np.float16)
    C0 = oracle.init_codebook(X, K, 11)
    C_fit, idx_fit, dist_fit, counts_fit, trace_fit = _gpu_fit(X, C0, iters)
    C = C0.copy()
    for it in range(iters):
        idx, dist, obj, nres = u.gpu_assign(X, C)
        assert obj == trace_fit[it]
        C, counts = u.gpu_update(X, idx, C)
    assert np.array_equal(idx_fit, idx) and np.array_equal(counts_fit, counts)
    assert np.array_equal(C_fit.view(np.uint32), C.view(np.uint32))
    C_or, counts_or = oracle.update(X, idx, C)            # fixed point check of the last state against the oracle
    assert np.array_equal(counts_or, counts)


def test_set_codebook_from_host_and_device():
    cc, u = _cc(), _u()
    C0 = wl.make_codebook(333, 6, 3)
    C = torch.zeros((333, 6), dtype=torch.float32, device="cuda")
    cc.cc_set_codebook(u.ctx(), C0, 333, 6, C)                       # pageable host memory
    torch.cuda.synchronize()
    assert np.array_equal(C.cpu().numpy(), C0)
    C2 = torch.zeros_like(C)
    cc.cc_set_codebook(u.ctx(), C, 333, 6, C2)                       # device to device
    torch.cuda.synchronize()
    assert np.array_equal(C2.cpu().numpy(), C0)
    with pytest.raises(cc.CCError) as e:
        cc.cc_set_codebook(u.ctx(), C0, 70000, 6, C)
    assert e.value.status == 4


def test_blobs_recovered_and_k_equals_n():
    u = _u()
    X, labels, centres = wl.make_blobs(12, 300, 4, seed=90, sep=1.0, sigma=0.01)
    first = np.array([np.flatnonzero(labels == b)[0] for b in range(12)])
    C, idx, dist, counts, trace = _gpu_fit(X, X[first].astype(np.float32), 4)
    assert np.array_equal(idx, labels) and np.all(counts == 300)
    Xd = X.astype(np.float64)
    for b in range(12):
        assert np.array_equal(C[b], Xd[labels == b].mean(0).astype(np.float32))
    Xu = np.unique(wl.make_points(3000, 4, 80), axis=0)
    N = len(Xu)
    C0 = oracle.init_codebook(Xu, N, 5)
    C, idx, dist, counts, trace = _gpu_fit(Xu, C0, 2)
    assert np.all(trace == 0) and np.all(counts == 1) and np.array_equal(C[idx], Xu.astype(np.float32))


def test_finalize_decode_identity_and_compress_host():
    cc, u = _cc(), _u()
    w = wl.WORKLOADS["cfg1_256x512_g4_k256"]
    W = wl.make_matrix(w.matrices[0])
    d_out, d_in = W.shape
    for layout in (0, 1):
        N = cc.cc_num_subvectors(d_out, d_in, w.g, layout)
        C16 = torch.empty((w.K, w.g), dtype=torch.float16).pin_memory()
        idx = torch.empty(N, dtype=torch.uint16).pin_memory()
        trace = torch.empty(w.iters + 1, dtype=torch.float64).pin_memory()
        What = torch.empty((d_out, d_in), dtype=torch.float16).pin_memory()
        Wh = torch.from_numpy(W.view(np.int16)).view(torch.float16).pin_memory()
        cc.cc_compress_host(u.ctx(), Wh, d_out, d_in, w.g, w.K, w.iters, w.matrices[0].init_seed, layout, C16, idx,
                            trace, What)
        C16n = C16.numpy()
        idxn = idx.view(torch.int16).numpy().view(np.uint16).astype(np.int32)
        Whn = What.numpy()
        err = ((W.astype(np.float64) - Whn.astype(np.float64)) ** 2).sum()
        assert err == pytest.approx(trace[-1].item(), rel=1e-6)             # ||W - decode||^2 = objective
        # the oracle agrees on every piece, given the GPU's stored codebook
        X = oracle.reshape_subvectors(W, w.g, layout)
        t, o_idx, d1 = u.check_assign_against_oracle(X, C16n.astype(np.float32), idxn, None)
        assert np.array_equal(Whn.view(np.uint16), oracle.decode(C16n, idxn, d_out, d_in, layout).view(np.uint16))
        assert trace[-1].item() == pytest.approx(d1.sum(), rel=u.REL_OBJECTIVE)
        # free-running oracle from the same start reaches the same objective
        C0 = oracle.init_codebook(X, w.K, w.matrices[0].init_seed)
        C_or = oracle.fit(X, C0, w.iters)[0]
        _, _, _, J_or = oracle.finalize(X, C_or)
        assert trace[-1].item() == pytest.approx(J_or, rel=u.REL_OBJECTIVE)
        assert np.array_equal(oracle.to_half(C_or).view(np.uint16), C16n.view(np.uint16)) or \
            u.centroid_rel_err(C16n.astype(np.float32), oracle.to_half(C_or).astype(np.float32), X) < 2e-3


# ------------------------------------------------------------------ the paper's own (g, n) settings

@pytest.mark.parametrize("name,frac", [("grid_g6_n65500", 0.001), ("grid_g9_n65500", 0.001),
                                       ("grid_g5_n50000", 0.001), ("grid_g7_n35000", 0.001)])
def test_paper_grid_settings_padded_and_sampled(name, frac):
    """The paper's own (g, n) settings on a 4096 x 4096 matrix: g does not divide 4096, so every
    in_feature's last sub-vector is zero-padded, and n is not a power of two.  Two lock-step
    iterations on a seeded sample, then the whole path from host buffers: decode must invert the
    codes exactly and the objective must exceed ||W - decode||^2 by the padded coordinates' share."""
    cc, u = _cc(), _u()
    w = wl.WORKLOADS[name]
    spec = w.matrices[0]
    W = wl.make_matrix(spec)
    X = oracle.reshape_subvectors(W, w.g)
    assert len(X) == w.n_subvectors(spec) == cc.cc_num_subvectors(spec.d_out, spec.d_in, w.g, 0)
    C0 = oracle.init_codebook(X, w.K, spec.init_seed)
    sel = wl.subset_positions(len(X), frac, 5)
    C, trace, tol = _lockstep(X, C0, 2, sel=sel)
    print(name, "tolerated near-ties on the sample:", tol, "objective", trace)
    assert trace[1] < trace[0]
    d_out, d_in = W.shape
    N = len(X)
    C16 = torch.empty((w.K, w.g), dtype=torch.float16).pin_memory()
    idx = torch.empty(N, dtype=torch.uint16).pin_memory()
    tr = torch.empty(3, dtype=torch.float64).pin_memory()
    What = torch.empty((d_out, d_in), dtype=torch.float16).pin_memory()
    Wh = torch.from_numpy(W.view(np.int16)).view(torch.float16).pin_memory()
    cc.cc_compress_host(u.ctx(), Wh, d_out, d_in, w.g, w.K, 2, spec.init_seed, 0, C16, idx, tr, What)
    C16n = C16.numpy()
    idxn = idx.view(torch.int16).numpy().view(np.uint16).astype(np.int32)
    assert idxn.max() < w.K
    assert np.array_equal(What.numpy().view(np.uint16), oracle.decode(C16n, idxn, d_out, d_in).view(np.uint16))
    err = ((W.astype(np.float64) - What.numpy().astype(np.float64)) ** 2).sum()
    # padded coordinates are ordinary zeros for the clustering: they add the square of the chosen centroid's
    # coordinate to the objective but are dropped by decode
    pad = (-d_out) % w.g
    rec = C16n.astype(np.float64)[idxn].reshape(d_in, -1)          # (in_features, out_pad)
    pad_share = (rec[:, d_out:] ** 2).sum() if pad else 0.0
    assert pad > 0 and pad_share > 0
    assert tr[-1].item() == pytest.approx(err + pad_share, rel=1e-7)   # dist is rounded to FP32 per point
    u.check_assign_against_oracle(X, C16n.astype(np.float32), idxn, None, sel)


# ------------------------------------------------------------------ bounded device-side waits

def test_a_barrier_wait_that_cannot_end_gives_up_and_reports_it():
    """The scan kernels wait on shared-memory barriers; each wait is bounded by a clock limit.  The
    self-test runs that wait code on a barrier nobody arrives on (limit 2e6 cycles, about 1 ms)."""
    cc, u = _cc(), _u()
    limit = 2_000_000
    res, cyc = cc.cc_selftest_bounded_wait(u.ctx(), limit)
    assert res == [1, 0, 1, 0]                 # completes; gives up; flag raised; later waits return at once
    assert limit < cyc[0] < 4 * limit          # gave up shortly after the limit
    assert cyc[1] < limit // 2                 # with the flag up a wait ends after 16 polls
    with pytest.raises(cc.CCError):
        cc.cc_selftest_bounded_wait(u.ctx(), 10)   # limit out of range


"""GPU parity of the options around the clustering path: codebook quantisation (Section 5.3), the
cluster-splitting rule for empty clusters, training-set subsampling, and the many-matrices call."""
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


# ------------------------------------------------------------------ uniform codebook quantisation

@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("K,g,kind", [(65536, 4, "t"), (65500, 9, "t"), (35001, 7, "t"), (256, 4, "grid"), (5, 3, "zero"),
                                      (4096, 16, "t")])
def test_quantize_codebook_matches_oracle_bit_for_bit(K, g, kind, bits):
    cc, u = _cc(), _u()
    rng = np.random.default_rng(K + g + bits)
    if kind == "t":
        C16 = (rng.standard_t(3.0, (K, g)) * 0.02).astype(np.float16)
    elif kind == "grid":
        C16 = (rng.integers(-7, 8, (K, g)) * 0.25).astype(np.float16)      # ties at exact halves of the 8-bit grid
        C16[0, 0] = 1.75
    else:
        C16 = np.zeros((K, g), np.float16)
    q_or, s_or, deq_or = oracle.quantize_codebook(C16, bits)
    c = u.ctx()
    c.ensure_workspace(1024, g, K)
    n = K * g
    q = torch.full((n if bits == 8 else (n + 1) // 2,), 0x55, dtype=torch.uint8, device="cuda")
    scale = torch.zeros(1, dtype=torch.float32, device="cuda")
    deq = torch.zeros((K, g), dtype=torch.float16, device="cuda")
    cc.cc_quantize_codebook(c, u.half_dev(C16), K, g, bits, q, scale, deq)
    cc.cc_poll_status(c)
    assert np.float32(scale.item()) == np.float32(s_or)
    want = q_or.reshape(-1).view(np.uint8) if bits == 8 else oracle.pack_nibbles(q_or)
    assert np.array_equal(q.cpu().numpy(), want)
    assert np.array_equal(u.u16_np(deq.view(torch.uint16)).reshape(K, g), deq_or.view(np.uint16))
    # the dequantised codebook is an ordinary FP16 codebook for decode
    d_out, d_in = 4 * g, 24
    idx = rng.integers(0, K, oracle.num_subvectors(d_out, d_in, g)).astype(np.uint16)
    What = torch.zeros((d_out, d_in), dtype=torch.float16, device="cuda")
    cc.cc_decode(c, deq, K, g, u.dev(idx.view(np.int16)).view(torch.uint16), d_out, d_in, 0, What)
    assert np.array_equal(u.u16_np(What.view(torch.uint16)).reshape(d_out, d_in),
                          oracle.decode(deq_or, idx.astype(np.int32), d_out, d_in).view(np.uint16))
    cc.cc_quantize_codebook(c, u.half_dev(C16), K, g, bits, q, scale, None)          # without the dequantised copy
    with pytest.raises(cc.CCError) as e:
        cc.cc_quantize_codebook(c, u.half_dev(C16), K, g, 2, q, scale, None)
    assert e.value.status == 2


# ------------------------------------------------------------------ cluster-splitting rule

def _gpu_update_rule(X, idx, C_prev, rule):
    cc, u = _cc(), _u()
    c = u.ctx()
    cc.cc_set_empty_rule(c, rule)
    try:
        return u.gpu_update(X, idx, C_prev)
    finally:
        cc.cc_set_empty_rule(c, cc.EMPTY_KEEP)


@pytest.mark.parametrize("N,g,K,used", [(5000, 4, 64, 40), (70001, 4, 1000, 700), (100000, 6, 65536, 65536),
                                        (3000, 16, 5000, 5000), (2000, 8, 300, 1), (500, 3, 40, 33)])
def test_update_with_split_rule_matches_oracle_bit_for_bit(N, g, K, used):
    """M-step followed by the splitting rule; `used` codes are drawn from, the other clusters (and, with
    more clusters than points, many more) are empty.  With `used` = 1 one cluster donates again and again."""
    cc, u = _cc(), _u()
    X = wl.make_points(N, g, 3100 + N)
    rng = np.random.default_rng(N + K)
    idx = rng.integers(0, used, N).astype(np.int32)
    C_prev = wl.make_codebook(K, g, 4100 + K)
    C_m, counts_or = oracle.update(X, idx, C_prev)
    C_or = oracle.split_empty(C_m, counts_or)
    C_gpu, counts_gpu = _gpu_update_rule(X, idx, C_prev, cc.EMPTY_SPLIT_LARGEST)
    assert np.array_equal(counts_gpu.astype(np.int64), counts_or)            # true member counts, untouched
    assert np.array_equal(C_gpu.view(np.uint32), C_or.view(np.uint32))
    assert (counts_or == 0).sum() > 0 and not np.array_equal(C_or, C_m)
    C_keep, _ = _gpu_update_rule(X, idx, C_prev, cc.EMPTY_KEEP)
    assert np.array_equal(C_keep.view(np.uint32), C_m.view(np.uint32))


def test_fit_with_split_rule_follows_the_oracle_in_lock_step():
    cc, u = _cc(), _u()
    X, labels, centres = wl.make_blobs(6, 200, 4, seed=4, sep=1.0, sigma=0.02)
    first = np.array([np.flatnonzero(labels == b)[0] for b in range(6)])
    C0 = X[first].astype(np.float32)
    C0[5] = 50.0                                         # a start far from every point: its cluster is empty
    N, g = X.shape
    K, iters = 6, 5
    c = u.ctx()
    c.ensure_workspace(N, g, K)
    cc.cc_set_empty_rule(c, cc.EMPTY_SPLIT_LARGEST)
    try:
        C = u.dev(C0)
        idx = torch.empty(N, dtype=torch.uint16, device="cuda")
        dist = torch.empty(N, dtype=torch.float32, device="cuda")
        counts = torch.empty(K, dtype=torch.int32, device="cuda")
        trace = torch.empty(iters, dtype=torch.float64, device="cuda")
        cc.cc_fit(c, u.half_dev(X), N, g, K, iters, C, idx, dist, counts, trace)
        cc.cc_poll_status(c)
    finally:
        cc.cc_set_empty_rule(c, cc.EMPTY_KEEP)
    C_or, idx_or, _, counts_or, obj_or = oracle.fit_ex(X, C0, iters, oracle.EMPTY_SPLIT)
    assert np.array_equal(u.u16_np(idx).astype(np.int32), idx_or)
    assert np.array_equal(counts.cpu().numpy().astype(np.int64), counts_or) and counts_or.min() > 0
    assert np.array_equal(C.cpu().numpy().view(np.uint32), C_or.view(np.uint32))
    assert np.allclose(trace.cpu().numpy(), obj_or, rtol=u.REL_OBJECTIVE)
    with pytest.raises(cc.CCError) as e:
        cc.cc_set_empty_rule(c, 2)
    assert e.value.status == 11


# ------------------------------------------------------------------ training-set subsampling

@pytest.mark.parametrize("N,g,K,mppc", [(60000, 4, 100, 30), (60000, 4, 100, 200), (20000, 8, 50, 1000), (9000, 5, 64, 7)])
def test_fit_sampled_matches_oracle(N, g, K, mppc):
    """30 points per centroid of 60000: few positions (only the touched entries of the shuffle are kept);
    200 per centroid: a third of all positions (the whole array is shuffled); 1000 per centroid: every point."""
    cc, u = _cc(), _u()
    X = wl.make_points(N, g, 900 + N + mppc)
    seed, iters = 17, 4
    C0 = oracle.init_codebook(X, K, 3)
    n = cc.cc_train_points(N, K, mppc)
    pos = oracle.train_positions(N, K, mppc, seed)
    assert n == (N if pos is None else len(pos))
    c = u.ctx()
    c.ensure_workspace(N, g, K)
    Xd = u.half_dev(X)
    Xt = torch.zeros((n, g), dtype=torch.float16, device="cuda")
    C = u.dev(C0)
    idx = torch.empty(N, dtype=torch.uint16, device="cuda")
    dist = torch.empty(N, dtype=torch.float32, device="cuda")
    counts = torch.empty(K, dtype=torch.int32, device="cuda")
    trace = torch.empty(iters, dtype=torch.float64, device="cuda")
    cc.cc_fit_sampled(c, Xd, N, g, K, iters, mppc, seed, Xt if n < N else None, C, idx, dist, counts, trace)
    cc.cc_poll_status(c)
    if n < N:
        assert np.array_equal(u.u16_np(Xt.view(torch.uint16)).reshape(n, g), X[pos].view(np.uint16))   # the drawn rows
    C_or, idx_or, d1_or, counts_or, obj_or = oracle.fit_sampled(X, C0, iters, mppc, seed)
    C_gpu = C.cpu().numpy()
    assert np.allclose(trace.cpu().numpy(), obj_or, rtol=u.REL_OBJECTIVE)
    assert counts.cpu().numpy().sum() == n
    # the final E-step over ALL points, in lock-step with the GPU's own fitted codebook
    idx_gpu = u.u16_np(idx).astype(np.int32)
    u.check_assign_against_oracle(X, C_gpu, idx_gpu, dist.cpu().numpy())
    if np.array_equal(idx_gpu, idx_or):
        assert np.array_equal(C_gpu.view(np.uint32), C_or.view(np.uint32))
        assert np.array_equal(counts.cpu().numpy().astype(np.int64), counts_or)
    else:
        assert u.centroid_rel_err(C_gpu, C_or, X) < 0.05


# ------------------------------------------------------------------ many matrices

def test_compress_many_equals_one_call_per_matrix():
    cc, u = _cc(), _u()
    shapes = [(64, 96), (40, 56), (128, 32)]
    g, K, iters = 4, 20, 3
    Ws, outs = [], []
    for k, (o, i) in enumerate(shapes):
        W = wl.make_matrix(wl.MatrixSpec("m%d" % k, o, i, "student_t3", 0.02, 0.0, 70 + k, 0))
        Ws.append(torch.from_numpy(W.view(np.int16)).view(torch.float16).pin_memory())
        N = cc.cc_num_subvectors(o, i, g, 0)
        outs.append([torch.empty((K, g), dtype=torch.float16).pin_memory(), torch.empty(N, dtype=torch.uint16).pin_memory(),
                     torch.empty(iters + 1, dtype=torch.float64).pin_memory(), torch.empty((o, i), dtype=torch.float16).pin_memory()])
    seeds = [5, 6, 7]
    cc.cc_compress_many(u.ctx(), Ws, [s[0] for s in shapes], [s[1] for s in shapes], g, K, iters, seeds, 0,
                        [o[0] for o in outs], [o[1] for o in outs], [o[2] for o in outs], [o[3] for o in outs])
    for k, (o, i) in enumerate(shapes):
        N = cc.cc_num_subvectors(o, i, g, 0)
        C16 = torch.empty((K, g), dtype=torch.float16).pin_memory()
        idx = torch.empty(N, dtype=torch.uint16).pin_memory()
        tr = torch.empty(iters + 1, dtype=torch.float64).pin_memory()
        What = torch.empty((o, i), dtype=torch.float16).pin_memory()
        cc.cc_compress_host(u.ctx(), Ws[k], o, i, g, K, iters, seeds[k], 0, C16, idx, tr, What)
        assert torch.equal(C16.view(torch.int16), outs[k][0].view(torch.int16))
        assert torch.equal(idx.view(torch.int16), outs[k][1].view(torch.int16))
        assert torch.equal(tr, outs[k][2]) and torch.equal(What.view(torch.int16), outs[k][3].view(torch.int16))
    # optional lists may be left out altogether
    cc.cc_compress_many(u.ctx(), Ws, [s[0] for s in shapes], [s[1] for s in shapes], g, K, iters, seeds, 0,
                        [o[0] for o in outs], [o[1] for o in outs])

"""GPU parity of the compressed linear layer's forward (appendix listing): y = x . codebook[code]-as-weight + bias
through the C ABI against the float64 oracle, element by element.

Tolerance: FP16 inputs are exact, their products are exact in FP32, and the only error is the FP32
accumulation over d_in terms on the tensor core; 1e-3 relative, with an absolute floor of 1e-3 of the
output's root mean square for outputs that cancel to (almost) zero.
"""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

RTOL = 1e-3


def _case(M, d_out, d_in, g, K, seed):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((M, d_in)) * 0.5).astype(np.float16)
    C16 = (rng.standard_t(3.0, (K, g)) * 0.02).astype(np.float16)
    idx = rng.integers(0, K, oracle.num_subvectors(d_out, d_in, g)).astype(np.uint16)
    bias = rng.standard_normal(d_out).astype(np.float32)
    return x, C16, idx, bias


def _gpu_forward(x, C16, idx, d_out, d_in, bias):
    from paper_2503_13089_b200 import binding as cc
    from tests import gpu_util as u
    M = x.shape[0]
    K, g = C16.shape
    c = u.ctx()
    c.ensure_workspace(len(idx), g, K, at_least=cc.cc_linear_workspace_bytes(c, M, d_out, d_in))
    y = torch.full((M, d_out), float("nan"), dtype=torch.float32, device="cuda")
    cc.cc_linear_forward(c, u.half_dev(x), M, u.half_dev(C16), K, g, u.dev(idx.view(np.int16)).view(torch.uint16),
                         d_out, d_in, None if bias is None else u.dev(bias), y)
    cc.cc_poll_status(c)
    return y.cpu().numpy()


def _check(y, want):
    assert np.isfinite(y).all()
    err = np.abs(y.astype(np.float64) - want)
    bound = RTOL * np.abs(want) + RTOL * np.sqrt(np.mean(want ** 2))
    assert np.all(err <= bound), "worst error / bound: %.3g" % float((err / bound).max())
    return float((err / bound).max())


@pytest.mark.parametrize("M,d_out,d_in,g,K", [
    (1, 256, 512, 4, 256),          # one token: 16-column MMA, split over the in_features
    (600, 260, 200, 4, 300), (1024, 130, 328, 8, 77),   # from 512 tokens on one weight tile serves 512 tokens (two MMAs)
    (16, 1000, 520, 4, 700),        # ragged last tile of out_features; in_features not a multiple of 64
    (5, 130, 67, 6, 50),            # padded out_features (130 = 21 x 6 + 4), in_features not a multiple of 8
    (7, 75, 40, 9, 33), (3, 64, 24, 1, 5), (9, 96, 72, 3, 40), (20, 250, 128, 5, 90), (11, 260, 64, 7, 300),
    (256, 512, 1024, 8, 4096),      # a full 256-token block
    (300, 384, 256, 16, 1000),      # two token blocks, the second ragged
    (130, 144, 328, 12, 77), (40, 280, 200, 10, 64), (33, 208, 136, 13, 21), (18, 300, 96, 14, 19),
    (24, 330, 80, 15, 23), (12, 132, 88, 11, 17), (50, 136, 4104, 2, 9),
    (64, 4096, 4096, 4, 65536),     # a 7B attention projection with the paper's largest codebook
])
def test_linear_forward_matches_oracle(M, d_out, d_in, g, K):
    x, C16, idx, bias = _case(M, d_out, d_in, g, K, M + d_out + d_in + g)
    want = oracle.linear_forward(x, C16, idx.astype(np.int32), d_out, d_in, bias)
    y = _gpu_forward(x, C16, idx, d_out, d_in, bias)
    worst = _check(y, want)
    y2 = _gpu_forward(x, C16, idx, d_out, d_in, bias)
    assert np.array_equal(y.view(np.uint32), y2.view(np.uint32))            # same bits on every call
    y0 = _gpu_forward(x, C16, idx, d_out, d_in, None)                       # without bias
    _check(y0, want - bias.astype(np.float64))
    print("M=%d %dx%d g=%d K=%d: worst error %.3f of the bound" % (M, d_out, d_in, g, K, worst))


def test_linear_forward_many_tokens_sampled_rows():
    """4096 tokens through a 4096 x 4096 layer (g = 4, K = 65536): the oracle computes a seeded sample of the rows."""
    M, d_out, d_in, g, K = 4096, 4096, 4096, 4, 65536
    x, C16, idx, bias = _case(M, d_out, d_in, g, K, 5)
    y = _gpu_forward(x, C16, idx, d_out, d_in, bias)
    rows = np.sort(np.random.default_rng(6).choice(M, 12, replace=False))
    want = oracle.linear_forward(np.ascontiguousarray(x[rows]), C16, idx.astype(np.int32), d_out, d_in, bias)
    _check(y[rows], want)
    assert np.isfinite(y).all()


def test_linear_forward_equals_decode_then_matmul():
    """The fused kernel against the unfused route on the GPU itself: cc_decode, then a float64 product on the host."""
    from paper_2503_13089_b200 import binding as cc
    from tests import gpu_util as u
    M, d_out, d_in, g, K = 32, 520, 384, 8, 3000
    x, C16, idx, bias = _case(M, d_out, d_in, g, K, 11)
    y = _gpu_forward(x, C16, idx, d_out, d_in, None)
    What = torch.zeros((d_out, d_in), dtype=torch.float16, device="cuda")
    cc.cc_decode(u.ctx(), u.half_dev(C16), K, g, u.dev(idx.view(np.int16)).view(torch.uint16), d_out, d_in, 0, What)
    W_hat = What.cpu().numpy().astype(np.float64)
    _check(y, x.astype(np.float64) @ W_hat.T)


# ------------------------------------------------------------------ 4-bit codebook (Section 5.3)

def _gpu_forward_q4(x, C16, idx, d_out, d_in, bias):
    """cc_quantize_codebook(bits = 4) on the device, then the forward on the packed codebook; also returns the
    dequantised FP16 codebook the quantiser wrote."""
    from paper_2503_13089_b200 import binding as cc
    from tests import gpu_util as u
    M = x.shape[0]
    K, g = C16.shape
    c = u.ctx()
    c.ensure_workspace(len(idx), g, K, at_least=cc.cc_linear_workspace_bytes(c, M, d_out, d_in))
    q = torch.zeros((K * g + 1) // 2, dtype=torch.uint8, device="cuda")
    scale = torch.zeros(1, dtype=torch.float32, device="cuda")
    deq = torch.zeros((K, g), dtype=torch.float16, device="cuda")
    cc.cc_quantize_codebook(c, u.half_dev(C16), K, g, 4, q, scale, deq)
    y = torch.full((M, d_out), float("nan"), dtype=torch.float32, device="cuda")
    cc.cc_linear_forward_q4(c, u.half_dev(x), M, q, scale, K, g, u.dev(idx.view(np.int16)).view(torch.uint16), d_out, d_in,
                            None if bias is None else u.dev(bias), y)
    cc.cc_poll_status(c)
    return y.cpu().numpy(), deq.cpu().numpy()


@pytest.mark.parametrize("M,d_out,d_in,g,K", [
    (1, 256, 512, 4, 256), (16, 1000, 520, 4, 700), (5, 130, 72, 6, 50), (9, 96, 72, 2, 40), (130, 144, 328, 12, 77),
    (40, 512, 256, 8, 30000),       # 120,000 bytes of packed codebook
    (24, 256, 128, 16, 16384),      # exactly the 131,072 bytes that fit
    (33, 208, 136, 10, 21), (18, 300, 96, 14, 19),
    (64, 4096, 4096, 4, 65536),     # the paper's largest codebook at g = 4: 128 KB packed
    (200, 384, 256, 4, 65535),      # four token blocks of 64; an odd number of bytes
    (300, 384, 520, 4, 65535),      # from 256 tokens on: blocks of 256 tokens, two stages beside the table
    (256, 200, 136, 8, 1000), (700, 130, 72, 6, 50),
])
def test_linear_forward_q4_matches_oracle(M, d_out, d_in, g, K):
    from paper_2503_13089_b200 import binding as cc
    x, C16, idx, bias = _case(M, d_out, d_in, g, K, 3 * M + d_out + g)
    q_or, s_or, deq_or = oracle.quantize_codebook(C16, 4)
    y, deq_gpu = _gpu_forward_q4(x, C16, idx, d_out, d_in, bias)
    assert np.array_equal(deq_gpu.view(np.uint16), deq_or.view(np.uint16))
    want = oracle.linear_forward(x, deq_or, idx.astype(np.int32), d_out, d_in, bias)      # the layer on the dequantised codebook
    _check(y, want)
    y_fp16 = _gpu_forward(x, deq_or, idx, d_out, d_in, bias)                             # the FP16 kernel on the same codebook
    few = 4 if g <= 8 else 2        # up to here the look-up kernel without the tensor core runs
    if few < M <= 64:      # same token blocks and splits: the same sums in the same order
        assert np.array_equal(y.view(np.uint32), y_fp16.view(np.uint32))
    else:
        _check(y_fp16, want)


@pytest.mark.parametrize("M,d_out,d_in,g,K", [
    (1, 4096, 4096, 4, 65536),      # one token through the paper's largest codebook at g = 4: 37 slices of 111 in_features
    (4, 4096, 4096, 4, 65536), (3, 1000, 520, 4, 700), (4, 130, 67, 4, 50), (2, 260, 1031, 4, 65535), (2, 28672, 256, 4, 4096),
    (1, 64, 24, 2, 5), (4, 75, 40, 2, 33), (4, 250, 300, 6, 90), (3, 4096, 2048, 8, 32768), (4, 200, 72, 8, 2900),
    (2, 144, 328, 10, 77), (1, 260, 64, 12, 300), (2, 300, 96, 14, 19), (2, 2048, 1024, 16, 16384), (1, 8200, 40, 16, 1400),
    (2, 128, 5000, 4, 256),         # one block of code groups, in_features cut into more slices than 16 each would give
    (1, 40, 9, 4, 3),               # fewer than 16 in_features
    (1, 123000, 2050, 2, 16),       # more blocks of code groups than arrival counters, three slices: the reduction is a kernel of its own
])
def test_linear_forward_q4_few_tokens_matches_oracle(M, d_out, d_in, g, K):
    """The kernel that serves a handful of tokens (no tensor core: table look-ups and FP32 FMAs) against the oracle's
    layer on the oracle's dequantised codebook; the same bits on every call; with and without bias."""
    x, C16, idx, bias = _case(M, d_out, d_in, g, K, 7 * M + d_in + g)
    _, _, deq_or = oracle.quantize_codebook(C16, 4)
    want = oracle.linear_forward(x, deq_or, idx.astype(np.int32), d_out, d_in, bias)
    y, _ = _gpu_forward_q4(x, C16, idx, d_out, d_in, bias)
    worst = _check(y, want)
    y2, _ = _gpu_forward_q4(x, C16, idx, d_out, d_in, bias)
    assert np.array_equal(y.view(np.uint32), y2.view(np.uint32))
    y0, _ = _gpu_forward_q4(x, C16, idx, d_out, d_in, None)
    _check(y0, want - bias.astype(np.float64))
    print("M=%d %dx%d g=%d K=%d: worst error %.3f of the bound" % (M, d_out, d_in, g, K, worst))


def test_linear_forward_q4_rejects_what_it_cannot_hold():
    from paper_2503_13089_b200 import binding as cc
    from tests import gpu_util as u
    c = u.ctx()
    c.ensure_workspace(70000, 4, 64)
    x = torch.zeros((4, 64), dtype=torch.float16, device="cuda")
    y = torch.full((4, 64), 5.0, dtype=torch.float32, device="cuda")
    q = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    scale = torch.ones(1, dtype=torch.float32, device="cuda")
    idx = torch.zeros(64 * 64, dtype=torch.uint16, device="cuda")
    for g, K, status in ((5, 64, 3), (1, 64, 3), (8, 65536, 2), (16, 16385, 2), (4, 0, 4)):
        with pytest.raises(cc.CCError) as e:
            cc.cc_linear_forward_q4(c, x, 4, q, scale, K, g, idx, 64, 64, None, y)
        assert e.value.status == status, (g, K)
    torch.cuda.synchronize()
    assert bool((y == 5).all())

"""Error paths of the C ABI: every status other than CC_OK, through every entry point that can return it.

The contract (include/cluscomp.h): arguments are validated on the host before anything is launched;
a call that returns a status other than CC_OK has enqueued nothing.  Each case below breaks exactly
one argument of an otherwise valid call, expects the matching status, and then checks that the
output arrays still hold the sentinel they were filled with.
"""
import numpy as np
import pytest
import torch

from paper_2503_13089_b200 import workloads as wl

pytestmark = pytest.mark.gpu

NULL, SHAPE, BAD_G, BAD_K, N_LT_K, ALIGN, WORKSPACE, LAYOUT = 1, 2, 3, 4, 5, 6, 7, 11
N, G, K = 5000, 4, 64
D_OUT, D_IN = 100, 200          # 100 x 200 matrix: 25 groups of 4 per in_feature -> 5000 sub-vectors


def _cc():
    from paper_2503_13089_b200 import binding
    return binding


class Args:
    """A valid argument set on the device; outputs are filled with sentinels."""

    def __init__(self, with_workspace=True):
        cc = _cc()
        self.ctx = cc.Context(0)
        if with_workspace:
            self.ctx.ensure_workspace(70000, G, K)       # large enough for every N tried below
        X = wl.make_points(N, G, 1)
        self.xbuf = torch.zeros(N * G + 8, dtype=torch.float16, device="cuda")
        self.xbuf[:N * G] = torch.from_numpy(X.view(np.int16)).cuda().view(torch.float16).reshape(-1)
        self.X = self.xbuf[:N * G].view(N, G)
        self.X_odd = self.xbuf[1:N * G + 1].view(N, G)                # starts 2 bytes past a 16-byte boundary
        self.cbuf = torch.full((K * G + 8,), 0.5, dtype=torch.float32, device="cuda")
        self.C = self.cbuf[:K * G].view(K, G)
        self.C_odd = self.cbuf[1:K * G + 1].view(K, G)                # 4 bytes past: still not 16-byte aligned
        self.c16buf = torch.full((K * G + 8,), 0.25, dtype=torch.float16, device="cuda")
        self.C16 = self.c16buf[:K * G].view(K, G)
        self.C16_odd = self.c16buf[1:K * G + 1].view(K, G)
        self.wbuf = torch.full((D_OUT * D_IN + 8,), 3.0, dtype=torch.float16, device="cuda")
        self.W = self.wbuf[:D_OUT * D_IN].view(D_OUT, D_IN)
        self.W_odd = self.wbuf[1:D_OUT * D_IN + 1].view(D_OUT, D_IN)
        self.idx = torch.full((N,), 7, dtype=torch.uint16, device="cuda")
        self.dist = torch.full((N,), -1.0, dtype=torch.float32, device="cuda")
        self.counts = torch.full((K,), -5, dtype=torch.int32, device="cuda")
        self.obj = torch.full((32,), -2.0, dtype=torch.float64, device="cuda")
        self.nres = torch.full((1,), -3, dtype=torch.int64, device="cuda")
        self.scores = torch.full((8, 256), -4.0, dtype=torch.float32, device="cuda")
        self.scan = torch.zeros((N, 2), dtype=torch.float32, device="cuda")
        self.xinbuf = torch.full((8 * D_IN + 8,), 0.5, dtype=torch.float16, device="cuda")
        self.xin = self.xinbuf[:8 * D_IN].view(8, D_IN)
        self.xin_odd = self.xinbuf[1:8 * D_IN + 1].view(8, D_IN)
        self.ybuf = torch.full((8 * D_OUT + 8,), -6.0, dtype=torch.float32, device="cuda")
        self.y = self.ybuf[:8 * D_OUT].view(8, D_OUT)
        self.y_odd = self.ybuf[1:8 * D_OUT + 1].view(8, D_OUT)
        self.q8 = torch.full((K * G,), 0x55, dtype=torch.uint8, device="cuda")
        self.scale = torch.full((1,), -7.0, dtype=torch.float32, device="cuda")
        self.c16out = torch.full((K, G), -8.0, dtype=torch.float16, device="cuda")
        self.xtbuf = torch.full((N * G + 8,), -9.0, dtype=torch.float16, device="cuda")
        self.xtrain = self.xtbuf[:N * G].view(N, G)
        self.xtrain_odd = self.xtbuf[1:N * G + 1].view(N, G)
        self.snapshot = None

    def outputs(self):
        return [self.xbuf, self.cbuf, self.c16buf, self.wbuf, self.idx, self.dist, self.counts, self.obj, self.nres,
                self.scores, self.ybuf, self.q8, self.scale, self.c16out, self.xtbuf]

    def take_snapshot(self):
        torch.cuda.synchronize()
        self.snapshot = [t.clone() for t in self.outputs()]

    def assert_untouched(self):
        torch.cuda.synchronize()
        for now, before in zip(self.outputs(), self.snapshot):
            assert torch.equal(now.view(torch.uint8), before.view(torch.uint8))


def _calls(a, o):
    """The entry points as closures over the argument set `a`, each argument replaceable through `o`."""
    cc = _cc()
    v = lambda name, default: o.get(name, default)          # noqa: E731
    ctx = a.ctx
    return {
        "cc_reshape_subvectors": lambda: cc.cc_reshape_subvectors(ctx, v("W", a.W), v("d_out", D_OUT), v("d_in", D_IN),
                                                                  v("g", G), v("layout", 0), v("X", a.X)),
        "cc_init_codebook": lambda: cc.cc_init_codebook(ctx, v("X", a.X), v("N", N), v("g", G), v("K", K), 5, v("C", a.C)),
        "cc_set_codebook": lambda: cc.cc_set_codebook(ctx, v("C0", a.C16.float()), v("K", K), v("g", G), v("C", a.C)),
        "cc_assign": lambda: cc.cc_assign(ctx, v("X", a.X), v("N", N), v("g", G), v("C", a.C), v("K", K), v("idx", a.idx),
                                          a.dist, a.obj, a.nres),
        "cc_tensor_scores": lambda: cc.cc_tensor_scores(ctx, v("X", a.X), v("N", 8), v("g", G), v("C", a.C), v("K", K),
                                                        v("scores", a.scores)),
        "cc_tensor_finish_only": lambda: cc.cc_tensor_finish_only(ctx, v("X", a.X), v("N", N), v("g", G), v("C", a.C),
                                                                  v("K", K), v("scan", a.scan), v("idx", a.idx), a.dist),
        "cc_last_flagged": lambda: cc.cc_last_flagged(ctx, v("N", N), v("g", G), v("K", K), v("points", a.dist), v("count", 1)),
        "cc_update": lambda: cc.cc_update(ctx, v("X", a.X), v("N", N), v("g", G), v("idx", a.idx), v("K", K), v("C", a.C),
                                          v("counts", a.counts)),
        "cc_codebook_grad": lambda: cc.cc_codebook_grad(ctx, v("X", a.X), v("N", N), v("g", G), v("idx", a.idx), v("K", K),
                                                        v("C", a.C)),
        "cc_fit": lambda: cc.cc_fit(ctx, v("X", a.X), v("N", N), v("g", G), v("K", K), v("iters", 2), v("C", a.C),
                                    v("idx", a.idx), a.dist, v("counts", a.counts), a.obj),
        "cc_finalize": lambda: cc.cc_finalize(ctx, v("X", a.X), v("N", N), v("g", G), v("C", a.C), v("K", K),
                                              v("C16", a.C16), v("idx", a.idx), a.dist, a.obj),
        "cc_decode": lambda: cc.cc_decode(ctx, v("C16", a.C16), v("K", K), v("g", G), v("idx", a.idx), v("d_out", D_OUT),
                                          v("d_in", D_IN), v("layout", 0), v("W", a.W)),
        "cc_linear_forward": lambda: cc.cc_linear_forward(ctx, v("x", a.xin), v("M", 8), v("C16", a.C16), v("K", K), v("g", G),
                                                          v("idx", a.idx), v("d_out", D_OUT), v("d_in", D_IN), None, v("y", a.y)),
        "cc_linear_forward_q4": lambda: cc.cc_linear_forward_q4(ctx, v("x", a.xin), v("M", 8), v("q", a.q8), v("scale", a.scale),
                                                                v("K", K), v("g", G), v("idx", a.idx), v("d_out", D_OUT),
                                                                v("d_in", D_IN), None, v("y", a.y)),
        "cc_quantize_codebook": lambda: cc.cc_quantize_codebook(ctx, v("C16", a.C16), v("K", K), v("g", G), v("bits", 8),
                                                                v("q", a.q8), v("scale", a.scale), a.c16out),
        "cc_fit_sampled": lambda: cc.cc_fit_sampled(ctx, v("X", a.X), v("N", N), v("g", G), v("K", K), v("iters", 1),
                                                    v("mppc", 10), 3, v("Xt", a.xtrain), v("C", a.C), v("idx", a.idx),
                                                    a.dist, v("counts", a.counts), a.obj),
        "cc_update_static": lambda: cc.cc_update_static(0, v("X", a.X), v("N", N), v("g", G), v("idx", a.idx), v("K", K),
                                                        v("C", a.C), v("counts", a.counts)),
    }


NEEDS_WS = ["cc_init_codebook", "cc_assign", "cc_tensor_scores", "cc_tensor_finish_only", "cc_last_flagged", "cc_update",
            "cc_codebook_grad", "cc_fit", "cc_finalize", "cc_fit_sampled"]

CASES = []
for fn in ("cc_reshape_subvectors", "cc_init_codebook", "cc_assign", "cc_tensor_scores", "cc_tensor_finish_only",
           "cc_last_flagged", "cc_update", "cc_codebook_grad", "cc_fit", "cc_finalize", "cc_decode", "cc_update_static",
           "cc_set_codebook"):
    CASES += [(fn, {"g": 0}, BAD_G), (fn, {"g": 17}, BAD_G)]
for fn in ("cc_init_codebook", "cc_assign", "cc_tensor_scores", "cc_tensor_finish_only", "cc_last_flagged", "cc_update",
           "cc_codebook_grad", "cc_fit", "cc_finalize", "cc_decode", "cc_update_static", "cc_set_codebook"):
    CASES += [(fn, {"K": 0}, BAD_K), (fn, {"K": 65537}, BAD_K)]
CASES += [
    # NULL pointers
    ("cc_reshape_subvectors", {"W": None}, NULL), ("cc_reshape_subvectors", {"X": None}, NULL),
    ("cc_init_codebook", {"X": None}, NULL), ("cc_init_codebook", {"C": None}, NULL),
    ("cc_set_codebook", {"C0": None}, NULL), ("cc_set_codebook", {"C": None}, NULL),
    ("cc_assign", {"X": None}, NULL), ("cc_assign", {"C": None}, NULL), ("cc_assign", {"idx": None}, NULL),
    ("cc_tensor_scores", {"scores": None}, NULL), ("cc_tensor_finish_only", {"scan": None}, NULL),
    ("cc_last_flagged", {"points": None}, NULL),
    ("cc_update", {"X": None}, NULL), ("cc_update", {"idx": None}, NULL), ("cc_update", {"C": None}, NULL),
    ("cc_update", {"counts": None}, NULL), ("cc_codebook_grad", {"C": None}, NULL),
    ("cc_fit", {"X": None}, NULL), ("cc_fit", {"C": None}, NULL), ("cc_fit", {"idx": None}, NULL),
    ("cc_fit", {"counts": None}, NULL),
    ("cc_finalize", {"C16": None}, NULL), ("cc_finalize", {"idx": None}, NULL),
    ("cc_decode", {"C16": None}, NULL), ("cc_decode", {"idx": None}, NULL), ("cc_decode", {"W": None}, NULL),
    ("cc_update_static", {"C": None}, NULL), ("cc_update_static", {"counts": None}, NULL),
    ("cc_update_static", {"X": None}, NULL),
    # pointers 2 (FP16) or 4 (FP32) bytes past a 16-byte boundary
    ("cc_reshape_subvectors", {"W": "W_odd"}, ALIGN), ("cc_reshape_subvectors", {"X": "X_odd"}, ALIGN),
    ("cc_init_codebook", {"X": "X_odd"}, ALIGN), ("cc_init_codebook", {"C": "C_odd"}, ALIGN),
    ("cc_set_codebook", {"C": "C_odd"}, ALIGN),
    ("cc_assign", {"X": "X_odd"}, ALIGN), ("cc_assign", {"C": "C_odd"}, ALIGN),
    ("cc_tensor_scores", {"X": "X_odd"}, ALIGN), ("cc_tensor_finish_only", {"C": "C_odd"}, ALIGN),
    ("cc_update", {"X": "X_odd"}, ALIGN), ("cc_update", {"C": "C_odd"}, ALIGN),
    ("cc_codebook_grad", {"X": "X_odd"}, ALIGN),
    ("cc_fit", {"X": "X_odd"}, ALIGN), ("cc_fit", {"C": "C_odd"}, ALIGN),
    ("cc_finalize", {"X": "X_odd"}, ALIGN), ("cc_finalize", {"C16": "C16_odd"}, ALIGN),
    ("cc_decode", {"C16": "C16_odd"}, ALIGN), ("cc_decode", {"W": "W_odd"}, ALIGN),
    ("cc_update_static", {"X": "X_odd"}, ALIGN), ("cc_update_static", {"C": "C_odd"}, ALIGN),
    # sizes
    ("cc_reshape_subvectors", {"d_out": 0}, SHAPE), ("cc_reshape_subvectors", {"d_in": -1}, SHAPE),
    ("cc_decode", {"d_out": 0}, SHAPE), ("cc_assign", {"N": -1}, SHAPE), ("cc_assign", {"N": 1 << 31}, SHAPE),
    ("cc_update", {"N": -1}, SHAPE), ("cc_fit", {"N": 0}, SHAPE), ("cc_fit", {"iters": -1}, SHAPE),
    ("cc_finalize", {"N": 0}, SHAPE), ("cc_tensor_scores", {"N": 0}, SHAPE), ("cc_tensor_scores", {"N": 65537}, SHAPE),
    ("cc_tensor_finish_only", {"N": 0}, SHAPE), ("cc_last_flagged", {"count": N + 1}, SHAPE),
    ("cc_update_static", {"N": -1}, SHAPE),
    ("cc_init_codebook", {"N": K - 1}, N_LT_K), ("cc_init_codebook", {"N": 0}, SHAPE),
    # layout constants
    ("cc_reshape_subvectors", {"layout": 2}, LAYOUT), ("cc_decode", {"layout": -1}, LAYOUT),
    # the rows beyond the clustering path
    ("cc_linear_forward", {"g": 0}, BAD_G), ("cc_linear_forward", {"g": 17}, BAD_G), ("cc_linear_forward", {"K": 0}, BAD_K),
    ("cc_linear_forward", {"K": 65537}, BAD_K), ("cc_linear_forward", {"x": None}, NULL), ("cc_linear_forward", {"C16": None}, NULL),
    ("cc_linear_forward", {"idx": None}, NULL), ("cc_linear_forward", {"y": None}, NULL), ("cc_linear_forward", {"M": 0}, SHAPE),
    ("cc_linear_forward", {"d_in": 0}, SHAPE), ("cc_linear_forward", {"M": 1 << 30}, SHAPE),
    ("cc_linear_forward", {"C16": "C16_odd"}, ALIGN), ("cc_linear_forward", {"y": "y_odd"}, ALIGN),
    ("cc_linear_forward", {"x": "xin_odd"}, ALIGN),
    ("cc_linear_forward_q4", {"g": 0}, BAD_G), ("cc_linear_forward_q4", {"g": 18}, BAD_G), ("cc_linear_forward_q4", {"g": 3}, BAD_G),
    ("cc_linear_forward_q4", {"K": 0}, BAD_K), ("cc_linear_forward_q4", {"K": 65537}, BAD_K),
    ("cc_linear_forward_q4", {"x": None}, NULL), ("cc_linear_forward_q4", {"q": None}, NULL),
    ("cc_linear_forward_q4", {"scale": None}, NULL), ("cc_linear_forward_q4", {"idx": None}, NULL),
    ("cc_linear_forward_q4", {"y": None}, NULL), ("cc_linear_forward_q4", {"M": 0}, SHAPE),
    ("cc_linear_forward_q4", {"d_out": 0}, SHAPE), ("cc_linear_forward_q4", {"y": "y_odd"}, ALIGN),
    ("cc_linear_forward_q4", {"x": "xin_odd"}, ALIGN),
    ("cc_quantize_codebook", {"g": 0}, BAD_G), ("cc_quantize_codebook", {"K": 65537}, BAD_K),
    ("cc_quantize_codebook", {"bits": 2}, SHAPE), ("cc_quantize_codebook", {"bits": 16}, SHAPE),
    ("cc_quantize_codebook", {"C16": None}, NULL), ("cc_quantize_codebook", {"q": None}, NULL),
    ("cc_quantize_codebook", {"scale": None}, NULL),
    ("cc_fit_sampled", {"g": 17}, BAD_G), ("cc_fit_sampled", {"K": 0}, BAD_K), ("cc_fit_sampled", {"X": None}, NULL),
    ("cc_fit_sampled", {"Xt": None}, NULL), ("cc_fit_sampled", {"C": None}, NULL), ("cc_fit_sampled", {"counts": None}, NULL),
    ("cc_fit_sampled", {"mppc": 0}, SHAPE), ("cc_fit_sampled", {"iters": -1}, SHAPE), ("cc_fit_sampled", {"N": 0}, SHAPE),
    ("cc_fit_sampled", {"X": "X_odd"}, ALIGN), ("cc_fit_sampled", {"Xt": "xtrain_odd"}, ALIGN),
]


@pytest.fixture(scope="module")
def args():
    return Args()


@pytest.mark.parametrize("fn,override,status", CASES, ids=["%s-%s-%d" % (f, "_".join("%s=%s" % kv for kv in o.items()), s)
                                                             for f, o, s in CASES])
def test_bad_argument_returns_its_status_and_enqueues_nothing(args, fn, override, status):
    cc = _cc()
    o = {k: (getattr(args, val) if isinstance(val, str) else val) for k, val in override.items()}
    args.take_snapshot()
    with pytest.raises(cc.CCError) as e:
        _calls(args, o)[fn]()
    assert e.value.status == status, (fn, override, e.value.status)
    args.assert_untouched()


@pytest.mark.parametrize("fn", NEEDS_WS)
def test_workspace_missing_or_one_byte_short(fn):
    cc = _cc()
    a = Args(with_workspace=False)
    a.take_snapshot()
    with pytest.raises(cc.CCError) as e:                    # no workspace at all
        _calls(a, {})[fn]()
    assert e.value.status == WORKSPACE
    need = cc.cc_workspace_bytes(N, G, K) if fn != "cc_tensor_scores" else cc.cc_workspace_bytes(8, G, K)
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    cc.cc_set_workspace(a.ctx, ws, need - 1)
    a.take_snapshot()
    with pytest.raises(cc.CCError) as e:                    # one byte short
        _calls(a, {})[fn]()
    assert e.value.status == WORKSPACE
    a.assert_untouched()
    cc.cc_set_workspace(a.ctx, ws, need)                    # exactly enough: the call goes through
    if fn != "cc_last_flagged":
        _calls(a, {})[fn]()
        cc.cc_poll_status(a.ctx)
    a.ctx.close()


def test_context_level_errors():
    cc = _cc()
    a = Args()
    with pytest.raises(cc.CCError) as e:
        cc.cc_set_path(a.ctx, 3)
    assert e.value.status == LAYOUT
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(cc.CCError) as e:
        cc.cc_set_workspace(a.ctx, ws[2:], 4000)            # workspace itself misaligned
    assert e.value.status == ALIGN
    with pytest.raises(cc.CCError) as e:
        cc.cc_set_workspace(a.ctx, ws, 100)                 # smaller than the status words
    assert e.value.status == ALIGN
    fresh = cc.Context(0)
    with pytest.raises(cc.CCError) as e:
        cc.cc_poll_status(fresh)                            # nothing to poll without a workspace
    assert e.value.status == WORKSPACE
    assert cc.load().cc_destroy(None) == NULL and cc.load().cc_create(None, 0) == NULL
    h = cc._vp()
    assert cc.load().cc_create(cc.ct.byref(h), 10_000) == 10          # no such device: CC_ERR_CUDA
    for s in range(0, 13):
        assert cc.cc_status_string(s) != "unknown status"
    assert cc.cc_status_string(99) == "unknown status"


def test_compress_host_rejects_bad_arguments():
    cc = _cc()
    ctx = cc.Context(0)
    W = torch.zeros((D_OUT, D_IN), dtype=torch.float16).pin_memory()
    C16 = torch.full((K, G), 9.0, dtype=torch.float16).pin_memory()
    idx = torch.full((N,), 9, dtype=torch.uint16).pin_memory()
    ok = dict(d_out=D_OUT, d_in=D_IN, g=G, K=K, iters=1, layout=0)
    for change, status in (({"g": 0}, BAD_G), ({"g": 17}, BAD_G), ({"K": 0}, BAD_K), ({"K": 65537}, BAD_K),
                           ({"layout": 5}, LAYOUT), ({"iters": -1}, SHAPE), ({"d_out": 0}, SHAPE),
                           ({"K": N + 1}, N_LT_K)):
        p = dict(ok, **change)
        with pytest.raises(cc.CCError) as e:
            cc.cc_compress_host(ctx, W, p["d_out"], p["d_in"], p["g"], p["K"], p["iters"], 1, p["layout"], C16, idx)
        assert e.value.status == status, change
    with pytest.raises(cc.CCError) as e:
        cc.cc_compress_host(ctx, None, D_OUT, D_IN, G, K, 1, 1, 0, C16, idx)
    assert e.value.status == NULL
    assert bool((C16 == 9).all()) and bool((idx == 9).all())

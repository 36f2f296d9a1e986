"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared
symbol, and its host helpers agree with the paper's printed values and with the oracle."""
import os
import re

import numpy as np
import pytest

import oracle
from paper_2503_13089_b200 import binding as cc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "cluscomp.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(cc_[a-z0-9_]+)\s*\(", header))
    assert len(declared) >= 20
    lib = cc.load()
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(cc.SIGNATURES), declared ^ set(cc.SIGNATURES)


def test_host_helpers_follow_listing_and_eq1():
    for (o, i, g) in [(4096, 4096, 4), (4096, 4096, 6), (4096, 4096, 9), (10, 7, 4), (11008, 4096, 5)]:
        for layout in (0, 1):
            assert cc.cc_num_subvectors(o, i, g, layout) == oracle.num_subvectors(o, i, g, layout)
        assert cc.cc_bits_per_param(o, i, g, 65500) == oracle.bits_per_param(o, i, g, 65500)
    assert round(cc.cc_bits_per_param(4096, 4096, 4, 65500), 2) == 4.25      # printed in the paper's table
    assert round(cc.cc_bits_per_param(4096, 4096, 6, 65500), 2) == 3.04
    assert round(cc.cc_bits_per_param(4096, 4096, 9, 65500), 2) == 2.34
    assert cc.cc_num_subvectors(0, 4, 4, 0) == -1 and cc.cc_num_subvectors(4, 4, 4, 9) == -1


def test_init_positions_match_oracle_and_reject_bad_sizes():
    for N, K, seed in [(1000003, 5, 1234567), (5000, 700, 42), (257, 257, 9), (58720256, 65536, 2004)]:
        assert np.array_equal(cc.cc_init_positions(N, K, seed), oracle.init_positions(N, K, seed))
    with pytest.raises(cc.CCError) as e:
        cc.cc_init_positions(10, 11, 0)
    assert e.value.status == 5
    with pytest.raises(cc.CCError) as e:
        cc.cc_init_positions(10, 0, 0)
    assert e.value.status == 4
    with pytest.raises(cc.CCError) as e:
        cc.cc_init_positions(1 << 31, 4, 0)
    assert e.value.status == 2


def test_workspace_size_and_status_strings():
    assert cc.cc_workspace_bytes(1000, 4, 16) > 0
    assert cc.cc_workspace_bytes(1000, 17, 16) == 0 and cc.cc_workspace_bytes(1000, 4, 65537) == 0
    assert cc.cc_workspace_bytes(-1, 4, 16) == 0
    big = cc.cc_workspace_bytes(58720256, 4, 65536)
    assert 18 * 58720256 <= big < 18 * 58720256 + (64 << 20)
    assert cc.cc_status_string(0) == "ok" and "aligned" in cc.cc_status_string(6)


def test_no_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(cc.CCError) as e:
        cc.Context(0)
    assert e.value.status == 10


def test_workload_sizes_follow_the_padding_rule():
    """Every shipped workload's sub-vector count is the listing's padded num_codes, as the library and the
    oracle compute it (the paper-grid workloads have out_features that g does not divide)."""
    from paper_2503_13089_b200 import workloads as wl
    padded = 0
    for w in wl.WORKLOADS.values():
        for m in w.matrices:
            n = w.n_subvectors(m)
            assert n == cc.cc_num_subvectors(m.d_out, m.d_in, w.g, 0) == oracle.num_subvectors(m.d_out, m.d_in, w.g, 0)
            assert 1 <= w.K <= 65536 and n >= w.K
            padded += m.d_out % w.g != 0
    assert padded >= 4


def test_schedule_matrices_is_the_size_balanced_split():
    """Longest-processing-time first, as documented in the header.  One 7B decoder layer over two ranks,
    worked out by hand: the three MLP matrices (2.8 M sub-vectors) go first -- rank 0, rank 1, rank 0 (equal
    loads: the lower rank) -- then the four attention matrices (1.05 M) go to rank 1 three times (3.9, 4.9,
    6.0 M against 5.6 M) and the last one to rank 0.  The Python helper of the multi-process tests states
    the same rule and must agree on random sizes."""
    from paper_2503_13089_b200 import sharding
    att, mlp = 1048576, 2818048
    sizes = [att, att, att, att, mlp, mlp, mlp]
    assert cc.cc_schedule_matrices(sizes, 2, 0) == [3, 4, 6]
    assert cc.cc_schedule_matrices(sizes, 2, 1) == [0, 1, 2, 5]
    rng = np.random.default_rng(0)
    for world in (1, 2, 3, 8):
        for n in (0, 1, 5, 40):
            sz = [int(v) for v in rng.integers(1, 1000, n)]
            want = sharding.assign_matrices(sz, world)
            got = [cc.cc_schedule_matrices(sz, world, r) for r in range(world)]
            assert got == want
            assert sorted(i for part in got for i in part) == list(range(n))
    with pytest.raises(cc.CCError):
        cc.cc_schedule_matrices([1, 2], 2, 2)


def test_sample_positions_match_the_oracle_shuffle_on_both_host_paths():
    """The training-set positions of a subsampled fit: few positions keep only the touched entries of
    the shuffle, many keep the whole array; both must be the oracle's full-array shuffle."""
    for N, n, seed in [(60000, 3000, 17), (60000, 20000, 17), (60000, 60000, 5), (1000, 0, 1), (1, 1, 9),
                       (3000000, 400000, 2), (3000000, 1000, 2)]:
        got = cc.cc_sample_positions(N, n, seed)
        want = oracle.init_positions(N, n, seed) if n else np.empty(0, np.int64)
        assert np.array_equal(got.astype(np.int64), want)
        assert len(set(got.tolist())) == n
    assert np.array_equal(cc.cc_sample_positions(5000, 700, 42).astype(np.int64), cc.cc_init_positions(5000, 700, 42))
    with pytest.raises(cc.CCError):
        cc.cc_sample_positions(10, 11, 0)

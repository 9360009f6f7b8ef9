"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared entry
point, its host helpers agree with the oracle, and argument errors are caught before any launch."""
import ctypes
import math
import os
import re

import numpy as np
import pytest

from oracle import compactor_oracle as orc
from paper_2507_08143_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_symbol_is_exported():
    header = open(os.path.join(ROOT, "include", "compactor.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(compactor_[a-z_0-9]+)\s*\(", header))
    assert {"compactor_score", "compactor_select", "compactor_compact", "compactor_compress"} <= declared
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS)
    assert B.version() >= 100


def test_keep_count_matches_oracle():
    for n in (0, 1, 2, 7, 100, 1024, 8192, 131072, 10 ** 6 + 3):
        for r in (1e-9, 0.07, 0.2, 0.3, 0.32, 0.5, 0.999999, 1.0):
            assert B.keep_count(n, r) == orc.keep_count(n, r), (n, r)
    assert B.keep_count(100, 0.07) == 8 and B.keep_count(8192, 0.3) == 2458 and B.keep_count(131072, 0.32) == 41944


def test_calibrated_ratio_matches_oracle():
    for b in (-10.0, -4.0, -1.0, -1e-8, 0.0, 2.0):
        for tau in (0.5, 0.9, 0.95, 1.0):
            got = B.calibrated_ratio(2.0, b / 4, b / 2, tau)
            assert abs(got - orc.calibrated_ratio(2.0, b / 4, b / 2, tau)) < 1e-12
            assert abs(orc.calibration_curve(got, b) - tau) < 1e-7
    with pytest.raises(B.CompactorError):
        B.calibrated_ratio(1.0, 1.0, 0.0, 0.0)
    with pytest.raises(B.CompactorError):
        B.calibrated_ratio(1.0, 1.0, 0.0, 1.5)


def test_fit_calibration_matches_oracle():
    rng = np.random.default_rng(21)
    nll = rng.uniform(0.5, 3.0, 80); r = rng.uniform(0.05, 1.0, 80)
    y_true = np.array([orc.calibration_curve(ri, -1.7 * ci - 0.8) for ri, ci in zip(r, nll)])
    a, b, loss = B.fit_calibration(r, nll, y_true)
    assert abs(a + 1.7) < 1e-6 and abs(b + 0.8) < 1e-6 and loss < 1e-20            # noise-free: exact recovery
    y = np.clip(y_true + 0.05 * rng.standard_normal(80), 0, 1)
    for w in (1.0, 4.0):
        a, b, loss = B.fit_calibration(r, nll, y, under_weight=w)
        ao, bo, lo = orc.fit_calibration(r, nll, y, under_weight=w)
        assert abs(loss - orc.calibration_loss(a, b, r, nll, y, w)) < 1e-12       # same objective
        assert loss <= lo * (1 + 1e-6) + 1e-15                                      # at least as good as the oracle's search
        assert abs(a - ao) < 2e-3 and abs(b - bo) < 2e-3
    with pytest.raises(B.CompactorError):
        B.fit_calibration([0.5], [1.0], [0.5])


def test_make_sketch_matches_oracle_generator():
    for seed, d, m in ((0, 128, 48), (12345, 128, 64), (7, 5, 3)):
        got = B.make_sketch(seed, d, m).numpy()
        want = orc.make_sketch(seed, d, m)
        # both follow the same counter-based recipe; libm and numpy may differ in the last bit
        np.testing.assert_allclose(got, want, rtol=3e-7, atol=1e-9)
    z = B.make_sketch(1, 128, 48).numpy().astype(np.float64) * math.sqrt(48)
    assert abs(z.mean()) < 0.05 and abs(z.std() - 1) < 0.05


def test_srht_sketch_matches_oracle_generator():
    for seed, d, m in ((0, 128, 48), (9, 128, 64), (3, 16, 16), (4, 8, 1)):
        np.testing.assert_array_equal(B.make_sketch_srht(seed, d, m).numpy(), orc.make_sketch_srht(seed, d, m))
    with pytest.raises(B.CompactorError):
        B.make_sketch_srht(0, 96, 48)                     # the Hadamard order must be a power of two


def test_workspace_bytes():
    small = B.workspace_bytes(B.Shape(1, 2, 128, 48, [1024]))
    big = B.workspace_bytes(B.Shape(64, 8, 128, 48, [131072]))
    assert 0 < small < big < 4 << 30
    assert small % 256 == 0
    assert B.workspace_bytes(B.Shape(1, 2, 64, 48, [1024])) == 0          # d != 128
    assert B.workspace_bytes(B.Shape(1, 2, 128, 129, [1024])) == 0        # m too large
    assert B.workspace_bytes(B.Shape(1, 2, 128, 128, [1024])) > small      # m = d: exact scores
    assert B.workspace_bytes(B.Shape(1, 2, 128, 48, [1024, 0, 77])) > 0   # empty sequences are fine


def test_workspace_sizes_of_the_other_entry_points():
    # selection across heads needs, per (layer, sequence), a histogram, a candidate list that grows with heads x n,
    # and two counts per slice; the one-call entry point needs the fused call's workspace plus what its options add
    shape = B.Shape(4, 8, 128, 48, [131072, 300, 0])
    tables = 256 * math.ceil(16 * (shape.batch + 1) / 256)
    across = B.across_heads_workspace_bytes(shape)
    groups = 4 * shape.batch
    assert across >= tables + groups * 2176 * 4 + 8 * (8 * shape.total_tokens // 256) and across % 256 == 0
    assert across < B.workspace_bytes(shape)
    base = B.workspace_bytes(shape)
    per_head = B.compress_full_workspace_bytes(shape, B.options(selection=B.SELECT_PER_HEAD))
    with_across = B.compress_full_workspace_bytes(shape, B.options(selection=B.SELECT_ACROSS_HEADS))
    with_attn = B.compress_full_workspace_bytes(shape, B.options(selection=B.SELECT_ACROSS_HEADS, q_per_kv=4, pool=7))
    plane = 4 * 4 * 8 * shape.total_tokens
    assert base <= per_head < with_across < with_attn
    assert with_attn - with_across >= 2 * plane          # the attention term and its unpooled copy
    # a ragged batch of the same size is planned with long blocks too: its Gram partials stay a small part of the workspace
    ragged = B.Shape(32, 8, 128, 48, [2278, 9042, 23584, 54094])
    uniform = B.Shape(32, 8, 128, 48, [22250] * 4)
    units, lh = 32 * 8 * 4, 32 * 8
    fixed = 4 * lh * ragged.total_tokens + units * (2 * 48 * 128 * 2 + 128 * 48 * 8)       # scores, W, the parts of A = Phi^T M Phi (G = A + A^T)
    partials = (B.workspace_bytes(ragged) - fixed) // (128 * 128 * 8 * lh)                  # Gram blocks per (layer, head)
    assert partials == 5                                  # blocks of 32768 tokens: 1 + 1 + 1 + 2
    fixed_u = 4 * lh * uniform.total_tokens + units * (2 * 48 * 128 * 2 + 128 * 48 * 8)
    assert (B.workspace_bytes(uniform) - fixed_u) // (128 * 128 * 8 * lh) == 4   # one block per sequence of 22250 tokens


def _mat(ptr=1 << 20, sl=1 << 20, sh=1 << 17, st=128):
    return B.CompactorMat(ptr, sl, sh, st)


def _score(shape, k, phi=1 << 21, out=1 << 22, ws=1 << 23, ws_bytes=1 << 40):
    return B.LIB.compactor_score(ctypes.byref(shape.c), k, ctypes.c_void_p(phi), None, 0.3, ctypes.c_void_p(out),
                                 None, ctypes.c_void_p(ws), ws_bytes, None)


def test_argument_errors_are_reported_before_any_launch():
    ok = B.Shape(1, 2, 128, 48, [1024])
    assert _score(B.Shape(1, 2, 96, 48, [1024]), _mat()) == -2
    assert _score(B.Shape(1, 2, 128, 0, [1024]), _mat()) == -2
    assert _score(B.Shape(0, 2, 128, 48, [1024]), _mat()) == -1
    assert _score(ok, _mat(ptr=0)) == -1
    assert _score(ok, _mat(ptr=(1 << 20) + 8)) == -1                   # 16-byte alignment
    assert _score(ok, _mat(st=120)) == -1                                # token stride below d
    assert _score(ok, _mat(st=132)) == -1                                # not a multiple of 8 elements
    assert _score(ok, _mat(), phi=0) == -1
    assert _score(ok, _mat(), out=0) == -1
    assert _score(ok, _mat(), ws=(1 << 23) + 64) == -1                   # workspace alignment
    assert _score(ok, _mat(), ws_bytes=1024) == -3
    bad = B.Shape(1, 2, 128, 48, [1024])
    bad._cu[1] = -5
    assert _score(bad, _mat()) == -1
    # select / compact: keep counts must lie in [0, n]
    keep = (ctypes.c_int32 * 1)(2000)
    rc = B.LIB.compactor_select(ctypes.byref(ok.c), ctypes.c_void_p(1 << 22), keep, ctypes.c_void_p(1 << 24), None,
                                ctypes.c_void_p(1 << 23), 1 << 20, None)
    assert rc == -1
    assert "workspace" in B.error_string(-3) and B.error_string(0) == "ok"


def test_variant_and_nll_argument_errors_are_reported_before_any_launch():
    ok = B.Shape(1, 2, 128, 48, [1024])
    wide = B.Shape(1, 2, 128, 128, [1024])
    dev = lambda a: ctypes.c_void_p(a)

    def variant(shape, fact, floor):
        return B.LIB.compactor_score_variant(ctypes.byref(shape.c), _mat(), dev(1 << 21), fact, floor, None, 0.3,
                                             dev(1 << 22), None, dev(1 << 23), 1 << 30, None)
    assert variant(ok, 7, 1e-6) == -1                                    # unknown factorisation
    assert variant(ok, B.FACTOR_EIG, 0.0) == -1 and variant(ok, B.FACTOR_EIG, float("nan")) == -1
    assert variant(wide, B.FACTOR_EIG, 1e-6) == -2                       # the eigen route stops at 64 columns
    assert B.workspace_bytes(wide) > B.workspace_bytes(ok)

    cu = (ctypes.c_int32 * 2)(0, 4)

    def nll(**kw):
        return B.LIB.compactor_nll(dev(kw.get("x", 1 << 20)), kw.get("dt", 0), kw.get("rows", 4), kw.get("vocab", 32),
                                   kw.get("stride", 32), dev(1 << 21), 1, kw.get("cu", cu), dev(1 << 22),
                                   dev(kw.get("out", 1 << 23)), None)
    assert nll(dt=5) == -1 and nll(vocab=0) == -1 and nll(rows=-1) == -1
    assert nll(stride=16) == -1                                          # rows overlap
    assert nll(stride=36) == -1                                          # 72 bytes: not a multiple of 16
    assert nll(x=(1 << 20) + 2) == -1 and nll(x=0) == -1 and nll(out=0) == -1
    assert nll(cu=(ctypes.c_int32 * 2)(0, 5)) == -1 and nll(cu=(ctypes.c_int32 * 2)(2, 4)) == -1

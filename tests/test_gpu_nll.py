"""GPU parity of the token-averaged negative log-likelihood (Section 3.5) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import compactor_oracle as orc

pytestmark = pytest.mark.gpu

# fp32 arithmetic on sums of up to ~1e5 exponentials: the row terms are O(10), their error O(1e-6)
NLL_ATOL = 2e-5


@pytest.fixture(scope="module")
def B():
    from paper_2507_08143_b200 import binding
    return binding


def _logits(rows, vocab, dtype, seed, stride=None, scale=4.0):
    g = torch.Generator(device="cpu"); g.manual_seed(seed)
    stride = vocab if stride is None else stride
    full = torch.randn(rows, stride, generator=g) * scale
    # a few dominant tokens per row, as a language model's head produces
    hot = torch.randint(0, vocab, (rows, 3), generator=g)
    full.scatter_(1, hot, 12.0 + 4.0 * torch.rand(rows, 3, generator=g))
    full = full.to(dtype)
    targets = torch.randint(0, vocab, (rows,), generator=g, dtype=torch.int32)
    targets[::3] = hot[::3, 0].int()                       # a third of the rows score a likely token
    return full, targets


def _run(B, full, vocab, targets, seq_rows):
    dev = full.cuda()
    view = dev[:, :vocab]
    row_nll = torch.full((full.shape[0],), -7.0, dtype=torch.float32, device="cuda")
    out = torch.full((len(seq_rows),), -7.0, dtype=torch.float64, device="cuda")
    B.nll(view, targets.cuda(), seq_rows, row_nll, out)
    torch.cuda.synchronize()
    return row_nll.cpu().numpy(), out.cpu().numpy()


def _check(full, vocab, targets, seq_rows, row_nll, out, loose_rows=()):
    # `loose_rows`: rows whose logits are so large that fp32 carries them to about 1e-3 only
    x = full[:, :vocab].double().numpy()
    t = targets.numpy()
    want_rows = orc.token_nll(x, t)
    tight = np.ones(len(t), dtype=bool); tight[list(loose_rows)] = False
    np.testing.assert_allclose(row_nll[tight], want_rows[tight], atol=NLL_ATOL, rtol=1e-5)
    np.testing.assert_allclose(row_nll[~tight], want_rows[~tight], atol=5e-3)
    r0 = 0
    for b, n in enumerate(seq_rows):
        want = orc.mean_nll(x[r0:r0 + n], t[r0:r0 + n])
        slack = 5e-3 * sum(1 for r in loose_rows if r0 <= r < r0 + n) / max(n, 1)
        assert abs(out[b] - want) <= NLL_ATOL + slack, (b, out[b], want)
        r0 += n


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("vocab,stride", [(5000, 5000), (4099, 4104), (1, 8), (37, 40), (128256, 128256)])
def test_nll_matches_the_oracle(B, dtype, vocab, stride):
    rows = 40 if vocab > 100000 else 333
    full, targets = _logits(rows, vocab, dtype, seed=vocab, stride=stride)
    seq_rows = [rows // 3, 0, rows - rows // 3 - 5, 5]
    row_nll, out = _run(B, full, vocab, targets, seq_rows)
    _check(full, vocab, targets, seq_rows, row_nll, out)


def test_unscored_rows_and_extreme_logits(B):
    rows, vocab = 64, 2048
    full, targets = _logits(rows, vocab, torch.float32, seed=5)
    targets[5] = -1; targets[6] = -100; targets[7] = vocab           # outside the vocabulary: unscored
    targets[40:48] = -1                                              # a sequence with no scored row
    full[10] = 0.0                                                   # uniform row: log(vocab)
    full[11] = -1e4; full[11, 3] = 50.0; targets[11] = 3             # one token holds all the mass
    full[12] = 3e4                                                   # large equal logits: no overflow
    seq_rows = [40, 8, 16]
    row_nll, out = _run(B, full, vocab, targets, seq_rows)
    t = targets.clone(); t[7] = -1
    _check(full, vocab, t, seq_rows, row_nll, out, loose_rows=[12])
    assert row_nll[5] == 0.0 and row_nll[7] == 0.0 and out[1] == 0.0
    assert abs(row_nll[10] - np.log(vocab)) < NLL_ATOL and abs(row_nll[11]) < NLL_ATOL
    assert abs(row_nll[12] - np.log(vocab)) < 5e-3


def test_nll_feeds_the_calibrated_ratio(B):
    # the path of Section 3.5 end to end: NLL(c) -> b = alpha NLL + beta -> r* -> kept tokens
    rows, vocab = 500, 3000
    full, targets = _logits(rows, vocab, torch.bfloat16, seed=9)
    _, out = _run(B, full, vocab, targets, [rows])
    want_nll = orc.mean_nll(full.double().numpy(), targets.numpy())
    alpha, beta, tau = 0.8, 0.5, 0.95
    r_gpu = B.calibrated_ratio(float(out[0]), alpha, beta, tau)
    r_cpu = orc.calibrated_ratio(want_nll, alpha, beta, tau)
    assert abs(r_gpu - r_cpu) < 1e-5
    assert B.keep_count(131072, r_gpu) == orc.keep_count(131072, r_cpu)


def test_nll_argument_checks(B):
    from ctypes import c_int32
    lib = B.LIB
    x = torch.zeros(4, 16, dtype=torch.float32, device="cuda")
    t = torch.zeros(4, dtype=torch.int32, device="cuda")
    rn = torch.zeros(4, dtype=torch.float32, device="cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    cu = (c_int32 * 2)(0, 4)
    ok = lambda **kw: lib.compactor_nll(kw.get("x", x.data_ptr()), kw.get("dt", 1), kw.get("rows", 4), kw.get("vocab", 16),
                                        kw.get("stride", 16), t.data_ptr(), 1, kw.get("cu", cu), rn.data_ptr(),
                                        kw.get("out", out.data_ptr()), None)
    assert ok() == 0
    assert ok(dt=2) == -1 and ok(vocab=0) == -1 and ok(stride=8) == -1 and ok(stride=18) == -1
    assert ok(x=x.data_ptr() + 4) == -1 and ok(out=None) == -1 and ok(x=None) == -1
    assert ok(cu=(c_int32 * 2)(0, 3)) == -1 and ok(cu=(c_int32 * 2)(1, 4)) == -1
    torch.cuda.synchronize()


def test_nll_throughput_is_reported(B):
    # not a pass/fail threshold: prints the streaming rate of the row kernel for the record
    rows, vocab = 8192, 128256
    x = torch.randn(rows, vocab, device="cuda", dtype=torch.bfloat16)
    t = torch.randint(0, vocab, (rows,), device="cuda", dtype=torch.int32)
    rn = torch.empty(rows, dtype=torch.float32, device="cuda")
    out = torch.empty(1, dtype=torch.float64, device="cuda")
    for _ in range(3):
        B.nll(x, t, [rows], rn, out)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        B.nll(x, t, [rows], rn, out)
    e1.record(); torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / 5
    print(f"nll bf16 {rows}x{vocab}: {ms:.3f} ms, {rows * vocab * 2 / ms / 1e6:.0f} GB/s")
    assert np.isfinite(out.cpu().numpy()).all()

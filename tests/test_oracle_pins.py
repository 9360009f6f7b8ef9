"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle's
own formulae.  No GPU needed."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import compactor_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


# ----------------------------------------------------------------------------- exact leverage
def _closed_form_cases():
    cases, name, rows = [], None, []
    for line in open(os.path.join(GOLDEN, "leverage_closed_forms.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("case "):
            name, rows = line.split()[1], []
        elif line.startswith("scores:"):
            want = [float(Fraction(t)) for t in line.split()[1:]]
            cases.append((name, np.array(rows, dtype=np.float64), np.array(want)))
        else:
            rows.append([float(t) for t in line.split()])
    return cases


@pytest.mark.parametrize("name,K,want", _closed_form_cases(), ids=lambda c: c if isinstance(c, str) else "")
def test_exact_leverage_closed_forms(name, K, want):
    np.testing.assert_allclose(orc.exact_leverage_scores(K), want, atol=1e-12)


def test_exact_leverage_hadamard_columns_are_uniform():
    # n x d matrix whose columns are d columns of a +-1 Hadamard matrix: K^T K = n I, so l_i = d / n.
    H = np.array([[1.0]])
    for _ in range(5):
        H = np.block([[H, H], [H, -H]])
    K = H[:, [1, 5, 9, 20, 31]] * 0.37
    np.testing.assert_allclose(orc.exact_leverage_scores(K), np.full(32, 5 / 32), atol=1e-12)


def test_exact_leverage_matches_gram_inverse_and_qr():
    # Eq. 2: U = K V Sigma^-1  =>  l_i = k_i (K^T K)^-1 k_i^T; Appendix C: l_i = ||Q_i||^2 for K = QR.
    K = _rng(1).standard_normal((200, 7)) * np.array([1, 10, 0.1, 3, 1, 1, 5.0])
    ell = orc.exact_leverage_scores(K)
    via_gram = np.einsum("ij,jk,ik->i", K, np.linalg.inv(K.T @ K), K)
    Q, _ = np.linalg.qr(K)
    np.testing.assert_allclose(ell, via_gram, rtol=1e-9)
    np.testing.assert_allclose(ell, np.sum(Q * Q, axis=1), rtol=1e-10)


def test_exact_leverage_invariants():
    rng = _rng(2)
    K = rng.standard_normal((300, 6))
    K[:, 5] = K[:, 0] - 2 * K[:, 1]                      # rank 5
    ell = orc.exact_leverage_scores(K)
    assert np.all(ell >= -1e-12) and np.all(ell <= 1 + 1e-12)
    assert abs(ell.sum() - 5.0) < 1e-9                   # sum = rank(K)
    A = rng.standard_normal((6, 6)) + 3 * np.eye(6)
    np.testing.assert_allclose(orc.exact_leverage_scores(K @ A), ell, atol=1e-9)   # K -> K A
    perm = rng.permutation(300)
    np.testing.assert_allclose(orc.exact_leverage_scores(K[perm]), ell[perm], atol=1e-10)


# ----------------------------------------------------------------------------- Algorithm 1
def test_alg1_full_sketch_equals_exact():
    rng = _rng(3)
    K = rng.standard_normal((500, 16)) * (np.arange(1, 17) ** -1.0)
    Phi = rng.standard_normal((16, 16))                  # m = d, invertible
    np.testing.assert_allclose(orc.approx_leverage_scores(K, Phi), orc.exact_leverage_scores(K), rtol=1e-7)


def test_alg1_single_column_sketch():
    # Phi = e_1 (m = 1): K_hat is the first column, so o_i = K_i1^2 / sum_j K_j1^2.
    K = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])
    e1 = np.array([[1.0], [0.0]])
    np.testing.assert_allclose(orc.approx_leverage_scores(K, e1), [0.5, 0.0, 0.5], atol=1e-14)
    K = _rng(4).standard_normal((50, 8))
    e3 = np.zeros((8, 1)); e3[3] = 1.0
    np.testing.assert_allclose(orc.approx_leverage_scores(K, e3), K[:, 3] ** 2 / np.sum(K[:, 3] ** 2), rtol=1e-12)


def test_alg1_invariants():
    rng = _rng(5)
    n, d, m = 400, 32, 12
    K = rng.standard_normal((n, d)) * (np.arange(1, d + 1) ** -0.7) + 0.5 * rng.standard_normal(d)
    Phi = rng.standard_normal((d, m)) / math.sqrt(m)
    o = orc.approx_leverage_scores(K, Phi)
    ell = orc.exact_leverage_scores(K)
    assert abs(o.sum() - m) < 1e-8                         # sum = rank(K Phi)
    assert np.all(o >= 0) and np.all(o <= ell + 1e-9)      # projection onto a subspace of col(K)
    np.testing.assert_allclose(orc.approx_leverage_scores(K, 7.5 * Phi), o, rtol=1e-9)       # scale of Phi
    A = rng.standard_normal((m, m)) + 2 * np.eye(m)
    np.testing.assert_allclose(orc.approx_leverage_scores(K, Phi @ A), o, rtol=1e-8)         # Phi -> Phi A
    extra = rng.standard_normal((d, 3))
    o_more = orc.approx_leverage_scores(K, np.hstack([Phi, extra]))
    assert np.all(o_more >= o - 1e-10)                     # appending columns never lowers a score
    perm = rng.permutation(n)
    np.testing.assert_allclose(orc.approx_leverage_scores(K[perm], Phi), o[perm], rtol=1e-9)


def test_alg1_matches_qr_route():
    # Appendix C: K_hat = QR, score = ||Q_i||^2.
    rng = _rng(6)
    K = rng.standard_normal((700, 24))
    Phi = rng.standard_normal((24, 9))
    Q, _ = np.linalg.qr(K @ Phi)
    np.testing.assert_allclose(orc.approx_leverage_scores(K, Phi), np.sum(Q * Q, axis=1), rtol=1e-9)


def test_alg1_rank_deficient_cases():
    rng = _rng(7)
    Phi = rng.standard_normal((16, 8))
    # fewer rows than sketch columns, full row rank: K_hat K_hat^+ = I_n, every score is 1
    K = rng.standard_normal((5, 16))
    np.testing.assert_allclose(orc.approx_leverage_scores(K, Phi), np.ones(5), atol=1e-9)
    # all-zero keys: no direction survives, all scores 0
    np.testing.assert_array_equal(orc.approx_leverage_scores(np.zeros((9, 16)), Phi), np.zeros(9))
    # copies of one row: rank 1, scores 1/n each
    K = np.tile(rng.standard_normal((1, 16)), (10, 1))
    np.testing.assert_allclose(orc.approx_leverage_scores(K, Phi), np.full(10, 0.1), atol=1e-9)
    # empty
    assert orc.approx_leverage_scores(np.zeros((0, 16)), Phi).shape == (0,)


def test_alg1_detects_a_transposed_or_dropped_factor():
    # An independent construction of the same number: o_i = k_hat_i G^+ k_hat_i^T.
    rng = _rng(8)
    K = rng.standard_normal((60, 10)); Phi = rng.standard_normal((10, 4))
    Kh = K @ Phi
    want = np.einsum("ij,jk,ik->i", Kh, np.linalg.pinv(Kh.T @ Kh), Kh)
    np.testing.assert_allclose(orc.approx_leverage_scores(K, Phi), want, rtol=1e-9)


def test_appendix_c_routes_agree_on_full_rank_input():
    # Full column rank and a floor far below the spectrum: all three routes give Algorithm 1's scores.
    rng = _rng(21)
    K = rng.standard_normal((300, 20)); Phi = rng.standard_normal((20, 7))
    o = orc.approx_leverage_scores(K, Phi)
    np.testing.assert_allclose(orc.approx_leverage_scores_qr(K, Phi), o, rtol=1e-9)
    np.testing.assert_allclose(orc.approx_leverage_scores_eig(K, Phi, 1e-6), o, rtol=1e-9)
    np.testing.assert_allclose(orc.approx_leverage_scores_qr(K, np.eye(20)), orc.exact_leverage_scores(K), rtol=1e-9)
    assert orc.approx_leverage_scores_eig(np.zeros((0, 20)), Phi).shape == (0,)
    assert orc.approx_leverage_scores_qr(np.zeros((0, 20)), Phi).shape == (0,)


def test_eig_route_clamp_closed_form():
    # K = Q diag(sigma) with orthonormal Q and Phi = the first m columns of the identity:
    # G = diag(sigma_j^2), so score_i = sum_j Q_ij^2 sigma_j^2 / max(sigma_j^2, eps).  Directions
    # above the floor count fully, directions below it are scaled by sigma_j^2 / eps.
    rng = _rng(22)
    n, d, m = 40, 6, 4
    Q, _ = np.linalg.qr(rng.standard_normal((n, d)))
    sigma = np.array([3.0, 1.0, 1e-2, 1e-4, 5.0, 2.0])
    K = Q * sigma[None, :]
    Phi = np.eye(d)[:, :m]
    for eps in (1e-12, 1e-6, 1e-3, 4.0):
        lam = sigma[:m] ** 2
        want = np.sum(Q[:, :m] ** 2 * (lam / np.maximum(lam, eps))[None, :], axis=1)
        np.testing.assert_allclose(orc.approx_leverage_scores_eig(K, Phi, eps), want, rtol=1e-7, atol=1e-12)
    # a floor above every eigenvalue turns the score into ||k_hat_i||^2 / eps
    big = orc.approx_leverage_scores_eig(K, Phi, 100.0)
    np.testing.assert_allclose(big, np.sum((K @ Phi) ** 2, axis=1) / 100.0, rtol=1e-9)
    # exactly rank-deficient input: the null directions contribute (numerically) nothing
    K2 = np.hstack([K[:, :3], K[:, :3]])
    got = orc.approx_leverage_scores_eig(K2, np.eye(6), 1e-6)
    np.testing.assert_allclose(got, orc.exact_leverage_scores(K2), atol=1e-7)


def test_bf16_widening_is_exact():
    import torch
    x = torch.randn(1000, dtype=torch.float32).to(torch.bfloat16)
    bits = x.view(torch.int16).numpy()
    np.testing.assert_array_equal(orc.bf16_bits_to_f64(bits), x.double().numpy())


# ----------------------------------------------------------------------------- sketch generator
def test_make_sketch_statistics_and_determinism():
    P = orc.make_sketch(7, 128, 48)
    assert P.dtype == np.float32 and P.shape == (128, 48)
    np.testing.assert_array_equal(P, orc.make_sketch(7, 128, 48))
    assert not np.array_equal(P, orc.make_sketch(8, 128, 48))
    z = P.astype(np.float64) * math.sqrt(48)
    assert abs(z.mean()) < 0.05 and abs(z.std() - 1.0) < 0.05
    assert abs(np.mean(z ** 4) - 3.0) < 0.3                # Gaussian fourth moment
    # first word of the splitmix64 stream for seed 0 is the published test value of that generator
    x = (0 + 0x9E3779B97F4A7C15) & (2 ** 64 - 1)
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & (2 ** 64 - 1)
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & (2 ** 64 - 1)
    x ^= x >> 31
    assert x == 0xE220A8397B1DCDAF


def test_srht_sketch_structure():
    P = orc.make_sketch_srht(5, 128, 48).astype(np.float64)
    assert P.shape == (128, 48)
    np.testing.assert_allclose(np.abs(P), 1 / math.sqrt(48))                  # entries are +-1/sqrt(m)
    np.testing.assert_allclose(P.T @ P, (128 / 48) * np.eye(48), atol=1e-9)    # distinct Hadamard columns are orthogonal
    assert not np.array_equal(P, orc.make_sketch_srht(6, 128, 48))
    # m = d: D H R^T is a scaled orthogonal matrix, so Algorithm 1 returns the exact leverage scores
    K = _rng(14).standard_normal((300, 16)) * (np.arange(1, 17) ** -1.0)
    np.testing.assert_allclose(orc.approx_leverage_scores(K, orc.make_sketch_srht(1, 16, 16)),
                               orc.exact_leverage_scores(K), rtol=1e-8)


# ----------------------------------------------------------------------------- attention term (Eq. 5)
def test_attention_scores_pins():
    import torch
    rng = _rng(12)
    n, d, G = 37, 8, 3
    Q = rng.standard_normal((G, n, d)); K = rng.standard_normal((n, d))
    # one chunk covering the sequence: the unchunked definition a = 1^T softmax(Q K^T), via a library softmax
    want = sum(torch.softmax(torch.from_numpy(Q[g] @ K.T * 0.5), dim=1).sum(dim=0).numpy() for g in range(G))
    np.testing.assert_allclose(orc.attention_scores(Q, K, chunk=64, scale=0.5), want, rtol=1e-12)
    # every query row spreads a mass of one over its chunk: total = G * n, per chunk = G * chunk length
    a = orc.attention_scores(Q, K, chunk=10, scale=0.5)
    assert abs(a.sum() - G * n) < 1e-9
    np.testing.assert_allclose([a[i:i + 10].sum() for i in range(0, n, 10)], [30, 30, 30, 21], rtol=1e-12)
    # zero queries: uniform attention, every key of a full chunk receives G
    np.testing.assert_allclose(orc.attention_scores(np.zeros((G, n, d)), K, chunk=10), np.full(n, float(G)), rtol=1e-12)
    # chunks are independent: changing keys and queries of chunk 0 leaves the other chunks' scores alone
    K2, Q2 = K.copy(), Q.copy(); K2[:10] += 1.0; Q2[:, :10] *= -2.0
    np.testing.assert_allclose(orc.attention_scores(Q2, K2, chunk=10, scale=0.5)[10:], a[10:], rtol=1e-12)
    # permuting the tokens of one chunk permutes its scores
    perm = np.arange(n); perm[10:20] = 10 + rng.permutation(10)
    np.testing.assert_allclose(orc.attention_scores(Q[:, perm], K[perm], chunk=10, scale=0.5), a[perm], rtol=1e-12)
    # two tokens, one channel, by hand: rows (x1, x2), keys (k1, k2)
    x, k = np.array([0.3, -1.2]), np.array([2.0, 0.5])
    p = lambda q: np.exp(q * k) / np.exp(q * k).sum()
    np.testing.assert_allclose(orc.attention_scores(x[None, :, None], k[:, None], chunk=2), p(x[0]) + p(x[1]), rtol=1e-13)
    # a key aligned with every query collects nearly all the mass of its chunk
    Kbig = 0.01 * rng.standard_normal((20, d)); Qpos = np.abs(rng.standard_normal((1, 20, d))) + 1.0
    Kbig[7] = 10.0
    a_big = orc.attention_scores(Qpos, Kbig, chunk=20)
    assert a_big.argmax() == 7 and a_big[7] > 19.9
    # pooling: centred mean with zero padding; window 1 is the identity
    base = orc.attention_scores(Q, K, chunk=10, scale=0.5)
    pooled = orc.attention_scores(Q, K, chunk=10, scale=0.5, pool=3)
    assert abs(pooled[5] - base[4:7].mean()) < 1e-12 and abs(pooled[0] - base[:2].sum() / 3) < 1e-12
    assert abs(pooled[-1] - base[-2:].sum() / 3) < 1e-12


# ----------------------------------------------------------------------------- blend (Eq. 6)
def test_blend_properties():
    rng = _rng(9)
    a = np.exp(rng.standard_normal(500)); o = rng.random(500)
    s = orc.blend(a, o, 0.3)
    za = (a - a.mean()) / a.std(); zo = (o - o.mean()) / o.std()
    np.testing.assert_allclose(s, za + 0.3 * zo, rtol=1e-12)
    assert abs(s.mean()) < 1e-12
    # affine changes of either term leave s unchanged
    np.testing.assert_allclose(orc.blend(3 * a + 2, 0.5 * o - 1, 0.3), s, atol=1e-10)
    # lambda -> 0 ranks like a; constant a ranks like o; no a returns o
    assert np.array_equal(np.argsort(orc.blend(a, o, 0.0)), np.argsort(a))
    assert np.array_equal(np.argsort(orc.blend(np.full(500, 2.0), o, 0.3)), np.argsort(o))
    np.testing.assert_array_equal(orc.blend(None, o, 0.3), o)
    # a term that is constant up to rounding has no z-score: the leverage scores of a sequence no longer than the sketch
    # are all one, through an SVD they come out as 1 +- 1e-15, and the blend must then be z(a) alone
    ones = 1.0 + 1e-15 * rng.standard_normal(500)
    np.testing.assert_allclose(orc.blend(a, ones, 0.3), za, rtol=1e-12)
    np.testing.assert_allclose(orc.blend(ones, o, 0.3), 0.3 * zo, rtol=1e-12)
    few = rng.standard_normal((30, 128))                 # 30 tokens, sketch of 48: every score is one
    lev = orc.approx_leverage_scores(few, orc.make_sketch(1, 128, 48))
    a30 = rng.random(30)
    np.testing.assert_allclose(orc.blend(a30, lev, 0.3), (a30 - a30.mean()) / a30.std(), rtol=1e-9)
    # hand example: a = (1,3), o = (0,2): z = (-1,1) for both
    np.testing.assert_allclose(orc.blend([1.0, 3.0], [0.0, 2.0], 0.5), [-1.5, 1.5], atol=1e-15)


# ----------------------------------------------------------------------------- keep count / r*
def test_keep_count_golden():
    for line in open(os.path.join(GOLDEN, "keep_counts.txt")):
        if line.startswith("#") or not line.strip():
            continue
        n, r, want = line.split()
        assert orc.keep_count(int(n), float(r)) == int(want)
    assert orc.keep_count(0, 0.5) == 0 and orc.keep_count(5, 1e-9) == 1 and orc.keep_count(5, 1.0) == 5


def test_calibrated_ratio():
    for line in open(os.path.join(GOLDEN, "calibrated_ratio.txt")):
        if line.startswith("#") or not line.strip():
            continue
        b, tau, want = map(float, line.split())
        assert abs(orc.calibrated_ratio(1.0, b, 0.0, tau) - want) < 1e-6
        assert abs(orc.calibrated_ratio(2.0, b / 4, b / 2, tau) - want) < 1e-6       # b = alpha nll + beta
    for b in (-12.0, -3.0, -0.5, 1e-9, 0.7, 5.0):
        assert abs(orc.calibration_curve(1.0, b) - 1.0) < 1e-12           # f(1) = 1
        assert abs(orc.calibration_curve(0.0, b)) < 1e-12                 # f(0) = 0
        for tau in (0.5, 0.9, 0.95, 1.0):
            r = orc.calibrated_ratio(1.0, b, 0.0, tau)
            assert 0.0 < r <= 1.0
            assert abs(orc.calibration_curve(r, b) - tau) < 1e-7          # f(r*) = tau
    assert orc.calibrated_ratio(1.0, 0.0, 0.0, 0.9) == 0.9                # b = 0: the straight line
    # more compressible (more negative b) => smaller r*
    assert orc.calibrated_ratio(1.0, -10, 0, 0.95) < orc.calibrated_ratio(1.0, -4, 0, 0.95)


def test_nll_pins():
    rng = _rng(61)
    # equal logits: every token has probability 1/V
    np.testing.assert_allclose(orc.token_nll(np.full((3, 50), 2.5), [0, 7, 49]), np.full(3, math.log(50)), rtol=1e-14)
    # two-way softmax is the logistic function: -log sigmoid(a - b)
    a, b = 1.3, -0.4
    np.testing.assert_allclose(orc.token_nll([[a, b]], [0]), [math.log1p(math.exp(b - a))], rtol=1e-14)
    np.testing.assert_allclose(orc.token_nll([[a, b]], [1]), [math.log1p(math.exp(a - b))], rtol=1e-14)
    # a dominant logit: picking it costs nothing, picking another costs the gap
    row = np.zeros(10); row[4] = 800.0
    np.testing.assert_allclose(orc.token_nll([row, row], [4, 2]), [0.0, 800.0], atol=1e-12)
    # brute force against probabilities multiplied out, and invariance under a shift of a row
    x = rng.standard_normal((6, 9)) * 3
    t = rng.integers(0, 9, size=6)
    p = np.exp(x) / np.sum(np.exp(x), axis=1, keepdims=True)
    want = -np.log(p[np.arange(6), t])
    np.testing.assert_allclose(orc.token_nll(x, t), want, rtol=1e-12)
    np.testing.assert_allclose(orc.token_nll(x + 1000.0, t), want, rtol=1e-9)
    assert abs(orc.mean_nll(x, t) - want.mean()) < 1e-12
    # the probabilities of all targets of one row sum to one
    full = np.tile(x[0], (9, 1))
    assert abs(np.sum(np.exp(-orc.token_nll(full, np.arange(9)))) - 1.0) < 1e-12
    # unscored rows: excluded from the average, and an average over nothing is 0
    t2 = t.copy(); t2[[1, 4]] = -1
    assert abs(orc.mean_nll(x, t2) - want[[0, 2, 3, 5]].mean()) < 1e-12
    assert orc.token_nll(x, t2)[1] == 0.0
    assert orc.mean_nll(x, np.full(6, -1)) == 0.0


def test_fit_calibration_recovers_known_parameters():
    rng = _rng(15)
    alpha, beta = -1.7, -0.8
    nll = rng.uniform(0.5, 3.0, 60); r = rng.uniform(0.05, 1.0, 60)
    y = np.array([orc.calibration_curve(ri, alpha * ci + beta) for ri, ci in zip(r, nll)])
    a, b, loss = orc.fit_calibration(r, nll, y)
    assert abs(a - alpha) < 1e-4 and abs(b - beta) < 1e-4 and loss < 1e-12     # noise-free triples: exact recovery
    assert orc.calibration_loss(alpha, beta, r, nll, y) < 1e-30
    # with noise, weighting over-predicted quality more moves the curve down: larger r* for the same tau
    y_noisy = np.clip(y + 0.05 * rng.standard_normal(60), 0.0, 1.0)
    a1, b1, _ = orc.fit_calibration(r, nll, y_noisy, under_weight=1.0)
    a4, b4, _ = orc.fit_calibration(r, nll, y_noisy, under_weight=8.0)
    r1 = np.mean([orc.calibrated_ratio(c, a1, b1, 0.9) for c in (1.0, 2.0)])
    r4 = np.mean([orc.calibrated_ratio(c, a4, b4, 0.9) for c in (1.0, 2.0)])
    assert r4 > r1
    # the loss counts a positive residual `under_weight` times
    assert abs(orc.calibration_loss(0.0, 0.0, [0.5], [1.0], [0.4], 3.0) - 3.0 * 0.01) < 1e-12
    assert abs(orc.calibration_loss(0.0, 0.0, [0.5], [1.0], [0.6], 3.0) - 0.01) < 1e-12


# ----------------------------------------------------------------------------- top-k
def _brute_topk(s, kk):
    order = sorted(range(len(s)), key=lambda i: (-s[i], i))
    return sorted(order[:kk])


def test_topk_exhaustive_small_with_ties():
    for n in range(1, 7):
        for s in itertools.product([0.0, 1.0, 2.0], repeat=n):
            for kk in range(1, n + 1):
                assert orc.top_k_indices(np.array(s), kk).tolist() == _brute_topk(s, kk)


def test_topk_random_and_edges():
    rng = _rng(10)
    s = np.round(rng.random(3000), 2)                     # many ties
    for kk in (1, 2, 1500, 2999, 3000):
        got = orc.top_k_indices(s, kk)
        assert got.dtype == np.int32 and got.tolist() == _brute_topk(s.tolist(), kk)
    assert orc.top_k_indices(np.full(10, 0.5), 4).tolist() == [0, 1, 2, 3]
    assert orc.top_k_indices(np.array([-1.0, -3.0, -2.0]), 2).tolist() == [0, 2]


def test_topk_across_heads_brute_force():
    rng = _rng(13)
    for H, n, budget in ((2, 5, 4), (3, 7, 10), (4, 6, 1), (3, 4, 12), (2, 9, 9)):
        for trial in range(20):
            S = np.round(rng.random((H, n)), 1)           # many ties, also across heads
            got = orc.top_k_across_heads(S, budget)
            triples = sorted(((-S[h, i], h, i) for h in range(H) for i in range(n)))[:budget]
            want = [sorted(i for (_, hh, i) in triples if hh == h) for h in range(H)]
            assert [g.tolist() for g in got] == want
            assert sum(len(g) for g in got) == budget
    # one head far above the others takes the whole budget; equal heads split like per-head selection
    S = np.stack([np.linspace(10, 11, 8), np.linspace(0, 1, 8)])
    assert [g.tolist() for g in orc.top_k_across_heads(S, 8)] == [list(range(8)), []]
    S = np.tile(rng.permutation(8).astype(float), (3, 1))
    per_head = orc.top_k_indices(S[0], 3).tolist()
    assert [g.tolist() for g in orc.top_k_across_heads(S, 9)] == [per_head] * 3


# ----------------------------------------------------------------------------- compaction / whole unit
def test_compact_and_compress_unit():
    import torch
    rng = _rng(11)
    n, d, m = 300, 128, 48
    K = torch.randn(n, d).to(torch.bfloat16); V = torch.randn(n, d).to(torch.bfloat16)
    kb, vb = K.view(torch.int16).numpy(), V.view(torch.int16).numpy()
    Phi = (rng.standard_normal((d, m)) / math.sqrt(m)).astype(np.float32)
    s, idx, Kc, Vc = orc.compress_unit(kb, kb, vb, Phi, orc.keep_count(n, 0.3))
    assert len(idx) == 90 and np.all(np.diff(idx) > 0)
    np.testing.assert_array_equal(Kc, kb[idx]); np.testing.assert_array_equal(Vc, vb[idx])
    assert s[idx].min() >= np.delete(s, idx).max()
    assert abs(s.sum() - m) < 1e-8

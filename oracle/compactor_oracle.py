"""CPU oracle for Compactor's prefill-time compression pass.  TEST INFRASTRUCTURE.

A plain, slow, fp64 numpy statement of what the pass computes, written from the
paper so that a reader can check it by eye.  It shares nothing with the CUDA
library (no code, tables, constants or pre/post-processing) and must only be
used by the tests, the smoke check and the benchmark's CPU-baseline leg -
never by the product path.

What follows the paper step by step:
  * `approx_leverage_scores` - Algorithm 1 (Gaussian right sketch, Gram matrix,
    small SVD, back-projection, squared row norms).
  * `exact_leverage_scores`  - Definition 1 / Eq. 1 (the quantity Algorithm 1
    approximates; used to pin the oracle, and as the m = d special case).
  * `approx_leverage_scores_eig`, `approx_leverage_scores_qr` - Appendix C's
    two other routes to the same scores (eigendecomposition of G with clamped
    eigenvalues; reduced QR of K Phi).
  * `attention_scores`       - Eq. 5 (column sums of chunked non-causal softmax
    attention, mean-pooled).
  * `blend`                  - Eq. 6 (z-scored attention term + lambda * z-scored
    outlier term).
  * `keep_count`             - the number of retained tokens, ceil(r N) (Section 3,
    Preliminaries; Section 3.4).
  * `top_k_indices`          - per-head top-k of the scores.
  * `top_k_across_heads`     - the same budget spent over all heads of a layer
    (Section 3.4's alternative; ties: lower head, then lower index).
  * `compact`                - the retained rows of K and V.
  * `token_nll`, `mean_nll`  - the token-averaged negative log-likelihood of
    Section 3.5, from logits and target ids.
  * `calibrated_ratio`       - inverse of the fitted curve f_{alpha,beta}
    (Section 3.5); `fit_calibration` - the asymmetric least-squares fit of
    (alpha, beta) on (r, NLL, y) triples.

Readings taken where the paper is silent or inconsistent:
  * Eq. 1 prints diag(U^T U); Definition 1 and Algorithm 1's last line make it
    the squared row norms diag(U U^T).
  * Sigma^-1 in Algorithm 1 is a pseudo-inverse: singular directions of G with
    lambda_j <= m * 2^-52 * lambda_max contribute nothing (Algorithm 1 has no
    clamp; the 1e-6 clamp appears only in Appendix C's eigen variant).
  * Entries of Phi have variance 1/m (Algorithm 1, line 1); the scale does not
    change the scores.
  * Ties in the top-k go to the lower token index, and the kept indices are
    emitted in ascending order (the paper does not say).
  * std in Eq. 6 is the population standard deviation; a term without spread
    (std <= 1e-3 |mean|: constant up to what the scores resolve) contributes 0.
    With no attention term the score is the outlier score o.
  * The calibration curve is increasing in r; the paper writes the choice of
    r* as an arg max subject to f >= tau, which is read as the smallest such r
    (Section 3.5 states the goal as the least retention that keeps quality).

  * Eq. 5 details (softmax scale, last chunk, grouped queries, pooling window)
    are not given by the paper; `attention_scores` states the reading taken.

Pins (see tests/test_oracle_pins.py): closed-form leverage scores, sum = rank,
range [0,1], invariance under K -> K A and Phi -> Phi A, m = d reduces to the
exact scores, Phi = e_1, n <= m gives all ones, agreement with a QR route
(Appendix C), brute-force top-k, f(r*) = tau.  Agreement with the authors'
own engine outputs is "parity unpinned": the paper prints no score values,
indices or worked example for this path.
"""
from __future__ import annotations

import math

import numpy as np


# ----------------------------------------------------------------------------
# Input widening (data handling only)
# ----------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16 / int16) exactly to float64."""
    u = np.ascontiguousarray(bits).view(np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------
# Algorithm 1, line 1: the Gaussian sketch from a seed
# ----------------------------------------------------------------------------
def make_sketch(seed: int, d: int, m: int) -> np.ndarray:
    """Phi [d, m] fp32 with iid N(0, 1/m) entries from a counter-based generator:
    word i (i = 0, 1, ...) is the splitmix64 finaliser of seed + (i+1)*0x9E3779B97F4A7C15;
    words (2p, 2p+1) give u1 = ((x >> 11) + 1) 2^-53 in (0,1] and u2 = (x >> 11) 2^-53 in
    [0,1); Box-Muller turns them into the row-major entries 2p and 2p+1; each is divided by
    sqrt(m) in double and rounded to fp32."""
    count = d * m
    pairs = (count + 1) // 2
    mask = (1 << 64) - 1

    def word(i):
        z = (seed + (i + 1) * 0x9E3779B97F4A7C15) & mask
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & mask
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & mask
        return z ^ (z >> 31)

    out = np.empty(2 * pairs, dtype=np.float64)
    for p in range(pairs):
        u1 = ((word(2 * p) >> 11) + 1) * 2.0 ** -53
        u2 = (word(2 * p + 1) >> 11) * 2.0 ** -53
        rad = math.sqrt(-2.0 * math.log(u1))
        out[2 * p] = rad * math.cos(2.0 * math.pi * u2)
        out[2 * p + 1] = rad * math.sin(2.0 * math.pi * u2)
    return (out[:count] / math.sqrt(m)).astype(np.float32).reshape(d, m)


def make_sketch_srht(seed: int, d: int, m: int) -> np.ndarray:
    """Appendix D: subsampled randomised Hadamard sketch Phi = c * D H R^T as an explicit [d, m] matrix
    (D random signs, H the Sylvester-Walsh-Hadamard matrix, R a choice of m columns without
    replacement).  The constant is 1/sqrt(m), which gives entries the variance of the Gaussian
    sketch; scores do not depend on it.  Random bits come from the same splitmix64 stream as
    `make_sketch`: word i (i < d) gives the sign of row i (bit 0: 1 = minus); word d + j drives step
    j of a Fisher-Yates shuffle of 0..d-1 whose first m entries are the chosen columns."""
    assert d & (d - 1) == 0 and 1 <= m <= d
    mask = (1 << 64) - 1

    def word(i):
        z = (seed + (i + 1) * 0x9E3779B97F4A7C15) & mask
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & mask
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & mask
        return z ^ (z >> 31)

    sign = np.array([-1.0 if word(i) & 1 else 1.0 for i in range(d)])
    perm = list(range(d))
    for j in range(m):
        r = j + word(d + j) % (d - j)
        perm[j], perm[r] = perm[r], perm[j]
    H = np.array([[1.0]])
    while H.shape[0] < d:
        H = np.block([[H, H], [H, -H]])
    Phi = (sign[:, None] * H[:, perm[:m]]) / math.sqrt(m)
    return Phi.astype(np.float32)


# ----------------------------------------------------------------------------
# Definition 1 / Eq. 1: exact leverage scores
# ----------------------------------------------------------------------------
def exact_leverage_scores(K: np.ndarray) -> np.ndarray:
    """l_i = ||U_i||^2 with K = U Sigma V^T the thin SVD, U restricted to the
    numerically non-zero singular values (Definition 1)."""
    K = np.asarray(K, dtype=np.float64)
    n, d = K.shape
    if n == 0:
        return np.zeros(0)
    U, sig, _ = np.linalg.svd(K, full_matrices=False)
    if sig.size == 0 or sig[0] == 0.0:
        return np.zeros(n)
    rank = int(np.sum(sig > max(n, d) * np.finfo(np.float64).eps * sig[0]))
    return np.sum(U[:, :rank] ** 2, axis=1)


# ----------------------------------------------------------------------------
# Algorithm 1: approximate leverage scores
# ----------------------------------------------------------------------------
def approx_leverage_scores(K: np.ndarray, Phi: np.ndarray) -> np.ndarray:
    """Algorithm 1, lines 2-6, for a given sketch Phi [d, m] (line 1 is the
    caller's draw of Phi)."""
    K = np.asarray(K, dtype=np.float64)
    Phi = np.asarray(Phi, dtype=np.float64)
    n = K.shape[0]
    m = Phi.shape[1]
    if n == 0:
        return np.zeros(0)
    K_hat = K @ Phi                                   # line 2
    G = K_hat.T @ K_hat                               # line 3
    V_t, lam, _ = np.linalg.svd(G)                    # line 4: G = V Sigma^2 V^T
    lam_max = lam[0] if lam.size else 0.0
    if lam_max <= 0.0:
        return np.zeros(n)
    keep = lam > m * 2.0 ** -52 * lam_max             # pseudo-inverse of Sigma
    sigma = np.sqrt(lam[keep])
    U_t = (K_hat @ V_t[:, keep]) / sigma[None, :]     # line 5
    return np.sum(U_t * U_t, axis=1)                  # line 6: diag(U U^T)


def approx_leverage_scores_eig(K: np.ndarray, Phi: np.ndarray, eps: float = 1e-6) -> np.ndarray:
    """Appendix C, eigendecomposition route: G = V Lambda V^T, every eigenvalue raised to at
    least eps (an absolute floor on the eigenvalues of G, so the result depends on the scale
    of K Phi once the floor is active), U~ = K^ V Lambda^-1/2, scores = squared row norms."""
    K = np.asarray(K, dtype=np.float64)
    Phi = np.asarray(Phi, dtype=np.float64)
    if K.shape[0] == 0:
        return np.zeros(0)
    K_hat = K @ Phi
    G = K_hat.T @ K_hat
    lam, V = np.linalg.eigh(G)
    lam = np.maximum(lam, float(eps))
    U_t = (K_hat @ V) / np.sqrt(lam)[None, :]
    return np.sum(U_t * U_t, axis=1)


def approx_leverage_scores_qr(K: np.ndarray, Phi: np.ndarray) -> np.ndarray:
    """Appendix C, QR route: K^ = Q R (reduced), scores = squared row norms of Q.  Defined for
    K^ of full column rank; rank-deficient input is left to the routes above."""
    K = np.asarray(K, dtype=np.float64)
    Phi = np.asarray(Phi, dtype=np.float64)
    if K.shape[0] == 0:
        return np.zeros(0)
    Q, _ = np.linalg.qr(K @ Phi, mode="reduced")
    return np.sum(Q * Q, axis=1)


# ----------------------------------------------------------------------------
# Eq. 6: blend
# ----------------------------------------------------------------------------
def _zscore(x: np.ndarray) -> np.ndarray:
    """Population z-score (Eq. 6).  A vector with no spread has no z-score and contributes nothing; "no spread"
    is read numerically: a standard deviation of at most 1e-3 of |mean| is below what the scores are asked to
    resolve (leverage scores of a sequence no longer than the sketch are all one, up to rounding)."""
    mu = np.mean(x)
    sd = np.sqrt(np.mean((x - mu) ** 2))
    if sd <= 1e-3 * abs(mu):
        return np.zeros_like(x)
    return (x - mu) / sd


def blend(a, o: np.ndarray, lam: float) -> np.ndarray:
    """s = z(a) + lam * z(o) (Eq. 6).  With a = None the score is o itself."""
    o = np.asarray(o, dtype=np.float64)
    if a is None:
        return o.copy()
    a = np.asarray(a, dtype=np.float64)
    if o.size == 0:
        return o.copy()
    return _zscore(a) + float(lam) * _zscore(o)


# ----------------------------------------------------------------------------
# Eq. 5: chunked non-causal attention scores
# ----------------------------------------------------------------------------
def attention_scores(Q: np.ndarray, K: np.ndarray, chunk: int = 256, scale: float = 1.0, pool: int = 1) -> np.ndarray:
    """a = concat_i 1^T softmax(Q[i] K[i]^T) over chunks of `chunk` consecutive tokens (Eq. 5),
    followed by mean pooling.

    Q [G, n, d]: the G query heads that share this KV head (their column sums are added);
    K [n, d].  Readings where the paper is silent: logits are multiplied by `scale` before the
    softmax (Eq. 5 prints none; 1/sqrt(d) is the usual choice); the last, shorter chunk is a
    softmax over its own keys; pooling is a centred window of `pool` (odd) tokens over the
    concatenated vector, zero beyond the ends of the sequence, divided by `pool`."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    if Q.ndim == 2:
        Q = Q[None]
    n = K.shape[0]
    a = np.zeros(n)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        for g in range(Q.shape[0]):
            S = (Q[g, lo:hi] @ K[lo:hi].T) * float(scale)
            S = S - S.max(axis=1, keepdims=True)
            P = np.exp(S)
            P /= P.sum(axis=1, keepdims=True)
            a[lo:hi] += P.sum(axis=0)                     # 1^T softmax(...)
    if pool > 1:
        half = pool // 2
        padded = np.concatenate([np.zeros(half), a, np.zeros(half)])
        a = np.array([padded[i:i + pool].sum() / pool for i in range(n)])
    return a


# ----------------------------------------------------------------------------
# Selection
# ----------------------------------------------------------------------------
def keep_count(n: int, r: float) -> int:
    """ceil(r * n) evaluated in double precision, clamped to [1, n] (0 if n = 0)."""
    n = int(n)
    if n <= 0:
        return 0
    return min(n, max(1, int(math.ceil(float(r) * float(n)))))


def top_k_indices(s: np.ndarray, kk: int) -> np.ndarray:
    """Indices of the kk largest scores; equal scores are ranked by lower index
    first; result in ascending index order."""
    s = np.asarray(s)
    n = s.shape[0]
    kk = int(kk)
    order = np.lexsort((np.arange(n), -s))            # primary key -s, then index
    return np.sort(order[:kk]).astype(np.int32)


def top_k_across_heads(S: np.ndarray, budget: int):
    """Selection across the heads of one layer (Section 3.4 allows the top scores to be taken over
    all heads instead of per head): S [H, n] holds the heads' scores of one sequence; the `budget`
    largest entries are kept, ranked by (score descending, head ascending, index ascending).
    Returns one ascending index array per head; their lengths add up to `budget`."""
    S = np.asarray(S)
    H, n = S.shape
    budget = int(budget)
    heads = np.repeat(np.arange(H), n)
    idxs = np.tile(np.arange(n), H)
    order = np.lexsort((idxs, heads, -S.reshape(-1)))      # primary -score, then head, then index
    chosen = order[:budget]
    return [np.sort(idxs[chosen][heads[chosen] == h]).astype(np.int32) for h in range(H)]


def compact(K_bits: np.ndarray, V_bits: np.ndarray, idx: np.ndarray):
    """K'[j] = K[idx[j]], V'[j] = V[idx[j]] as bit copies."""
    idx = np.asarray(idx, dtype=np.int64)
    return K_bits[idx].copy(), V_bits[idx].copy()


# ----------------------------------------------------------------------------
# Section 3.5: context-calibrated ratio
# ----------------------------------------------------------------------------
def token_nll(logits: np.ndarray, targets: np.ndarray) -> np.ndarray:
    """-log softmax(logits_i)[targets_i] for every row i (Section 3.5: the summand of the
    token-averaged NLL).  Rows whose target is negative are not scored and give 0."""
    x = np.asarray(logits, dtype=np.float64)
    t = np.asarray(targets, dtype=np.int64)
    out = np.zeros(x.shape[0])
    for i in range(x.shape[0]):
        if t[i] < 0:
            continue
        row = x[i]
        top = np.max(row)
        log_z = top + math.log(float(np.sum(np.exp(row - top))))     # log of the softmax denominator
        out[i] = log_z - row[t[i]]
    return out


def mean_nll(logits: np.ndarray, targets: np.ndarray) -> float:
    """NLL(t; c) = -(1/L) sum_i log LM(t_i | ...) (Section 3.5), L counting the scored rows;
    0 when no row is scored."""
    t = np.asarray(targets, dtype=np.int64)
    scored = int(np.sum(t >= 0))
    if scored == 0:
        return 0.0
    return float(np.sum(token_nll(logits, targets)) / scored)


def calibration_curve(r: float, b: float) -> float:
    """f(r) = (exp(r b - b) - exp(-b)) / (1 - exp(-b)); f(r) = r in the limit b -> 0."""
    if b == 0.0:
        return float(r)
    return (math.exp(r * b - b) - math.exp(-b)) / (1.0 - math.exp(-b))


def calibrated_ratio(nll: float, alpha: float, beta: float, tau: float) -> float:
    """The r in (0,1] with f_{alpha,beta}(r) = tau, b = alpha * nll + beta:
    r* = log(1 + tau (e^b - 1)) / b, and r* = tau when b = 0."""
    b = float(alpha) * float(nll) + float(beta)
    if b == 0.0:
        return float(tau)
    return math.log1p(float(tau) * math.expm1(b)) / b


def calibration_loss(alpha: float, beta: float, r, nll, y, under_weight: float = 1.0) -> float:
    """Asymmetric mean squared error of the fitted curve (Section 3.5): residual e_i =
    f_{alpha,beta}(r_i, NLL_i) - y_i; a positive residual predicts more quality than was measured,
    which would make r* too small, and is weighted by `under_weight` >= 1 (the paper says such
    errors are weighted higher but not by how much)."""
    r = np.asarray(r, dtype=np.float64); nll = np.asarray(nll, dtype=np.float64); y = np.asarray(y, dtype=np.float64)
    total = 0.0
    for ri, ci, yi in zip(r, nll, y):
        e = calibration_curve(float(ri), alpha * float(ci) + beta) - float(yi)
        total += (under_weight if e > 0.0 else 1.0) * e * e
    return total / max(1, r.size)


def fit_calibration(r, nll, y, under_weight: float = 1.0):
    """(alpha, beta) minimising `calibration_loss` over the training triples (r_i, NLL_i, y_i): a
    derivative-free simplex search from a coarse grid of starting points (slow and plain)."""
    from scipy.optimize import minimize
    best = None
    for a0 in (-4.0, -1.0, 0.0, 1.0):
        for b0 in (-6.0, -2.0, 0.5):
            res = minimize(lambda p: calibration_loss(p[0], p[1], r, nll, y, under_weight), x0=[a0, b0],
                           method="Nelder-Mead", options={"xatol": 1e-10, "fatol": 1e-16, "maxiter": 4000})
            if best is None or res.fun < best.fun:
                best = res
    return float(best.x[0]), float(best.x[1]), float(best.fun)


# ----------------------------------------------------------------------------
# The whole pass for one unit
# ----------------------------------------------------------------------------
def compress_unit(K_score_bits, K_cache_bits, V_bits, Phi, kk, attn=None, lam=0.3):
    """Score, select and compact one (sequence, layer, head) unit.

    *_bits are bf16 bit patterns [n, d] (uint16); Phi fp32/fp64 [d, m]; attn an
    optional fp32 [n].  Returns (scores fp64 [n], idx int32 [kk], K' bits, V' bits)."""
    K = bf16_bits_to_f64(np.asarray(K_score_bits))
    o = approx_leverage_scores(K, np.asarray(Phi, dtype=np.float64))
    s = blend(None if attn is None else np.asarray(attn, dtype=np.float64), o, lam)
    idx = top_k_indices(s, kk)
    Kc, Vc = compact(np.asarray(K_cache_bits), np.asarray(V_bits), idx)
    return s, idx, Kc, Vc

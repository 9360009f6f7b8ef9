"""GPU parity of the scorer's variants (Appendix C): the eigendecomposition route with its
eigenvalue floor, and the Cholesky route read as the appendix's QR route."""
import numpy as np
import pytest
import torch

from paper_2507_08143_b200 import inputs
from oracle import compactor_oracle as orc
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2507_08143_b200 import binding
    return binding


def _score_variant(B, w, factorization, floor, phi_scale=1.0):
    _, kr, _ = inputs.make_tensors(w, device="cpu", want_pre=False)
    kr = kr.cuda()
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, w.seed) * phi_scale
    ws = torch.empty(B.workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    scores = torch.full((w.layers, w.heads, sum(w.seqlens)), -1.0, dtype=torch.float32, device="cuda")
    status = torch.full((w.layers * w.heads * len(w.seqlens),), -1, dtype=torch.int32, device="cuda")
    B.score_variant(shape, kr, phi.cuda(), scores, ws, factorization, floor, status=status)
    torch.cuda.synchronize()
    return kr.cpu(), phi.double().numpy(), scores.cpu().numpy(), status.cpu().numpy().reshape(w.layers, w.heads, -1)


def _units(w):
    cu = np.concatenate([[0], np.cumsum(w.seqlens)])
    for layer in range(w.layers):
        for head in range(w.heads):
            for b, n in enumerate(w.seqlens):
                yield layer, head, b, int(cu[b]), int(n)


def _bits(k, layer, head, t0, n):
    return k[layer, head, t0:t0 + n].view(torch.int16).numpy().view(np.uint16)


def test_eig_route_with_inactive_floor_matches_algorithm_1(B):
    w = inputs.Workload("eig-inactive", 2, 2, 128, [1500, 260, 4100], [0.3, 0.3, 0.3], p=0.7, seed=31)
    k, phi, got, status = _score_variant(B, w, B.FACTOR_EIG, 1e-6)
    worst = 0.0
    for layer, head, b, t0, n in _units(w):
        K = orc.bf16_bits_to_f64(_bits(k, layer, head, t0, n))
        want_eig = orc.approx_leverage_scores_eig(K, phi, 1e-6)
        want = orc.approx_leverage_scores(K, phi)
        np.testing.assert_allclose(want_eig, want, rtol=1e-6)            # the floor is far below the spectrum here
        g = got[layer, head, t0:t0 + n]
        err = np.max(np.abs(g - want_eig) / np.maximum(np.abs(want_eig), 1e-30))
        worst = max(worst, err)
        assert status[layer, head, b] == 0
    print(f"eig route, inactive floor: max rel err {worst:.2e}")
    assert worst <= H.SCORE_RTOL


@pytest.mark.parametrize("frac", [1e-3, 0.05, 10.0])
def test_eig_route_with_active_floor(B, frac):
    # A floor inside (or above) the spectrum of G: the scores are no longer leverage scores, and the
    # library has to make the same change the oracle makes.  The floor is set from the spectrum the
    # oracle sees, as a fraction of the largest eigenvalue of the first unit's G.
    w = inputs.Workload("eig-active", 1, 2, 128, [2000, 700], [0.3, 0.3], p=1.0, seed=32)
    _, kr, _ = inputs.make_tensors(w, device="cpu", want_pre=False)
    phi0 = inputs.make_sketch_matrix(w.d, w.m, w.seed).double().numpy()
    K0 = orc.bf16_bits_to_f64(_bits(kr, 0, 0, 0, w.seqlens[0])) @ phi0
    floor = float(frac * np.linalg.eigvalsh(K0.T @ K0)[-1])
    k, phi, got, status = _score_variant(B, w, B.FACTOR_EIG, floor)
    worst = 0.0
    for layer, head, b, t0, n in _units(w):
        K = orc.bf16_bits_to_f64(_bits(k, layer, head, t0, n))
        want = orc.approx_leverage_scores_eig(K, phi, floor)
        g = got[layer, head, t0:t0 + n]
        worst = max(worst, np.max(np.abs(g - want) / np.maximum(np.abs(want), 1e-30)))
        lam = np.linalg.eigvalsh((K @ phi).T @ (K @ phi))
        assert (status[layer, head, b] & 2) == (2 if lam[0] < floor else 0)
    print(f"eig route, floor {frac} of lambda_max: max rel err {worst:.2e}")
    assert worst <= H.SCORE_RTOL


def test_eig_floor_makes_scores_depend_on_the_sketch_scale(B):
    # Algorithm 1 is invariant under Phi -> c Phi; the floored route is not: G scales by c^2.
    w = inputs.Workload("eig-scale", 1, 1, 128, [1200], [0.3], p=1.0, seed=33)
    k, phi, got, _ = _score_variant(B, w, B.FACTOR_EIG, 1e-2, phi_scale=1e-3)
    K = orc.bf16_bits_to_f64(_bits(k, 0, 0, 0, 1200))
    want = orc.approx_leverage_scores_eig(K, phi, 1e-2)
    plain = orc.approx_leverage_scores(K, phi)
    assert np.max(np.abs(want - plain) / plain) > 0.05                 # the floor really is active
    np.testing.assert_allclose(got[0, 0], want, rtol=H.SCORE_RTOL)


def test_cholesky_variant_is_the_qr_route_and_the_default(B):
    w = inputs.Workload("chol-qr", 1, 2, 128, [900, 3000], [0.3, 0.3], p=0.7, seed=34)
    k, phi, got, status = _score_variant(B, w, B.FACTOR_CHOLESKY, 0.0)
    for layer, head, b, t0, n in _units(w):
        K = orc.bf16_bits_to_f64(_bits(k, layer, head, t0, n))
        np.testing.assert_allclose(got[layer, head, t0:t0 + n], orc.approx_leverage_scores_qr(K, phi),
                                   rtol=H.SCORE_RTOL)
    # bit-identical to the plain entry point
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    ws = torch.empty(B.workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    ref = torch.empty((w.layers, w.heads, sum(w.seqlens)), dtype=torch.float32, device="cuda")
    B.score(shape, k.cuda(), torch.from_numpy(phi).float().cuda(), ref, ws)
    torch.cuda.synchronize()
    assert np.array_equal(ref.cpu().numpy(), got)


@pytest.mark.parametrize("m", [7, 16, 33, 64])
def test_eig_route_other_sketch_dimensions(B, m):
    w = inputs.Workload(f"eig-m{m}", 1, 2, 128, [800, 1700], [0.3, 0.3], p=0.7, seed=40 + m, m=m)
    k, phi, got, status = _score_variant(B, w, B.FACTOR_EIG, 1e-6)
    for layer, head, b, t0, n in _units(w):
        K = orc.bf16_bits_to_f64(_bits(k, layer, head, t0, n))
        np.testing.assert_allclose(got[layer, head, t0:t0 + n], orc.approx_leverage_scores_eig(K, phi, 1e-6),
                                   rtol=H.SCORE_RTOL)


def test_variant_argument_checks(B):
    w = inputs.Workload("eig-args", 1, 1, 128, [300], [0.3], p=0.7, seed=35)
    _, kr, _ = inputs.make_tensors(w, device="cpu", want_pre=False)
    shape = B.Shape(1, 1, 128, w.m, w.seqlens)
    ws = torch.empty(B.workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    out = torch.empty((1, 1, 300), dtype=torch.float32, device="cuda")
    phi = inputs.make_sketch_matrix(w.d, w.m, w.seed).cuda()
    for fact, floor in ((2, 1e-6), (-1, 1e-6), (B.FACTOR_EIG, 0.0), (B.FACTOR_EIG, -1.0), (B.FACTOR_EIG, float("nan")),
                        (B.FACTOR_EIG, float("inf"))):
        with pytest.raises(B.CompactorError) as e:
            B.score_variant(shape, kr.cuda(), phi, out, ws, fact, floor)
        assert e.value.code == -1


# ----------------------------------------------------------------------------- m = d: exact leverage scores
def _score_with_phi(B, w, phi):
    _, kr, _ = inputs.make_tensors(w, device="cpu", want_pre=False)
    shape = B.Shape(w.layers, w.heads, w.d, phi.shape[1], w.seqlens)
    ws = torch.empty(B.workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    scores = torch.full((w.layers, w.heads, sum(w.seqlens)), -1.0, dtype=torch.float32, device="cuda")
    status = torch.full((w.layers * w.heads * len(w.seqlens),), -1, dtype=torch.int32, device="cuda")
    B.score(shape, kr.cuda(), phi.cuda(), scores, ws, status=status)
    torch.cuda.synchronize()
    return kr, scores.cpu().numpy(), status.cpu().numpy().reshape(w.layers, w.heads, -1)


@pytest.mark.parametrize("sketch", ["identity", "rotation"])
def test_full_width_sketch_gives_exact_leverage_scores(B, sketch):
    # Definition 1 / Eq. 1 (the "exact" row of the ablation): any invertible 128 x 128 sketch
    # leaves the column space of K unchanged, so Algorithm 1 returns the exact scores.  The second
    # sketch is a well-conditioned one (orthogonal times a mild column scaling): a square Gaussian
    # matrix squares its own condition number into G, below what fp32 Gram sums resolve.
    w = inputs.Workload("exact", 1, 2, 128, [1500, 5000, 300], [0.3, 0.3, 0.3], p=0.5, seed=51)
    if sketch == "identity":
        phi = torch.eye(128)
    else:
        q, _ = torch.linalg.qr(inputs.make_sketch_matrix(128, 128, 51).double())
        phi = (q * torch.linspace(0.5, 2.0, 128, dtype=torch.float64)[None, :]).float()
    k, got, status = _score_with_phi(B, w, phi)
    worst = 0.0
    for layer, head, b, t0, n in _units(w):
        K = orc.bf16_bits_to_f64(_bits(k, layer, head, t0, n))
        want = orc.exact_leverage_scores(K)
        g = got[layer, head, t0:t0 + n]
        worst = max(worst, np.max(np.abs(g - want) / want))
        assert abs(g.sum() - 128.0) < 0.05                              # sum of leverage scores = rank
        assert status[layer, head, b] == 0
    print(f"exact scores ({sketch}): max rel err {worst:.2e}")
    assert worst <= H.SCORE_RTOL


def test_wide_sketch_between_64_and_128_columns(B):
    w = inputs.Workload("m100", 1, 2, 128, [2100, 640], [0.3, 0.3], p=0.5, seed=52, m=100)
    phi = inputs.make_sketch_matrix(128, 100, 52)
    k, got, status = _score_with_phi(B, w, phi)
    for layer, head, b, t0, n in _units(w):
        K = orc.bf16_bits_to_f64(_bits(k, layer, head, t0, n))
        np.testing.assert_allclose(got[layer, head, t0:t0 + n], orc.approx_leverage_scores(K, phi.double().numpy()),
                                   rtol=H.SCORE_RTOL)


def test_exact_scores_of_a_short_rank_deficient_sequence(B):
    # fewer tokens than channels: rank n, every exact score is 1
    w = inputs.Workload("exact-short", 1, 1, 128, [90], [0.5], p=0.5, seed=53)
    k, got, status = _score_with_phi(B, w, torch.eye(128))
    np.testing.assert_allclose(got[0, 0], np.ones(90), rtol=H.SCORE_RTOL)
    assert status[0, 0, 0] & 2                                          # rank deficiency is reported


def test_eig_route_rejects_wide_sketches(B):
    w = inputs.Workload("eig-wide", 1, 1, 128, [300], [0.3], p=0.7, seed=54)
    _, kr, _ = inputs.make_tensors(w, device="cpu", want_pre=False)
    shape = B.Shape(1, 1, 128, 128, w.seqlens)
    ws = torch.empty(B.workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    out = torch.empty((1, 1, 300), dtype=torch.float32, device="cuda")
    with pytest.raises(B.CompactorError) as e:
        B.score_variant(shape, kr.cuda(), torch.eye(128).cuda(), out, ws, B.FACTOR_EIG, 1e-6)
    assert e.value.code == -2


@pytest.mark.parametrize("shift", [-24, 20])
def test_scores_do_not_depend_on_the_scale_of_the_keys(B, shift):
    # K -> 2^shift K is exact in bf16 and in every sum of the Cholesky route: the scores are bit-identical.
    # The eigen route with an inactive floor agrees to rounding (its rotation angles are rounded differently).
    w = inputs.Workload("scale", 1, 2, 128, [3000, 500], [0.3, 0.3], p=0.7, seed=61)
    _, kr, _ = inputs.make_tensors(w, device="cpu", want_pre=False)
    scaled = (kr.float() * 2.0 ** shift).bfloat16()
    assert torch.equal(scaled.float() * 2.0 ** -shift, kr.float())              # the scaling was exact
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, w.seed).cuda()
    ws = torch.empty(B.workspace_bytes(shape), dtype=torch.uint8, device="cuda")
    out = [torch.empty((1, 2, 3500), dtype=torch.float32, device="cuda") for _ in range(4)]
    B.score(shape, kr.cuda(), phi, out[0], ws)
    B.score(shape, scaled.cuda(), phi, out[1], ws)
    floor = 1e-6 * 4.0 ** min(shift, 0)                                          # far below either spectrum
    B.score_variant(shape, kr.cuda(), phi, out[2], ws, B.FACTOR_EIG, floor)
    B.score_variant(shape, scaled.cuda(), phi, out[3], ws, B.FACTOR_EIG, floor)
    torch.cuda.synchronize()
    assert torch.equal(out[0], out[1])
    np.testing.assert_allclose(out[3].cpu().numpy(), out[2].cpu().numpy(), rtol=2e-5)
    np.testing.assert_allclose(out[2].cpu().numpy(), out[0].cpu().numpy(), rtol=2e-4)

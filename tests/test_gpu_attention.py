"""GPU parity of the attention term (Eq. 5) and of the blended pass that consumes it."""
import math

import numpy as np
import pytest
import torch

from oracle import compactor_oracle as orc
from paper_2507_08143_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

# exponentials are rounded to fp16 (2^-11) before the fp32 column sums; logits come from exact bf16 products
RTOL, ATOL = 1e-3, 2e-4


@pytest.fixture(scope="module")
def B():
    from paper_2507_08143_b200 import binding
    return binding


def _attention(B, w, q_per_kv, pool, scale, q=None, k=None):
    if k is None:
        _, k, _ = inputs.make_tensors(w, device="cpu", want_pre=False)
        k = k.cuda()
    if q is None:
        q = inputs.make_queries(w, q_per_kv, device="cpu").cuda()
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    out = torch.full((w.layers, w.heads, shape.total_tokens), float("nan"), dtype=torch.float32, device="cuda")
    ws = B.alloc_workspace(shape)
    status = torch.full((w.layers * w.heads * w.batch,), -1, dtype=torch.int32, device="cuda")
    B.attention_scores(shape, q, k, q_per_kv, out, ws, scale=scale, pool=pool, status=status)
    torch.cuda.synchronize()
    assert int(status.abs().max()) == 0, "no bounded wait may run out in a healthy run (status is cleared by the call)"
    return shape, q, k, out


def _check(w, shape, q, k, out, q_per_kv, pool, scale, units=None):
    cu = shape.cu_seqlens
    todo = units or [(l, h, b) for l in range(w.layers) for h in range(w.heads) for b in range(w.batch)]
    worst = 0.0
    for (l, h, b) in todo:
        sl = slice(cu[b], cu[b + 1])
        if cu[b + 1] == cu[b]:
            continue
        K = orc.bf16_bits_to_f64(H.bits(k[l, h, sl]))
        Q = np.stack([orc.bf16_bits_to_f64(H.bits(q[l, h * q_per_kv + g, sl])) for g in range(q_per_kv)])
        want = orc.attention_scores(Q, K, chunk=256, scale=scale, pool=pool)
        got = out[l, h, sl].cpu().numpy().astype(np.float64)
        err = np.abs(got - want) / (RTOL * np.abs(want) + ATOL)
        assert np.all(err <= 1.0), f"unit {(l, h, b)}: worst {err.max():.2f}x tolerance at {int(err.argmax())}"
        worst = max(worst, float(np.max(np.abs(got - want) / (np.abs(want) + 1e-3))))
    return worst


@pytest.mark.parametrize("q_per_kv,pool", [(1, 1), (4, 1), (4, 7), (5, 3)])
def test_attention_scores_ragged(B, q_per_kv, pool):
    w = inputs.Workload("attn", 2, 2, 128, [1000, 256, 100, 129, 0, 513], [0.5] * 6, p=0.7, seed=81)
    scale = 1.0 / math.sqrt(128)
    shape, q, k, out = _attention(B, w, q_per_kv, pool, scale)
    worst = _check(w, shape, q, k, out, q_per_kv, pool, scale)
    print(f"attention G={q_per_kv} pool={pool}: worst relative error {worst:.2e}")


def test_attention_mass_and_uniform_case(B):
    # every query row spreads a mass of one over its chunk; zero queries give exactly G per key
    w = inputs.Workload("attn-mass", 1, 2, 128, [2048 + 77], [0.5], p=0.7, seed=82)
    G, scale = 3, 0.1
    shape, q, k, out = _attention(B, w, G, 1, scale)
    tot = out.double().sum(dim=2)
    assert torch.all((tot - G * w.seqlens[0]).abs() < 1e-3 * G * w.seqlens[0])
    q0 = torch.zeros_like(q)
    _, _, _, out0 = _attention(B, w, G, 1, scale, q=q0, k=k)
    np.testing.assert_allclose(out0.cpu().numpy(), float(G), rtol=1e-3)


def test_attention_token_major_layout(B):
    w = inputs.Workload("attn-tm", 1, 2, 128, [700], [0.5], p=0.7, seed=83)
    G = 2
    _, k, _ = inputs.make_tensors(w, device="cpu", want_pre=False)
    q = inputs.make_queries(w, G, device="cpu")
    tm = lambda t: t.cuda().permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)      # [L, T, H, d] storage
    k, q = tm(k), tm(q)
    scale = 1.0 / math.sqrt(128)
    shape, q, k, out = _attention(B, w, G, 1, scale, q=q, k=k)
    _check(w, shape, q, k, out, G, 1, scale)


def test_full_compactor_score_pipeline(B):
    # attention term -> blend with the leverage term (Eq. 6) -> top-k -> gather, all on the GPU, against the oracle
    w = inputs.Workload("full", 2, 2, 128, [1500, 640], [0.3, 0.5], p=1.0, seed=84)
    G, pool, scale, lam = 4, 7, 1.0 / math.sqrt(128), 0.3
    kp, kr, v = [t.cuda() for t in inputs.make_tensors(w, device="cpu")]
    q = inputs.make_queries(w, G, device="cpu").cuda()
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, 3)
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    attn = torch.empty(w.layers, w.heads, shape.total_tokens, dtype=torch.float32, device="cuda")
    ws = B.alloc_workspace(shape)
    B.attention_scores(shape, q, kr, G, attn, ws, scale=scale, pool=pool)
    outs = H.run_compress(B, shape, kp, kr, v, phi, keep, attn=attn, lam=lam)
    # the oracle is given the GPU's attention term (checked on its own above) so that this compares the blend
    H.compare_all_units(shape, keep, outs, kp, kr, v, phi, attn=attn, lam=lam, what="full")
    # and the attention term itself once more, against Eq. 5
    _check(w, shape, q, kr, attn, G, pool, scale)


def test_attention_llama_shape_long(B):
    # one layer of the Llama-3.1-8B shape (8 KV heads x 4 query heads) at n = 8192; two units against the oracle
    w = inputs.Workload("attn-llama", 1, 8, 128, [8192], [0.3], p=0.7, seed=85)
    G, scale = 4, 1.0 / math.sqrt(128)
    _, k, _ = inputs.make_tensors(w, device="cuda", want_pre=False)
    q = inputs.make_queries(w, G, device="cuda")
    shape, q, k, out = _attention(B, w, G, 7, scale, q=q, k=k)
    worst = _check(w, shape, q, k, out, G, 7, scale, units=[(0, 0, 0), (0, 7, 0)])
    print(f"attention llama shape n=8192: worst relative error {worst:.2e}")


def test_attention_many_items_per_cta(B):
    # 864 work items on 148 persistent CTAs: every CTA walks full and ragged chunks of several heads in turn
    w = inputs.Workload("attn-many", 3, 4, 128, [5000, 257, 33, 12345], [0.5] * 4, p=0.7, seed=83)
    scale = 1.0 / math.sqrt(128)
    shape, q, k, out = _attention(B, w, 2, 1, scale)
    assert not torch.isnan(out).any()
    worst = _check(w, shape, q, k, out, 2, 1, scale,
                   units=[(l, h, b) for l in (0, 2) for h in (0, 3) for b in range(4)])
    print(f"attention, many items per CTA: worst rel err {worst:.2e}")

"""The paper's whole method through one call (compactor_compress_full) against the oracle's composition of
its steps: attention term (Eq. 5), leverage scores (Algorithm 1), blend (Eq. 6), selection per head or across
the heads of a layer (Section 3.4), gather."""
import math

import numpy as np
import pytest
import torch

from oracle import compactor_oracle as orc
from paper_2507_08143_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

G, POOL, LAM = 4, 7, 0.3
SCALE = 1.0 / math.sqrt(128)


@pytest.fixture(scope="module")
def B():
    from paper_2507_08143_b200 import binding
    return binding


def _oracle_scores(w, shape, q, k_score, k_cache, phi, with_attn):
    """Final score of every unit from the oracle: [layers][heads] lists of per-sequence arrays."""
    cu = shape.cu_seqlens
    out = {}
    for l in range(w.layers):
        for h in range(w.heads):
            for b in range(w.batch):
                sl = slice(cu[b], cu[b + 1])
                o = orc.approx_leverage_scores(orc.bf16_bits_to_f64(H.bits(k_score[l, h, sl])), phi)
                if with_attn:
                    K = orc.bf16_bits_to_f64(H.bits(k_cache[l, h, sl]))
                    Q = np.stack([orc.bf16_bits_to_f64(H.bits(q[l, h * G + g, sl])) for g in range(G)])
                    a = orc.attention_scores(Q, K, chunk=256, scale=SCALE, pool=POOL)
                    o = orc.blend(a, o, LAM)
                out[(l, h, b)] = o
    return out


@pytest.mark.parametrize("with_attn", [True, False])
def test_full_method_per_head(B, with_attn):
    w = inputs.Workload("full-ph", 2, 2, 128, [1500, 640, 0, 300], [0.3, 0.5, 0.5, 0.25], p=1.0, seed=184)
    kp, kr, v = [t.cuda() for t in inputs.make_tensors(w, device="cpu")]
    q = inputs.make_queries(w, G, device="cpu").cuda()
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, 3)
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    opt = B.options(selection=B.SELECT_PER_HEAD, lam=LAM, q_per_kv=G if with_attn else 0, scale=SCALE, pool=POOL)
    L, Hh, T, tk = w.layers, w.heads, shape.total_tokens, sum(keep)
    scores = torch.full((L, Hh, T), float("nan"), dtype=torch.float32, device="cuda")
    idx = torch.full((L, Hh, tk), -1, dtype=torch.int32, device="cuda")
    ko = torch.zeros(L, Hh, tk, 128, dtype=torch.bfloat16, device="cuda"); vo = torch.zeros_like(ko)
    status = torch.full((w.units,), -1, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.compress_full_workspace_bytes(shape, opt), dtype=torch.uint8, device="cuda")
    B.compress_full(shape, opt, q if with_attn else None, kp, kr, v, phi.cuda(), keep, idx, ko, vo, ws,
                    scores_out=scores, status=status)
    torch.cuda.synchronize()
    st = status.cpu().numpy().reshape(L * Hh, w.batch)
    assert np.all(st[:, [0, 1, 3]] == 0) and np.all(st[:, 2] == 2)       # the empty sequence's Gram matrix has rank 0
    ref = _oracle_scores(w, shape, q, kp, kr, phi.numpy(), with_attn)
    cu, ck = shape.cu_seqlens, np.concatenate([[0], np.cumsum(keep)])
    s_np, idx_np = scores.cpu().numpy().astype(np.float64), idx.cpu().numpy()
    kb, vb, kob, vob = H.bits(kr), H.bits(v), H.bits(ko), H.bits(vo)
    for (l, h, b), want in ref.items():
        got = s_np[l, h, cu[b]:cu[b + 1]]
        if with_attn:          # blended scores cross zero; the attention term carries its own (fp16 exponentials) tolerance
            assert np.all(np.abs(got - want) <= 3e-3 * (1.0 + np.abs(want))), f"{(l, h, b)}: {np.max(np.abs(got - want) / (1 + np.abs(want))):.2e}"
        else:
            assert np.all(np.abs(got - want) <= H.SCORE_RTOL * np.abs(want) + 1e-30), (l, h, b)
        sel = idx_np[l, h, ck[b]:ck[b + 1]]
        np.testing.assert_array_equal(sel, orc.top_k_indices(scores[l, h, cu[b]:cu[b + 1]].cpu().numpy(), keep[b]))
        np.testing.assert_array_equal(kob[l, h, ck[b]:ck[b + 1]], kb[l, h, cu[b]:cu[b + 1]][sel])
        np.testing.assert_array_equal(vob[l, h, ck[b]:ck[b + 1]], vb[l, h, cu[b]:cu[b + 1]][sel])
    # the one call equals the calls it is made of
    if with_attn:
        attn = torch.empty(L, Hh, T, dtype=torch.float32, device="cuda")
        ws2 = B.alloc_workspace(shape)
        B.attention_scores(shape, q, kr, G, attn, ws2, scale=SCALE, pool=POOL)
        outs = H.run_compress(B, shape, kp, kr, v, phi, keep, attn=attn, lam=LAM)
        assert torch.equal(outs[0], scores) and torch.equal(outs[1], idx)


def test_full_method_as_in_the_papers_experiments(B):
    # chunk 256, lambda 0.3, m 48, budgets shared across the heads of a layer
    w = inputs.Workload("full-ah", 2, 4, 128, [2100, 700], [0.3, 0.4], p=1.0, seed=185)
    kp, kr, v = [t.cuda() for t in inputs.make_tensors(w, device="cpu")]
    q = inputs.make_queries(w, G, device="cpu").cuda()
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, 4)
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    opt = B.options(selection=B.SELECT_ACROSS_HEADS, lam=LAM, q_per_kv=G, scale=SCALE, pool=POOL)
    L, Hh, T, tk = w.layers, w.heads, shape.total_tokens, sum(keep)
    scores = torch.full((L, Hh, T), float("nan"), dtype=torch.float32, device="cuda")
    idx = torch.full((L, Hh * tk), -1, dtype=torch.int32, device="cuda")
    offs = torch.full((L, w.batch, Hh + 1), -1, dtype=torch.int32, device="cuda")
    ko = torch.zeros(L, Hh * tk, 128, dtype=torch.bfloat16, device="cuda"); vo = torch.zeros_like(ko)
    ws = torch.empty(B.compress_full_workspace_bytes(shape, opt), dtype=torch.uint8, device="cuda")
    B.compress_full(shape, opt, q, kp, kr, v, phi.cuda(), keep, idx, ko, vo, ws, head_offsets_out=offs, scores_out=scores)
    torch.cuda.synchronize()
    ref = _oracle_scores(w, shape, q, kp, kr, phi.numpy(), True)
    cu, ck = shape.cu_seqlens, np.concatenate([[0], np.cumsum(keep)])
    s_np, idx_np, offs_np = scores.cpu().numpy(), idx.cpu().numpy(), offs.cpu().numpy()
    kb, vb, kob, vob = H.bits(kr), H.bits(v), H.bits(ko), H.bits(vo)
    for (l, h, b), want in ref.items():
        got = s_np[l, h, cu[b]:cu[b + 1]].astype(np.float64)
        assert np.all(np.abs(got - want) <= 3e-3 * (1.0 + np.abs(want))), (l, h, b)
    for l in range(L):
        for b in range(w.batch):
            budget = Hh * keep[b]
            # the selection is exact on the GPU's own scores ...
            want_idx = orc.top_k_across_heads(s_np[l, :, cu[b]:cu[b + 1]].astype(np.float64), budget)
            # ... and agrees with the oracle's choice on its own scores except near the cut
            ref_block = np.stack([ref[(l, h, b)] for h in range(Hh)])
            ref_idx = orc.top_k_across_heads(ref_block, budget)
            cut = np.sort(ref_block.ravel())[::-1][budget - 1]
            base = Hh * ck[b]
            for h in range(Hh):
                lo, hi = base + offs_np[l, b, h], base + offs_np[l, b, h + 1]
                got = idx_np[l, lo:hi]
                np.testing.assert_array_equal(got, want_idx[h], err_msg=f"layer {l} seq {b} head {h}")
                diff = np.setxor1d(got, ref_idx[h])
                assert np.all(np.abs(ref_block[h][diff] - cut) <= 2 * 3e-3 * (1.0 + abs(cut))), f"layer {l} seq {b} head {h}"
                rows = cu[b] + got
                np.testing.assert_array_equal(kob[l, lo:hi], kb[l, h, rows])
                np.testing.assert_array_equal(vob[l, lo:hi], vb[l, h, rows])
            assert offs_np[l, b, Hh] == budget


def test_full_method_argument_errors(B):
    shape = B.Shape(1, 2, 128, 48, [300])
    bad = B.options(selection=7)
    assert B.compress_full_workspace_bytes(shape, bad) == 0
    opt = B.options(q_per_kv=2, pool=4)                  # even pooling window
    k = torch.zeros(1, 2, 300, 128, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros(1, 4, 300, 128, dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros(1, 2, 100, dtype=torch.int32, device="cuda")
    ko = torch.zeros(1, 2, 100, 128, dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.compress_full_workspace_bytes(shape, opt), dtype=torch.uint8, device="cuda")
    phi = inputs.make_sketch_matrix(128, 48, 1).cuda()
    with pytest.raises(B.CompactorError) as e:
        B.compress_full(shape, opt, q, k, k, k, phi, [100], idx, ko, ko.clone(), ws)
    assert e.value.code == -1
    opt = B.options(q_per_kv=2, pool=3)
    with pytest.raises(B.CompactorError) as e:
        B.compress_full(shape, opt, q, k, k, k, phi, [100], idx, ko, ko.clone(), ws[:1024])
    assert e.value.code == -3

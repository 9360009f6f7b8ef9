"""Shared parity-test harness: runs the CUDA library through its binding and compares every
unit with the CPU oracle on the same bits."""
import math

import numpy as np
import torch

from oracle import compactor_oracle as orc

SCORE_RTOL = 1e-3          # fp32 accumulation of bf16 products vs the fp64 oracle

# Index mismatches seen so far, by where the oracle's score of the index lies: within SCORE_RTOL of the
# oracle's kk-th score (the band the acceptance rule allows), or between one and two times that (what two
# scores that are each off by SCORE_RTOL could still produce).  The second count has to stay zero.
BAND_STATS = {"units": 0, "mismatches_in_band": 0, "mismatches_between_1x_and_2x": 0}


def bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def check_unit(scores_gpu, idx_gpu, k_out_bits, v_out_bits, k_score_bits, k_cache_bits, v_bits, phi, kk,
               attn=None, lam=0.3, what=""):
    """All comparisons for one unit.  Returns (max relative score error, boundary-band size)."""
    n = k_score_bits.shape[0]
    s_ref, idx_ref, _, _ = orc.compress_unit(k_score_bits, k_cache_bits, v_bits, phi, kk, attn=attn, lam=lam)
    s_gpu = np.asarray(scores_gpu, dtype=np.float64)
    if attn is None:
        err = np.abs(s_gpu - s_ref) / np.maximum(np.abs(s_ref), 1e-300)
        assert np.all(np.abs(s_gpu - s_ref) <= SCORE_RTOL * np.abs(s_ref) + 1e-30), \
            f"{what}: score error {err.max():.3e} at {int(err.argmax())}"
        max_err = float(err.max()) if n else 0.0
    else:
        err = np.abs(s_gpu - s_ref) / (1.0 + np.abs(s_ref))
        assert np.all(err <= SCORE_RTOL), f"{what}: blended score error {err.max():.3e}"
        max_err = float(err.max()) if n else 0.0

    idx_gpu = np.asarray(idx_gpu, dtype=np.int64)
    assert idx_gpu.shape[0] == kk, what
    band = 0
    if kk > 0:
        assert idx_gpu.min() >= 0 and idx_gpu.max() < n, what
        assert np.all(np.diff(idx_gpu) > 0), f"{what}: indices not strictly ascending"
        # identical sets except inside the tolerance band around the oracle's kk-th score
        kth = np.sort(s_ref)[::-1][kk - 1]
        tol = SCORE_RTOL * (abs(kth) if attn is None else 1.0 + abs(kth))
        in_band = np.abs(s_ref - kth) <= tol
        in_wide = np.abs(s_ref - kth) <= 2 * tol
        band = int(in_band.sum())
        diff = np.setxor1d(idx_gpu, idx_ref.astype(np.int64))
        BAND_STATS["units"] += 1
        BAND_STATS["mismatches_in_band"] += int(in_band[diff].sum())
        BAND_STATS["mismatches_between_1x_and_2x"] += int((in_wide[diff] & ~in_band[diff]).sum())
        assert np.all(in_wide[diff]), f"{what}: {int((~in_wide[diff]).sum())} index mismatches outside what the score tolerance allows"
        assert np.all(in_band[diff]), (f"{what}: {int((~in_band[diff]).sum())} index mismatches whose oracle score is more than "
                                       f"{SCORE_RTOL:g} (relative) away from the oracle's kk-th score")
        # the GPU's own choice is a valid top-kk of the GPU's own scores (ties to the lower index)
        np.testing.assert_array_equal(idx_gpu, orc.top_k_indices(np.asarray(scores_gpu), kk), err_msg=what)
        np.testing.assert_array_equal(k_out_bits, k_cache_bits[idx_gpu], err_msg=what)
        np.testing.assert_array_equal(v_out_bits, v_bits[idx_gpu], err_msg=what)
    return max_err, band


def run_compress(B, shape, k_score, k_cache, v, phi, keep, attn=None, lam=0.3, want_scores=True):
    """Calls the fused entry point; returns (scores, idx, k_out, v_out, status) as torch tensors."""
    dev = k_cache.device
    L, H, T = shape.layers, shape.heads, shape.total_tokens
    total_keep = int(sum(keep))
    scores = torch.full((L, H, T), float("nan"), dtype=torch.float32, device=dev) if want_scores else None
    idx = torch.full((L, H, total_keep), -1, dtype=torch.int32, device=dev)
    k_out = torch.zeros(L, H, total_keep, shape.d, dtype=torch.bfloat16, device=dev)
    v_out = torch.zeros(L, H, total_keep, shape.d, dtype=torch.bfloat16, device=dev)
    status = torch.full((L * H * shape.batch,), -1, dtype=torch.int32, device=dev)
    ws = B.alloc_workspace(shape, dev)
    B.compress(shape, k_score, k_cache, v, phi.to(dev), keep, idx, k_out, v_out, ws, attn=attn, lam=lam,
               scores_out=scores, status=status)
    torch.cuda.synchronize()
    return scores, idx, k_out, v_out, status


def compare_all_units(shape, keep, outs, k_score, k_cache, v, phi, attn=None, lam=0.3, units=None, what=""):
    scores, idx, k_out, v_out, status = outs
    cu = shape.cu_seqlens
    ck = [0]
    for kcount in keep:
        ck.append(ck[-1] + int(kcount))
    phi_np = phi.cpu().numpy()
    worst, band = 0.0, 0
    todo = units if units is not None else [(l, h, b) for l in range(shape.layers) for h in range(shape.heads)
                                           for b in range(shape.batch)]
    for (l, h, b) in todo:
        sl = slice(cu[b], cu[b + 1]); ko = slice(ck[b], ck[b + 1])
        a = None if attn is None else attn[l, h, sl].cpu().numpy()
        e, bd = check_unit(scores[l, h, sl].cpu().numpy(), idx[l, h, ko].cpu().numpy(),
                           bits(k_out[l, h, ko]), bits(v_out[l, h, ko]),
                           bits(k_score[l, h, sl]), bits(k_cache[l, h, sl]), bits(v[l, h, sl]),
                           phi_np, int(keep[b]), attn=a, lam=lam, what=f"{what} unit(l={l},h={h},b={b})")
        worst, band = max(worst, e), max(band, bd)
    return worst, band

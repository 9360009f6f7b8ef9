"""Selection across the heads of a layer and the matching gather, against the oracle."""
import numpy as np
import pytest
import torch

from oracle import compactor_oracle as orc
from paper_2507_08143_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2507_08143_b200 import binding
    return binding


def _select_and_check(B, shape, scores, keep):
    L, Hh = shape.layers, shape.heads
    total_keep = int(sum(keep))
    idx = torch.full((L, Hh * total_keep), -1, dtype=torch.int32, device="cuda")
    offs = torch.full((L, shape.batch, Hh + 1), -1, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(256, B.across_heads_workspace_bytes(shape)), dtype=torch.uint8, device="cuda")
    B.select_across_heads(shape, scores, keep, idx, offs, ws)
    torch.cuda.synchronize()
    s_np, idx_np, offs_np = scores.cpu().numpy(), idx.cpu().numpy(), offs.cpu().numpy()
    cu = shape.cu_seqlens
    ck = np.concatenate([[0], np.cumsum(keep)])
    for l in range(L):
        for b in range(shape.batch):
            n, kk = shape.seqlens[b], keep[b]
            if n == 0 or kk == 0:
                assert np.all(offs_np[l, b] == 0)
                continue
            want = orc.top_k_across_heads(s_np[l, :, cu[b]:cu[b + 1]].astype(np.float64), Hh * kk)
            block = idx_np[l, Hh * ck[b]:Hh * ck[b + 1]]
            assert offs_np[l, b, 0] == 0 and offs_np[l, b, Hh] == Hh * kk
            for h in range(Hh):
                got = block[offs_np[l, b, h]:offs_np[l, b, h + 1]]
                np.testing.assert_array_equal(got, want[h], err_msg=f"layer {l} seq {b} head {h}")
    return idx, offs, ws


def test_across_heads_random_scores_with_ties(B):
    rng = np.random.default_rng(3)
    seqlens, keep = [3000, 1, 0, 9000, 257], [900, 1, 0, 4500, 0]
    shape = B.Shape(2, 3, 128, 48, seqlens)
    T = shape.total_tokens
    s = rng.standard_normal((2, 3, T)).astype(np.float32)
    s[0] = np.round(s[0], 1)                               # heavy ties, also across heads
    s[1, 1] *= 3.0                                         # one head dominates
    s[1, 2] = 0.5                                          # one constant head
    _select_and_check(B, shape, torch.from_numpy(s).cuda(), keep)


def test_across_heads_keep_everything_and_single_head(B):
    rng = np.random.default_rng(4)
    shape = B.Shape(1, 4, 128, 48, [500, 300])
    s = torch.from_numpy(rng.standard_normal((1, 4, 800)).astype(np.float32)).cuda()
    _select_and_check(B, shape, s, [500, 100])             # first sequence: kk = n
    shape1 = B.Shape(2, 1, 128, 48, [2000])
    s1 = torch.from_numpy(rng.standard_normal((2, 1, 2000)).astype(np.float32)).cuda()
    idx, offs, ws = _select_and_check(B, shape1, s1, [700])
    # with one head, across-head selection is per-head selection
    idx_ph = torch.empty(2, 1, 700, dtype=torch.int32, device="cuda")
    B.select(shape1, s1, [700], idx_ph, ws)
    torch.cuda.synchronize()
    assert torch.equal(idx_ph.view(2, 700), idx)


def test_across_heads_pipeline_on_leverage_scores(B):
    # real scores from the scoring pass; the gather must deliver the rows the indices name, in order
    w = inputs.Workload("across", 2, 4, 128, [4000, 1500], [0.3, 0.5], p=1.0, seed=95)
    kp, kr, v = [t.cuda() for t in inputs.make_tensors(w, device="cpu")]
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, 8).cuda()
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    scores = torch.empty(w.layers, w.heads, shape.total_tokens, dtype=torch.float32, device="cuda")
    ws = B.alloc_workspace(shape)
    B.score(shape, kp, phi, scores, ws)
    idx, offs, ws2 = _select_and_check(B, shape, scores, keep)
    total_keep = sum(keep)
    ko = torch.full((w.layers, w.heads * total_keep, 128), 7.0, dtype=torch.bfloat16, device="cuda"); vo = ko.clone()
    B.compact_across_heads(shape, kr, v, idx, offs, keep, ko, vo, ws2)
    torch.cuda.synchronize()
    kb, vb, kob, vob = H.bits(kr), H.bits(v), H.bits(ko), H.bits(vo)
    idx_np, offs_np = idx.cpu().numpy(), offs.cpu().numpy()
    cu, ck = shape.cu_seqlens, np.concatenate([[0], np.cumsum(keep)])
    for l in range(w.layers):
        for b in range(w.batch):
            base = w.heads * ck[b]
            for h in range(w.heads):
                lo, hi = base + offs_np[l, b, h], base + offs_np[l, b, h + 1]
                rows = cu[b] + idx_np[l, lo:hi]
                np.testing.assert_array_equal(kob[l, lo:hi], kb[l, h, rows])
                np.testing.assert_array_equal(vob[l, lo:hi], vb[l, h, rows])
    counts = np.diff(offs_np, axis=2)
    assert counts.min() >= 0 and np.all(counts.sum(axis=2) == w.heads * np.array(keep)[None, :])
    print("tokens kept per head (layer 0, sequence 0):", counts[0, 0].tolist())


def test_across_heads_long_sequence_large_budget(B):
    # more than 2^16 kept indices in a head, stretches of more than 2^16 scores per warp
    rng = np.random.default_rng(5)
    n, kk = 600000, 250000
    shape = B.Shape(1, 3, 128, 48, [n])
    s = rng.standard_normal((1, 3, n)).astype(np.float32)
    s[0, 0] += 1.0                                         # the first head takes most of the budget
    s[0, 2] = np.round(s[0, 2], 1)
    _select_and_check(B, shape, torch.from_numpy(s).cuda(), [kk])


def test_across_heads_scores_that_defeat_the_histogram(B):
    # non-finite scores, and a bulk far narrower than the sampled range (every score in one bin): both groups are
    # redone by one CTA over all scores, and the neighbouring well-behaved layer is not disturbed
    rng = np.random.default_rng(6)
    n = 90000
    shape = B.Shape(3, 2, 128, 48, [n, 2000])
    T = shape.total_tokens
    s = rng.standard_normal((3, 2, T)).astype(np.float32)
    s[0, 1, 5::11] = np.inf
    s[0, 0, 6::13] = -np.inf
    s[1] *= 1e-4
    s[1, 0, 3] = 1000.0; s[1, 0, 9] = -1000.0              # the range estimate spans 2000, the bulk 1e-3
    _select_and_check(B, shape, torch.from_numpy(s).cuda(), [30000, 700])


def test_across_heads_with_extreme_scores_at_the_start(B):
    # a real context's first tokens have leverage scores near one, the rest near m/n: the sampled range is lopsided and
    # every CTA of the group narrows it in the same way
    rng = np.random.default_rng(8)
    n = 150000
    shape = B.Shape(1, 4, 128, 48, [n])
    s = np.abs((48.0 / n) * (1.0 + 0.3 * rng.standard_normal((1, 4, n)))).astype(np.float32)
    s[..., 0] = 1.0
    s[..., 1] = 0.6
    s[0, 2, 99999] = 0.8
    _select_and_check(B, shape, torch.from_numpy(s).cuda(), [45000])

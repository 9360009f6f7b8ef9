"""Guard bands: every output and the workspace are carved out of larger buffers filled with a
pattern, and after the call every byte outside the declared extents must still hold the pattern.
This stands in for a memory checker: a write past the end of `scores_out`, `idx_out`, `k_out`,
`v_out`, `status`, `attn_out` or the workspace shows up on the host, without any fault."""
import numpy as np
import pytest
import torch

from paper_2507_08143_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu

GUARD = 8192           # bytes on either side
PATTERN = 0xA5


class Guarded:
    """A device tensor of the given shape and dtype with GUARD patterned bytes before and after it."""

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) if len(shape) else 1
        self.nbytes = n * torch.empty(0, dtype=dtype).element_size()
        self.raw = torch.full((GUARD + self.nbytes + GUARD + 256,), PATTERN, dtype=torch.uint8, device="cuda")
        off = (-self.raw.data_ptr()) % 256 + GUARD                        # 256-byte aligned payload
        off += (-off) % 256 if (self.raw.data_ptr() + off) % 256 else 0
        self.off = off
        self.t = self.raw[off:off + self.nbytes].view(dtype).view(*shape) if n else torch.empty(shape, dtype=dtype, device="cuda")
        assert n == 0 or self.t.data_ptr() % 256 == 0
        if fill is not None and n:
            self.t.fill_(fill)

    def check(self, what):
        raw = self.raw.cpu().numpy()
        before, after = raw[:self.off], raw[self.off + self.nbytes:]
        assert np.all(before == PATTERN), f"{what}: {int((before != PATTERN).sum())} bytes written before the buffer"
        assert np.all(after == PATTERN), f"{what}: {int((after != PATTERN).sum())} bytes written past the end of the buffer"


@pytest.fixture(scope="module")
def B():
    from paper_2507_08143_b200 import binding
    return binding


def _compress_guarded(B, w, with_attn=False):
    kp, kr, v = [t.cuda() for t in inputs.make_tensors(w, device="cpu")]
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, w.seed).cuda()
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    L, Hh, T, tk = w.layers, w.heads, shape.total_tokens, sum(keep)
    g = {"scores_out": Guarded((L, Hh, T), torch.float32, float("nan")),
         "idx_out": Guarded((L, Hh, tk), torch.int32, -1),
         "k_out": Guarded((L, Hh, tk, w.d), torch.bfloat16, 0),
         "v_out": Guarded((L, Hh, tk, w.d), torch.bfloat16, 0),
         "status": Guarded((L * Hh * w.batch,), torch.int32, -1),
         "workspace": Guarded((B.workspace_bytes(shape),), torch.uint8)}
    attn = inputs.make_attention_scores(w, seed=3, device="cuda") if with_attn else None
    B.compress(shape, kp, kr, v, phi, keep, g["idx_out"].t, g["k_out"].t, g["v_out"].t, g["workspace"].t,
               attn=attn, scores_out=g["scores_out"].t, status=g["status"].t)
    torch.cuda.synchronize()
    for name, buf in g.items():
        buf.check(f"{w.name}: {name}")
    # the call did its work inside the extents
    assert not torch.isnan(g["scores_out"].t).any() and int(g["idx_out"].t.min()) >= 0
    outs = (g["scores_out"].t, g["idx_out"].t, g["k_out"].t, g["v_out"].t, g["status"].t)
    H.compare_all_units(shape, keep, outs, kp, kr, v, phi.cpu(), attn=attn, units=[(0, 0, 0)], what=w.name)


def test_c0_writes_nothing_outside_its_buffers(B):
    _compress_guarded(B, inputs.workload("c0"))
    _compress_guarded(B, inputs.workload("c0"), with_attn=True)


def test_few_long_units_write_nothing_outside_their_buffers(B):
    # two heads with one long sequence: the blend's per-slice statistics and the sliced selection's histograms,
    # candidate lists and counts live in the part of the workspace that the scoring stage has finished with
    w = inputs.Workload("guard-long", 1, 2, 128, [140001, 77], [0.3, 0.5], p=0.7, seed=14)
    _compress_guarded(B, w, with_attn=True)
    _compress_guarded(B, w)


def test_ragged_batch_with_tail_tiles_writes_nothing_outside_its_buffers(B):
    # lengths that end inside a tile, a piece and a Gram block; an empty sequence; total tokens not a multiple of anything
    w = inputs.Workload("guard-ragged", 2, 3, 128, [1000, 129, 0, 2501, 47, 4099, 1], [0.3, 0.5, 0.5, 0.3, 0.5, 0.11, 1.0],
                        p=0.7, seed=13)
    _compress_guarded(B, w)


def test_wide_sketches_write_nothing_outside_their_buffers(B):
    # sketches of more than 64 columns keep two 128 x 128 parts of the projected Gram matrix per unit, more than the
    # narrow ones need; m = 80 is padded to 128 columns, m = 128 is the exact-score route
    for m in (80, 128):
        _compress_guarded(B, inputs.Workload(f"guard-wide-{m}", 1, 3, 128, [1500, 200, 333], [0.3, 0.5, 0.4], p=0.7, seed=16, m=m))


def test_across_heads_selection_writes_nothing_outside_its_buffers(B):
    w = inputs.Workload("guard-across", 2, 3, 128, [700, 1301], [0.3, 0.4], p=0.7, seed=14)
    _, kr, v = [None if t is None else t.cuda() for t in inputs.make_tensors(w, device="cpu", want_pre=False)]
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, 2).cuda()
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    L, Hh, T, tk = w.layers, w.heads, shape.total_tokens, sum(keep)
    scores = Guarded((L, Hh, T), torch.float32, float("nan"))
    ws = Guarded((B.workspace_bytes(shape),), torch.uint8)
    B.score(shape, kr, phi, scores.t, ws.t)
    idx = Guarded((L, Hh * tk), torch.int32, -1)
    offs = Guarded((L, w.batch, Hh + 1), torch.int32, -1)
    ws2 = Guarded((B.across_heads_workspace_bytes(shape),), torch.uint8)
    B.select_across_heads(shape, scores.t, keep, idx.t, offs.t, ws2.t)
    ko = Guarded((L, Hh * tk, w.d), torch.bfloat16, 0)
    vo = Guarded((L, Hh * tk, w.d), torch.bfloat16, 0)
    B.compact_across_heads(shape, kr, v, idx.t, offs.t, keep, ko.t, vo.t, ws2.t)
    torch.cuda.synchronize()
    for name, buf in [("scores", scores), ("workspace", ws), ("idx", idx), ("head_offsets", offs),
                      ("across workspace", ws2), ("k_out", ko), ("v_out", vo)]:
        buf.check(f"across heads: {name}")
    assert int(idx.t.min()) >= 0 and int(offs.t.min()) >= 0


def test_builtin_scratch_entry_and_attention_write_nothing_outside_their_buffers(B):
    w = inputs.Workload("guard-misc", 1, 2, 128, [900, 300], [0.3, 0.5], p=0.7, seed=15)
    _, kr, _ = inputs.make_tensors(w, device="cpu", want_pre=False)
    kr = kr.cuda()
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, 2).cuda()
    scores = Guarded((1, 2, shape.total_tokens), torch.float32, float("nan"))
    status = Guarded((4,), torch.int32, -1)
    B.score_builtin_scratch(shape, kr, phi, scores.t, status=status.t)
    q = inputs.make_queries(w, 2, device="cpu").cuda()
    attn = Guarded((1, 2, shape.total_tokens), torch.float32, float("nan"))
    ws = Guarded((B.workspace_bytes(shape),), torch.uint8)
    B.attention_scores(shape, q, kr, 2, attn.t, ws.t, scale=128 ** -0.5, pool=5)
    torch.cuda.synchronize()
    for name, buf in [("scores", scores), ("status", status), ("attn_out", attn), ("workspace", ws)]:
        buf.check(f"misc: {name}")
    assert not torch.isnan(scores.t).any() and not torch.isnan(attn.t).any()

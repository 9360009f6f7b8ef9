"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (one fused
call over the whole workload, rotated keys scored and gathered): sampled units against the oracle
element by element, and properties that hold at any size checked on every unit."""
import numpy as np
import pytest
import torch

from paper_2507_08143_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _properties_all_units(w, shape, keep, scores, idx, k_out, v_out, kr, v):
    cu = shape.cu_seqlens
    ck = np.concatenate([[0], np.cumsum(keep)]).tolist()
    m = w.m
    for b in range(w.batch):
        n, kk = w.seqlens[b], keep[b]
        if n == 0:
            continue
        s = scores[:, :, cu[b]:cu[b + 1]]
        total = s.double().sum(dim=2)
        assert torch.all((total - m).abs() <= 1e-3 * m), f"sum of scores != sketch rank (seq {b})"   # sum o = rank(K Phi)
        assert float(s.min()) >= 0.0 and float(s.max()) <= 1.0 + 1e-3
        sel = idx[:, :, ck[b]:ck[b + 1]].long()
        assert int(sel.min()) >= 0 and int(sel.max()) < n
        assert torch.all(sel[:, :, 1:] > sel[:, :, :-1]), "indices not strictly ascending"
        kept_min = s.gather(2, sel).min(dim=2).values
        assert torch.all((s > kept_min[..., None]).sum(dim=2) < kk)          # everything above the cut is kept
        assert torch.all((s >= kept_min[..., None]).sum(dim=2) >= kk)
        for l in range(w.layers):                                          # bit-exact gather, layer by layer
            rows = sel[l][..., None].expand(-1, -1, w.d)
            src_k = kr[l, :, cu[b]:cu[b + 1]].view(torch.int16)
            src_v = v[l, :, cu[b]:cu[b + 1]].view(torch.int16)
            assert torch.equal(k_out[l, :, ck[b]:ck[b + 1]].view(torch.int16), src_k.gather(1, rows))
            assert torch.equal(v_out[l, :, ck[b]:ck[b + 1]].view(torch.int16), src_v.gather(1, rows))


def _full(B, name, sample_units):
    w = name if isinstance(name, inputs.Workload) else inputs.workload(name)
    need = 2 * w.layers * w.heads * w.total_tokens * w.d * 2 * 1.45 + (4 << 30)
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        pytest.skip(f"needs {need / 2**30:.0f} GiB of device memory")
    _, kr, v = inputs.make_tensors(w, device="cuda", want_pre=False)
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, w.seed)
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    scores, idx, k_out, v_out, status = H.run_compress(B, shape, kr, kr, v, phi, keep)
    assert int(status.max()) == 0
    _properties_all_units(w, shape, keep, scores, idx, k_out, v_out, kr, v)
    worst, band = H.compare_all_units(shape, keep, (scores, idx, k_out, v_out, status), kr, kr, v, phi,
                                      units=sample_units, what=w.name)
    print(f"{w.name} full size: {w.units} units, {len(sample_units)} against the oracle, "
          f"max rel score err {worst:.2e}, boundary band {band}, index mismatches so far {H.BAND_STATS}")


@pytest.fixture(scope="module")
def B():
    from paper_2507_08143_b200 import binding
    return binding


def test_c1_full(B):
    _full(B, "c1", [(l, h, 0) for l in (0, 13, 31) for h in (0, 3, 7)])


def test_c2_full(B):
    _full(B, "c2", [(0, 0, 0), (11, 2, 0), (27, 3, 0)])


def test_c4_full_ragged(B):
    w = inputs.workload("c4")
    order = np.argsort(w.seqlens)
    picks = [int(order[0]), int(order[len(order) // 2]), int(order[-1])]      # shortest, median, longest sequence
    _full(B, "c4", [(0, 0, picks[0]), (17, 5, picks[1]), (31, 7, picks[2]), (9, 2, picks[0])])


def test_c3_full(B):
    _full(B, "c3", [(0, 0, 0), (9, 1, 0), (18, 2, 0), (27, 3, 0), (36, 4, 0), (45, 5, 0), (54, 6, 0), (63, 7, 0)])


def test_one_million_token_sequence_beside_a_short_one(B):
    # the longest context of the paper's Fig. 1 (2^20 tokens) packed with a 300-token sequence:
    # 32 Gram blocks of 32768 tokens per unit, fp64 across them
    w = inputs.Workload("1m", 1, 2, 128, [1 << 20, 300], [0.1, 0.5], p=0.7, seed=77)
    _full(B, w, [(0, 0, 0), (0, 1, 1)])

"""The allocation-free scoring entry point against the ordinary one and against the oracle.

Some users of the library cannot allocate device memory at the moment they need scores (an
engine whose own allocator owns the whole device, code inside a stream capture), so
compactor_score_builtin_scratch keeps its scratch in a fixed array inside the library.  The
array is shared by every call and is never cleared, so the check is made on calls in a row
with different inputs: a later one must not be affected by what an earlier one left behind.
Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import compactor_oracle as orc
from paper_2507_08143_b200 import inputs
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _one_call(B, w, sketch_seed, oracle_units):
    kp, _, _ = inputs.make_tensors(w, device="cpu")
    kp = kp.cuda()
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, sketch_seed)
    phi_d = phi.cuda()
    want = torch.full((w.layers, w.heads, shape.total_tokens), float("nan"), dtype=torch.float32, device="cuda")
    got = torch.full_like(want, float("nan"))
    st_want = torch.full((w.units,), -1, dtype=torch.int32, device="cuda")
    st_got = torch.full_like(st_want, -1)
    ws = B.alloc_workspace(shape)
    B.score(shape, kp, phi_d, want, ws, status=st_want)
    B.score_builtin_scratch(shape, kp, phi_d, got, status=st_got)      # the entry point under test
    torch.cuda.synchronize()
    want_np, got_np = want.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got_np))
    # same tolerance as the parity tests: the two may split the Gram sums into different blocks
    assert np.all(np.abs(got_np - want_np) <= 1e-3 * np.abs(want_np) + 1e-30), np.max(np.abs(got_np - want_np) / np.abs(want_np))
    assert torch.equal(st_want, st_got)
    # and directly against the oracle, at the tolerance of the parity tests (not two tolerances in a row)
    cu = shape.cu_seqlens
    phi_np = phi.numpy()
    for (l, h, b) in oracle_units:
        ref = orc.approx_leverage_scores(orc.bf16_bits_to_f64(H.bits(kp[l, h, cu[b]:cu[b + 1]])), phi_np)
        mine = got_np[l, h, cu[b]:cu[b + 1]]
        assert np.all(np.abs(mine - ref) <= H.SCORE_RTOL * np.abs(ref) + 1e-30), \
            f"unit {(l, h, b)}: {np.max(np.abs(mine - ref) / np.abs(ref)):.3e}"


def test_builtin_scratch_matches_workspace_entry_point_and_oracle():
    from paper_2507_08143_b200 import binding as B
    assert B.builtin_scratch_bytes() == 32 << 20
    first = inputs.Workload("noalloc-a", 2, 2, 128, [3000, 700], [0.3, 0.3], p=0.7, seed=91)
    second = inputs.Workload("noalloc-b", 1, 4, 128, [40000], [0.3], p=1.0, n_out=8, seed=92)
    _one_call(B, first, 1, [(0, 0, 0), (1, 1, 1)])
    _one_call(B, second, 2, [(0, 3, 0)])       # larger, and reuses the dirty scratch
    _one_call(B, first, 3, [(1, 0, 0)])


def test_builtin_scratch_shrinks_its_plan_to_fit():
    # a problem whose ordinary plan needs more than the 32 MiB array for everything but the scores, and which
    # fits once the entry point has traded scratch for longer Gram blocks (or a shorter ring of partial sums)
    from paper_2507_08143_b200 import binding as B
    w = inputs.Workload("noalloc-c", 4, 8, 128, [40000], [0.3], p=0.7, seed=93)
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    scores_bytes = 4 * w.layers * w.heads * shape.total_tokens
    assert B.workspace_bytes(shape) - scores_bytes > B.builtin_scratch_bytes(), \
        "the ordinary plan fits the array: this case no longer exercises the shrinking"
    _one_call(B, w, 4, [(0, 0, 0), (3, 7, 0)])


def test_builtin_scratch_rejects_oversized_problem():
    from paper_2507_08143_b200 import binding as B
    shape = B.Shape(64, 8, 128, 48, [131072])           # far more scratch than the array holds, however the plan is shrunk
    k = torch.empty(8, dtype=torch.bfloat16, device="cuda")
    fake = B.CompactorMat(k.data_ptr(), 128, 128, 128)   # never dereferenced: the size check comes first
    out = torch.empty(8, dtype=torch.float32, device="cuda")
    rc = B.LIB.compactor_score_builtin_scratch(B.byref(shape.c), fake, B.c_void_p(out.data_ptr()), None, 0.3,
                                               B.c_void_p(out.data_ptr()), None, None)
    assert rc == -5
    assert "scratch" in B.error_string(rc)

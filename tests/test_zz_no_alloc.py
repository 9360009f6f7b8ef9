"""The allocation-free scoring entry point against the ordinary one.

Some users of the library cannot allocate device memory at the moment they need scores (an
engine whose own allocator owns the whole device, code inside a stream capture), so
compactor_score_builtin_scratch keeps its scratch in a fixed array inside the library.  The
array is shared by every call and is never cleared, so the check is made on two calls in a row
with different inputs: the second must not be affected by what the first left behind.
Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2507_08143_b200 import inputs

pytestmark = pytest.mark.gpu


def _one_call(B, w, sketch_seed):
    kp, _, _ = inputs.make_tensors(w, device="cpu")
    kp = kp.cuda()
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    phi = inputs.make_sketch_matrix(w.d, w.m, sketch_seed).cuda()
    want = torch.full((w.layers, w.heads, shape.total_tokens), float("nan"), dtype=torch.float32, device="cuda")
    got = torch.full_like(want, float("nan"))
    st_want = torch.full((w.units,), -1, dtype=torch.int32, device="cuda")
    st_got = torch.full_like(st_want, -1)
    ws = B.alloc_workspace(shape)
    B.score(shape, kp, phi, want, ws, status=st_want)
    B.score_builtin_scratch(shape, kp, phi, got, status=st_got)      # the entry point under test
    torch.cuda.synchronize()
    want, got = want.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    # same tolerance as the parity tests: the two may split the Gram sums into different blocks
    assert np.all(np.abs(got - want) <= 1e-3 * np.abs(want) + 1e-30), np.max(np.abs(got - want) / np.abs(want))
    assert torch.equal(st_want, st_got)


def test_builtin_scratch_matches_workspace_entry_point_twice():
    from paper_2507_08143_b200 import binding as B
    assert B.builtin_scratch_bytes() == 32 << 20
    first = inputs.Workload("noalloc-a", 2, 2, 128, [3000, 700], [0.3, 0.3], p=0.7, seed=91)
    second = inputs.Workload("noalloc-b", 1, 4, 128, [40000], [0.3], p=1.0, n_out=8, seed=92)
    _one_call(B, first, 1)
    _one_call(B, second, 2)       # larger: forces longer Gram blocks and reuses the dirty scratch
    _one_call(B, first, 3)


def test_builtin_scratch_rejects_oversized_problem():
    from paper_2507_08143_b200 import binding as B
    shape = B.Shape(64, 8, 128, 48, [131072])           # needs 128 MiB of Gram blocks even at the longest block length
    k = torch.empty(8, dtype=torch.bfloat16, device="cuda")
    fake = B.CompactorMat(k.data_ptr(), 128, 128, 128)   # never dereferenced: the size check comes first
    out = torch.empty(8, dtype=torch.float32, device="cuda")
    rc = B.LIB.compactor_score_builtin_scratch(B.byref(shape.c), fake, B.c_void_p(out.data_ptr()), None, 0.3,
                                               B.c_void_p(out.data_ptr()), None, None)
    assert rc == -5
    assert "scratch" in B.error_string(rc)

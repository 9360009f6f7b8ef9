"""The fused call recorded into a CUDA graph and replayed: every step is a kernel or a memset on the
caller's stream (the prefix tables travel as kernel arguments, 239 sequences per launch), so a replay
with new contents in the same buffers gives what a direct call gives."""
import pytest
import torch

from paper_2507_08143_b200 import inputs

pytestmark = pytest.mark.gpu


def test_compress_replayed_from_a_cuda_graph_matches_direct_calls():
    from paper_2507_08143_b200 import binding as B
    w = inputs.Workload("graph", 2, 2, 128, [3000, 1, 517], [0.3, 1.0, 0.5], p=0.7, seed=71)
    shape = B.Shape(w.layers, w.heads, w.d, w.m, w.seqlens)
    keep = [B.keep_count(n, r) for n, r in zip(w.seqlens, w.ratios)]
    phi = inputs.make_sketch_matrix(w.d, w.m, w.seed).cuda()
    T, KK = shape.total_tokens, sum(keep)
    k = torch.empty(w.layers, w.heads, T, 128, dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(k)
    ws = B.alloc_workspace(shape)

    def outputs():
        return (torch.full((w.layers, w.heads, T), -1.0, dtype=torch.float32, device="cuda"),
                torch.full((w.layers, w.heads, KK), -1, dtype=torch.int32, device="cuda"),
                torch.zeros(w.layers, w.heads, KK, 128, dtype=torch.bfloat16, device="cuda"),
                torch.zeros(w.layers, w.heads, KK, 128, dtype=torch.bfloat16, device="cuda"))

    def fill(seed):
        _, kr, vv = inputs.make_tensors(inputs.Workload("graph", 2, 2, 128, w.seqlens, w.ratios, p=0.7, seed=seed),
                                        device="cpu", want_pre=False)
        k.copy_(kr); v.copy_(vv)

    fill(71)
    g_out = outputs()
    B.compress(shape, k, k, v, phi, keep, g_out[1], g_out[2], g_out[3], ws, scores_out=g_out[0])   # set-up before capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        B.compress(shape, k, k, v, phi, keep, g_out[1], g_out[2], g_out[3], ws, scores_out=g_out[0])
    for seed in (71, 72, 73):
        fill(seed)
        for t in g_out:
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        d_out = outputs()
        B.compress(shape, k, k, v, phi, keep, d_out[1], d_out[2], d_out[3], ws, scores_out=d_out[0])
        torch.cuda.synchronize()
        for a, b in zip(g_out, d_out):
            assert torch.equal(a, b), f"replay differs from a direct call (seed {seed})"
        assert int(g_out[1].min()) >= 0


def test_batch_of_several_hundred_sequences_under_capture():
    # more sequences than one table launch carries: still nothing but kernels and memsets, so capture works,
    # and the units come out as in separate one-sequence calls
    from paper_2507_08143_b200 import binding as B
    import numpy as np
    rng = np.random.default_rng(5)
    seqlens = [int(x) for x in rng.integers(1, 700, size=523)]
    w = inputs.Workload("many", 1, 2, 128, seqlens, [0.4] * len(seqlens), p=0.7, seed=81)
    _, kr, v = [None if t is None else t.cuda() for t in inputs.make_tensors(w, device="cpu", want_pre=False)]
    shape = B.Shape(1, 2, 128, 48, seqlens)
    keep = [B.keep_count(n, 0.4) for n in seqlens]
    phi = inputs.make_sketch_matrix(128, 48, 1).cuda()
    T, KK = shape.total_tokens, sum(keep)
    scores = torch.full((1, 2, T), -1.0, dtype=torch.float32, device="cuda")
    idx = torch.full((1, 2, KK), -1, dtype=torch.int32, device="cuda")
    ko = torch.zeros(1, 2, KK, 128, dtype=torch.bfloat16, device="cuda"); vo = torch.zeros_like(ko)
    ws = B.alloc_workspace(shape)
    B.compress(shape, kr, kr, v, phi, keep, idx, ko, vo, ws, scores_out=scores)
    torch.cuda.synchronize()
    direct = (scores.clone(), idx.clone(), ko.clone(), vo.clone())
    for t in (scores, idx, ko, vo):
        t.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        B.compress(shape, kr, kr, v, phi, keep, idx, ko, vo, ws, scores_out=scores)
    graph.replay()
    torch.cuda.synchronize()
    for a, b in zip((scores, idx, ko, vo), direct):
        assert torch.equal(a, b)
    cu, ck = shape.cu_seqlens, np.concatenate([[0], np.cumsum(keep)])
    for b in (0, 239, 240, 522):                      # either side of the first table launch, and the last sequence
        one = B.Shape(1, 2, 128, 48, [seqlens[b]])
        s1 = torch.empty(1, 2, seqlens[b], dtype=torch.float32, device="cuda")
        B.score(one, kr[:, :, cu[b]:cu[b + 1]], phi, s1, B.alloc_workspace(one))
        torch.cuda.synchronize()
        # the two calls may cut the Gram sums into different blocks: equal up to fp32 rounding of those sums
        assert torch.allclose(s1, scores[:, :, cu[b]:cu[b + 1]], rtol=1e-4, atol=0), f"sequence {b}"

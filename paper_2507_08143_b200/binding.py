"""ctypes binding of the C-ABI library: argument marshalling only.

Function names mirror the C entry points of `include/compactor.h`.  Device buffers are torch
CUDA tensors (torch is used for device memory and streams, nothing else); every step of the
path runs in the library's kernels.  Importing this module fails loudly if the library cannot
be built or loaded - there is no fallback."""
from __future__ import annotations

import ctypes
from ctypes import POINTER, Structure, byref, c_char_p, c_double, c_float, c_int32, c_int64, c_size_t, c_uint64, c_void_p
from typing import Optional, Sequence

import torch

from . import build as _build


class CompactorMat(Structure):
    _fields_ = [("ptr", c_void_p), ("stride_layer", c_int64), ("stride_head", c_int64), ("stride_token", c_int64)]


class CompactorShape(Structure):
    _fields_ = [("layers", c_int32), ("heads", c_int32), ("d", c_int32), ("m", c_int32),
                ("batch", c_int32), ("cu_seqlens", POINTER(c_int32))]


class CompactorOptions(Structure):
    _fields_ = [("selection", c_int32), ("factorization", c_int32), ("eig_floor", c_double), ("lam", c_float),
                ("q_per_kv", c_int32), ("chunk", c_int32), ("scale", c_float), ("pool", c_int32)]


class CompactorError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {error_string(code)} ({code})")


def _load() -> ctypes.CDLL:
    path = _build.build()
    lib = ctypes.CDLL(path)
    lib.compactor_version.restype = ctypes.c_int
    lib.compactor_error_string.restype = c_char_p
    lib.compactor_error_string.argtypes = [ctypes.c_int]
    lib.compactor_make_sketch.argtypes = [c_uint64, c_int32, c_int32, POINTER(c_float)]
    lib.compactor_make_sketch_srht.argtypes = [c_uint64, c_int32, c_int32, POINTER(c_float)]
    lib.compactor_keep_count.restype = c_int64
    lib.compactor_keep_count.argtypes = [c_int64, c_double]
    lib.compactor_calibrated_ratio.argtypes = [c_double, c_double, c_double, c_double, POINTER(c_double)]
    lib.compactor_fit_calibration.argtypes = [c_int64, POINTER(c_double), POINTER(c_double), POINTER(c_double), c_double,
                                              POINTER(c_double), POINTER(c_double), POINTER(c_double)]
    lib.compactor_workspace_bytes.restype = c_size_t
    lib.compactor_workspace_bytes.argtypes = [POINTER(CompactorShape)]
    lib.compactor_score.argtypes = [POINTER(CompactorShape), CompactorMat, c_void_p, c_void_p, c_float, c_void_p,
                                    c_void_p, c_void_p, c_size_t, c_void_p]
    lib.compactor_score_variant.argtypes = [POINTER(CompactorShape), CompactorMat, c_void_p, c_int32, c_double, c_void_p,
                                            c_float, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.compactor_nll.argtypes = [c_void_p, c_int32, c_int64, c_int32, c_int64, c_void_p, c_int32, POINTER(c_int32),
                                  c_void_p, c_void_p, c_void_p]
    lib.compactor_select.argtypes = [POINTER(CompactorShape), c_void_p, POINTER(c_int32), c_void_p, c_void_p,
                                     c_void_p, c_size_t, c_void_p]
    lib.compactor_compact.argtypes = [POINTER(CompactorShape), CompactorMat, CompactorMat, c_void_p, POINTER(c_int32),
                                      c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.compactor_compress.argtypes = [POINTER(CompactorShape), CompactorMat, CompactorMat, CompactorMat, c_void_p,
                                       c_void_p, c_float, POINTER(c_int32), c_void_p, c_void_p, c_void_p, c_void_p,
                                       c_void_p, c_void_p, c_size_t, c_void_p]
    lib.compactor_compress_profiled.argtypes = lib.compactor_compress.argtypes + [POINTER(c_void_p), c_int32]
    lib.compactor_attention_scores.argtypes = [POINTER(CompactorShape), CompactorMat, CompactorMat, c_int32, c_int32,
                                               c_float, c_int32, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.compactor_attention_scores_status.argtypes = [POINTER(CompactorShape), CompactorMat, CompactorMat, c_int32, c_int32,
                                                      c_float, c_int32, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.compactor_across_heads_workspace_bytes.restype = c_size_t
    lib.compactor_across_heads_workspace_bytes.argtypes = [POINTER(CompactorShape)]
    lib.compactor_select_across_heads.argtypes = [POINTER(CompactorShape), c_void_p, POINTER(c_int32), c_void_p, c_void_p,
                                                  c_void_p, c_size_t, c_void_p]
    lib.compactor_compact_across_heads.argtypes = [POINTER(CompactorShape), CompactorMat, CompactorMat, c_void_p, c_void_p,
                                                   POINTER(c_int32), c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.compactor_compress_full_workspace_bytes.restype = c_size_t
    lib.compactor_compress_full_workspace_bytes.argtypes = [POINTER(CompactorShape), POINTER(CompactorOptions)]
    lib.compactor_compress_full.argtypes = [POINTER(CompactorShape), POINTER(CompactorOptions), CompactorMat, CompactorMat,
                                            CompactorMat, CompactorMat, c_void_p, POINTER(c_int32), c_void_p, c_void_p,
                                            c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.compactor_wait_selftest.argtypes = [c_void_p, c_void_p]
    lib.compactor_builtin_scratch_bytes.restype = c_size_t
    lib.compactor_score_builtin_scratch.argtypes = [POINTER(CompactorShape), CompactorMat, c_void_p, c_void_p, c_float,
                                                    c_void_p, c_void_p, c_void_p]
    return lib


LIB = _load()
LIB_PATH = _build.LIB

EXPORTS = ["compactor_version", "compactor_error_string", "compactor_make_sketch", "compactor_make_sketch_srht", "compactor_keep_count",
           "compactor_calibrated_ratio", "compactor_fit_calibration", "compactor_workspace_bytes", "compactor_score", "compactor_select",
           "compactor_compact", "compactor_compress", "compactor_compress_profiled",
           "compactor_builtin_scratch_bytes", "compactor_score_builtin_scratch", "compactor_attention_scores", "compactor_attention_scores_status", "compactor_wait_selftest",
           "compactor_across_heads_workspace_bytes", "compactor_select_across_heads", "compactor_compact_across_heads",
           "compactor_score_variant", "compactor_nll", "compactor_compress_full_workspace_bytes", "compactor_compress_full"]

FACTOR_CHOLESKY = 0
FACTOR_EIG = 1
SELECT_PER_HEAD = 0
SELECT_ACROSS_HEADS = 1

N_STAGE_EVENTS = 7
STAGE_NAMES = ["gram", "factor", "score", "blend", "select", "compact"]


def version() -> int:
    return LIB.compactor_version()


def error_string(code: int) -> str:
    return LIB.compactor_error_string(code).decode()


def _check(code: int, where: str) -> None:
    if code != 0:
        raise CompactorError(code, where)


class Shape:
    """Owns the host arrays a compactor_shape points to."""

    def __init__(self, layers: int, heads: int, d: int, m: int, seqlens: Sequence[int]):
        self.seqlens = [int(n) for n in seqlens]
        cu = [0]
        for n in self.seqlens:
            cu.append(cu[-1] + n)
        self._cu = (c_int32 * len(cu))(*cu)
        self.cu_seqlens = cu
        self.c = CompactorShape(layers, heads, d, m, len(self.seqlens), self._cu)
        self.layers, self.heads, self.d, self.m = layers, heads, d, m
        self.total_tokens = cu[-1]

    @property
    def batch(self) -> int:
        return len(self.seqlens)


def mat(t: torch.Tensor) -> CompactorMat:
    """A [layers, heads, tokens, d] bf16 CUDA tensor (any strides with a contiguous last axis)."""
    assert t.is_cuda and t.dtype == torch.bfloat16 and t.dim() == 4 and t.stride(3) == 1
    return CompactorMat(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else c_void_p(t.data_ptr())


def _stream() -> c_void_p:
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _keep_array(keep_counts: Sequence[int]):
    return (c_int32 * len(keep_counts))(*[int(k) for k in keep_counts])


def make_sketch(seed: int, d: int, m: int) -> torch.Tensor:
    out = torch.empty(d, m, dtype=torch.float32)
    _check(LIB.compactor_make_sketch(seed, d, m, ctypes.cast(out.data_ptr(), POINTER(c_float))), "compactor_make_sketch")
    return out


def make_sketch_srht(seed: int, d: int, m: int) -> torch.Tensor:
    out = torch.empty(d, m, dtype=torch.float32)
    _check(LIB.compactor_make_sketch_srht(seed, d, m, ctypes.cast(out.data_ptr(), POINTER(c_float))),
           "compactor_make_sketch_srht")
    return out


def keep_count(n: int, r: float) -> int:
    return int(LIB.compactor_keep_count(int(n), float(r)))


def calibrated_ratio(nll: float, alpha: float, beta: float, tau: float) -> float:
    r = c_double()
    _check(LIB.compactor_calibrated_ratio(nll, alpha, beta, tau, byref(r)), "compactor_calibrated_ratio")
    return r.value


def fit_calibration(r: Sequence[float], nll: Sequence[float], y: Sequence[float], under_weight: float = 1.0):
    """Returns (alpha, beta, loss) of the asymmetric least-squares fit of the calibration curve."""
    n = len(r)
    arr = lambda v: (c_double * n)(*[float(x) for x in v])
    al, be, loss = c_double(), c_double(), c_double()
    _check(LIB.compactor_fit_calibration(n, arr(r), arr(nll), arr(y), under_weight, byref(al), byref(be), byref(loss)),
           "compactor_fit_calibration")
    return al.value, be.value, loss.value


def workspace_bytes(shape: Shape) -> int:
    return int(LIB.compactor_workspace_bytes(byref(shape.c)))


def alloc_workspace(shape: Shape, device="cuda") -> torch.Tensor:
    return torch.empty(max(256, workspace_bytes(shape)), dtype=torch.uint8, device=device)


def score(shape: Shape, k_score: torch.Tensor, phi: torch.Tensor, scores_out: torch.Tensor, workspace: torch.Tensor,
          attn: Optional[torch.Tensor] = None, lam: float = 0.3, status: Optional[torch.Tensor] = None) -> None:
    _check(LIB.compactor_score(byref(shape.c), mat(k_score), _ptr(phi), _ptr(attn), lam, _ptr(scores_out),
                               _ptr(status), _ptr(workspace), workspace.numel(), _stream()), "compactor_score")


def score_variant(shape: Shape, k_score: torch.Tensor, phi: torch.Tensor, scores_out: torch.Tensor,
                  workspace: torch.Tensor, factorization: int, eig_floor: float = 1e-6,
                  attn: Optional[torch.Tensor] = None, lam: float = 0.3, status: Optional[torch.Tensor] = None) -> None:
    """Appendix C: `score` with the small factorisation chosen (FACTOR_CHOLESKY or FACTOR_EIG)."""
    _check(LIB.compactor_score_variant(byref(shape.c), mat(k_score), _ptr(phi), factorization, eig_floor, _ptr(attn), lam,
                                       _ptr(scores_out), _ptr(status), _ptr(workspace), workspace.numel(), _stream()),
           "compactor_score_variant")


def nll(logits: torch.Tensor, targets: torch.Tensor, seq_rows: Sequence[int], row_nll_out: torch.Tensor,
        nll_out: torch.Tensor) -> None:
    """Section 3.5: token-averaged NLL of each sequence from `logits` [rows, vocab] (bf16 or fp32,
    unit stride along the vocabulary) and `targets` [rows] (int32, negative = unscored)."""
    if logits.dtype == torch.bfloat16:
        dtype = 0
    elif logits.dtype == torch.float32:
        dtype = 1
    else:
        raise TypeError("logits must be bf16 or fp32")
    if logits.dim() != 2 or logits.stride(1) != 1 or targets.dtype != torch.int32:
        raise ValueError("logits [rows, vocab] with unit inner stride and int32 targets expected")
    cu = [0]
    for n in seq_rows:
        cu.append(cu[-1] + int(n))
    cu_arr = (c_int32 * len(cu))(*cu)
    _check(LIB.compactor_nll(_ptr(logits), dtype, logits.shape[0], logits.shape[1], logits.stride(0), _ptr(targets),
                             len(seq_rows), cu_arr, _ptr(row_nll_out), _ptr(nll_out), _stream()), "compactor_nll")


def select(shape: Shape, scores: torch.Tensor, keep_counts: Sequence[int], idx_out: torch.Tensor,
           workspace: torch.Tensor, status: Optional[torch.Tensor] = None) -> None:
    _check(LIB.compactor_select(byref(shape.c), _ptr(scores), _keep_array(keep_counts), _ptr(idx_out), _ptr(status),
                                _ptr(workspace), workspace.numel(), _stream()), "compactor_select")


def compact(shape: Shape, k_cache: torch.Tensor, v_cache: torch.Tensor, idx: torch.Tensor, keep_counts: Sequence[int],
            k_out: torch.Tensor, v_out: torch.Tensor, workspace: torch.Tensor) -> None:
    _check(LIB.compactor_compact(byref(shape.c), mat(k_cache), mat(v_cache), _ptr(idx), _keep_array(keep_counts),
                                 _ptr(k_out), _ptr(v_out), _ptr(workspace), workspace.numel(), _stream()),
           "compactor_compact")


def compress(shape: Shape, k_score: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, phi: torch.Tensor,
             keep_counts: Sequence[int], idx_out: torch.Tensor, k_out: torch.Tensor, v_out: torch.Tensor,
             workspace: torch.Tensor, attn: Optional[torch.Tensor] = None, lam: float = 0.3,
             scores_out: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None) -> None:
    _check(LIB.compactor_compress(byref(shape.c), mat(k_score), mat(k_cache), mat(v_cache), _ptr(phi), _ptr(attn), lam,
                                  _keep_array(keep_counts), _ptr(scores_out), _ptr(idx_out), _ptr(k_out), _ptr(v_out),
                                  _ptr(status), _ptr(workspace), workspace.numel(), _stream()), "compactor_compress")


def compress_profiled(shape: Shape, k_score: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                      phi: torch.Tensor, keep_counts: Sequence[int], idx_out: torch.Tensor, k_out: torch.Tensor,
                      v_out: torch.Tensor, workspace: torch.Tensor, events: Sequence[torch.cuda.Event],
                      attn: Optional[torch.Tensor] = None, lam: float = 0.3,
                      scores_out: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None) -> None:
    """`events`: N_STAGE_EVENTS torch events with timing enabled that have been recorded once before
    (so that their CUDA handles exist); the library re-records them between its kernels."""
    handles = (c_void_p * len(events))(*[c_void_p(e.cuda_event) for e in events])
    _check(LIB.compactor_compress_profiled(byref(shape.c), mat(k_score), mat(k_cache), mat(v_cache), _ptr(phi),
                                           _ptr(attn), lam, _keep_array(keep_counts), _ptr(scores_out), _ptr(idx_out),
                                           _ptr(k_out), _ptr(v_out), _ptr(status), _ptr(workspace), workspace.numel(),
                                           _stream(), handles, len(events)), "compactor_compress_profiled")


def builtin_scratch_bytes() -> int:
    return int(LIB.compactor_builtin_scratch_bytes())


def score_builtin_scratch(shape: Shape, k_score: torch.Tensor, phi: torch.Tensor, scores_out: torch.Tensor,
                          attn: Optional[torch.Tensor] = None, lam: float = 0.3,
                          status: Optional[torch.Tensor] = None) -> None:
    """compactor_score without a workspace: for callers that may not allocate device memory.  The
    scratch is the library's fixed 32 MiB array; problems that do not fit raise CompactorError(-5)."""
    _check(LIB.compactor_score_builtin_scratch(byref(shape.c), mat(k_score), _ptr(phi), _ptr(attn), lam,
                                               _ptr(scores_out), _ptr(status), _stream()),
           "compactor_score_builtin_scratch")


def attention_scores(shape: Shape, q: torch.Tensor, k: torch.Tensor, q_per_kv: int, attn_out: torch.Tensor,
                     workspace: torch.Tensor, scale: float, pool: int = 1, chunk: int = 256,
                     status: Optional[torch.Tensor] = None) -> None:
    """Eq. 5: chunked non-causal attention column sums of `q` [layers, heads*q_per_kv, tokens, d] against `k`."""
    if status is None:
        _check(LIB.compactor_attention_scores(byref(shape.c), mat(q), mat(k), q_per_kv, chunk, scale, pool, _ptr(attn_out),
                                              _ptr(workspace), workspace.numel(), _stream()), "compactor_attention_scores")
    else:
        _check(LIB.compactor_attention_scores_status(byref(shape.c), mat(q), mat(k), q_per_kv, chunk, scale, pool,
                                                     _ptr(attn_out), _ptr(status), _ptr(workspace), workspace.numel(),
                                                     _stream()), "compactor_attention_scores_status")


def across_heads_workspace_bytes(shape: Shape) -> int:
    return int(LIB.compactor_across_heads_workspace_bytes(byref(shape.c)))


def select_across_heads(shape: Shape, scores: torch.Tensor, keep_counts: Sequence[int], idx_out: torch.Tensor,
                        head_offsets_out: torch.Tensor, workspace: torch.Tensor) -> None:
    _check(LIB.compactor_select_across_heads(byref(shape.c), _ptr(scores), _keep_array(keep_counts), _ptr(idx_out),
                                             _ptr(head_offsets_out), _ptr(workspace), workspace.numel(), _stream()),
           "compactor_select_across_heads")


def compact_across_heads(shape: Shape, k_cache: torch.Tensor, v_cache: torch.Tensor, idx: torch.Tensor,
                         head_offsets: torch.Tensor, keep_counts: Sequence[int], k_out: torch.Tensor,
                         v_out: torch.Tensor, workspace: torch.Tensor) -> None:
    _check(LIB.compactor_compact_across_heads(byref(shape.c), mat(k_cache), mat(v_cache), _ptr(idx), _ptr(head_offsets),
                                              _keep_array(keep_counts), _ptr(k_out), _ptr(v_out), _ptr(workspace),
                                              workspace.numel(), _stream()), "compactor_compact_across_heads")


def options(selection: int = SELECT_PER_HEAD, factorization: int = FACTOR_CHOLESKY, eig_floor: float = 1e-6,
            lam: float = 0.3, q_per_kv: int = 0, chunk: int = 256, scale: float = 128 ** -0.5, pool: int = 1) -> CompactorOptions:
    return CompactorOptions(selection, factorization, eig_floor, lam, q_per_kv, chunk, scale, pool)


def compress_full_workspace_bytes(shape: Shape, opt: CompactorOptions) -> int:
    return int(LIB.compactor_compress_full_workspace_bytes(byref(shape.c), byref(opt)))


def compress_full(shape: Shape, opt: CompactorOptions, q: Optional[torch.Tensor], k_score: torch.Tensor,
                  k_cache: torch.Tensor, v_cache: torch.Tensor, phi: torch.Tensor, keep_counts: Sequence[int],
                  idx_out: torch.Tensor, k_out: torch.Tensor, v_out: torch.Tensor, workspace: torch.Tensor,
                  head_offsets_out: Optional[torch.Tensor] = None, scores_out: Optional[torch.Tensor] = None,
                  status: Optional[torch.Tensor] = None) -> None:
    """The paper's whole method in one call (attention term, leverage scores, blend, selection, gather)."""
    qm = mat(q) if q is not None else CompactorMat(None, 0, 0, 0)
    _check(LIB.compactor_compress_full(byref(shape.c), byref(opt), qm, mat(k_score), mat(k_cache), mat(v_cache), _ptr(phi),
                                       _keep_array(keep_counts), _ptr(scores_out), _ptr(idx_out), _ptr(head_offsets_out),
                                       _ptr(k_out), _ptr(v_out), _ptr(status), _ptr(workspace), workspace.numel(),
                                       _stream()), "compactor_compress_full")


def wait_selftest() -> int:
    """Runs the bounded-wait self-test and returns the status word (4 = the wait gave up as designed)."""
    out = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    _check(LIB.compactor_wait_selftest(_ptr(out), _stream()), "compactor_wait_selftest")
    torch.cuda.synchronize()
    return int(out.item())

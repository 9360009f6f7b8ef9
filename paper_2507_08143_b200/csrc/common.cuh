// Internal declarations shared by the kernels and the host entry points of the library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "compactor.h"

namespace compactor {

constexpr int kD = 128;            // head dimension the kernels are written for
constexpr int kMaxM = 128;          // largest sketch dimension
constexpr int kMaxChunk = 65536;   // most tokens per block (one CTA of a streaming kernel)
constexpr int kMinChunk = 256;
constexpr int kGramFlushTokens = 512;    // most tokens whose Gram matrix is summed in fp32 (tensor-core accumulators) before going to fp64
constexpr int kGramElems = kD * kD;
constexpr int kFactorSlices = 4;   // 32-row slices of the Gram matrix in its fp64 projection
constexpr int kTinyExtra = 16;     // a unit of at most m + kTinyExtra tokens is factored with pivoting and scored in fp64 by the factor kernel
constexpr int kFactorParts = 2;    // parts of A (G = A + A^T) per unit, one per pair of slices and work item

// Device-side view of one call: shapes plus the four prefix-sum tables that live at the start
// of the workspace.  Passed to kernels by value.
struct Plan {
    int layers, heads, batch;
    int m;                 // sketch dimension
    int mp;                // m rounded up to a multiple of 16 (padded columns of W are zero)
    int chunk;             // tokens per block = per Gram partial (multiple of 128)
    int total_chunks;      // Gram partials per (layer, head): sum_b ceil(n_b / chunk)
    int total_tokens;      // per (layer, head)
    int total_keep;        // per (layer, head)
    const int* cu_seqlens; // device [batch+1]
    const int* cu_keep;    // device [batch+1]
    const int* cu_chunks;  // device [batch+1]
    int schunk;            // tokens per block of the scoring sweep (no partial sums there: shorter blocks balance better)
    int total_schunks;     // its blocks per (layer, head): sum_b ceil(n_b / schunk)
    const int* cu_schunks; // device [batch+1]
};

struct Mat {               // compactor_mat with a typed pointer
    const __nv_bfloat16* ptr;
    long long stride_layer, stride_head, stride_token;
};

// Shared state of the fused sweep's work queue (global memory, zeroed before every launch).  Both
// 64-bit words are only ever changed by compare-and-swap.
struct SweepSched {
    unsigned long long fstate;   // high half: leading units whose slices are all claimed; low half: leading units whose Gram pieces are all in
    unsigned long long sstate;   // high half: leading units whose scoring pieces are all claimed; low half: leading units whose W is written
    unsigned int gram_next;      // Gram pieces claimed
    unsigned int abort;          // a bounded wait ran out somewhere: everybody leaves
    unsigned int pad[10];
};

// Arguments of the fused sweep.  `p.chunk` is the piece length and `p.total_chunks` / `p.cu_chunks`
// count pieces; `p.total_schunks` / `p.cu_schunks` count the row slices of the factor tasks.
struct SweepArgs {
    Plan p;
    Mat k;
    int units, total_pieces;
    int total_ftasks;            // factor tasks: (layer, head) x sum over sequences of their row slices (p.cu_schunks, p.total_schunks)
    int window;                  // Gram pieces may run this far ahead of the scoring front
    int n_slots;                 // partial slots (>= window + CTAs); piece i uses slot i % n_slots
    int phase;                   // 0: one launch does everything; 1: Gram pieces and factor tasks only; 2: scoring pieces only
    int resident16;              // sixteenths of a unit's pieces whose keys are meant to wait in L2 for the second read
    SweepSched* sched;
    int* gram_done;              // [units] finished Gram pieces
    int* slices_claimed;         // [units] claimed slice tasks (may overshoot)
    int* slices_done;            // [units] finished slice tasks
    int* score_claimed;          // [units] claimed scoring pieces (may overshoot)
    int* w_ready;                // [units] 1 once W is written
    float* partials;             // [n_slots][128][128] fp32
    double* t_buf;               // [units][128][mp] fp64: T = C Phi
    __nv_bfloat16* w;            // [units][2][mp][128]
    const float* phi;            // [128][m] fp32
    float* scores;
    int* status;
    long long* prof;             // per-CTA cycle counters of an instrumented build, else null
};

// Largest b with table[b] <= x, for a non-decreasing table of nb+1 entries with table[0] = 0.
__device__ __forceinline__ int find_segment(const int* __restrict__ table, int nb, int x) {
    int lo = 0, hi = nb;          // invariant: table[lo] <= x < table[hi] (table[nb] > x by construction)
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (table[mid] <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// Programmatic dependent launch.  A kernel of the fused call's chain is launched so that it may start
// while its predecessor in the stream is still running: its CTAs are scheduled as soon as every CTA of the
// predecessor has called pdl_trigger() (first thing) or exited, do their set-up (shared memory, barriers,
// operands that come from the caller), and then pdl_wait() until the predecessor has finished and its
// writes are visible.  Everything a kernel reads that an earlier kernel of the call wrote is read after
// pdl_wait(); a kernel launched without the attribute passes through both calls.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
bool pdl_enabled(int which);
enum { kPdlProject = 1, kPdlCholesky = 2, kPdlScore = 4, kPdlSelect = 8, kPdlCompact = 16, kPdlOther = 32 };
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(int which, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                  Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled(which) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Kernel launchers (each defined next to its kernel).  All enqueue on `stream` and return the
// launch status.
cudaError_t launch_gram(const Plan& p, const Mat& k, double* partials, int* status, cudaStream_t stream);
// `scores`: where the Cholesky route writes the scores of its tiny units (see kTinyExtra); the scoring sweep is then
// told to leave those units alone (`tiny_done`).
cudaError_t launch_factor(const Plan& p, const Mat& k, const double* partials, const float* phi, double* a_parts,
                          __nv_bfloat16* w, float* scores, int* status, int factorization, double eig_floor, int sm_count,
                          cudaStream_t stream);
cudaError_t launch_score(const Plan& p, const Mat& k, const __nv_bfloat16* w, float* scores, int* status, bool tiny_done,
                         cudaStream_t stream);
cudaError_t launch_sweep(const SweepArgs& a, int sm_count, cudaStream_t stream);
// parts > 1 (with `stats`, 4 doubles per unit and part): every unit's vectors are cut into that many slices.
cudaError_t launch_blend(const Plan& p, const float* attn, float lambda, float* scores, int parts, double* stats,
                         cudaStream_t stream);
cudaError_t launch_select(const Plan& p, const float* scores, int* idx, cudaStream_t stream);
cudaError_t launch_compact(const Plan& p, const Mat& k, const Mat& v, const int* idx,
                           __nv_bfloat16* k_out, __nv_bfloat16* v_out, cudaStream_t stream);

cudaError_t launch_nll(const void* logits, int is_fp32, long long rows, int vocab, long long row_stride,
                       const int* targets, int batch, const int* cu_rows_host, float* row_nll, double* nll_out,
                       cudaStream_t stream);

// Scratch of the selection that spreads a score vector over several CTAs (select.cu).  A group is what
// shares a threshold: one unit, or, when selecting across heads, a (layer, sequence) pair with all its heads.
constexpr int kSelStateInts = 2176;       // per group: 2048 histogram bins, range, counters, per-head counts
constexpr int kSelCandBase = 4096;        // candidate capacity of a group: this + (scores of the group) / kSelCandDiv
constexpr int kSelCandDiv = 256;
struct MultiSelect {
    int* state;                // [groups][kSelStateInts]
    uint2* cand;               // (key, head) pairs; a group's list starts where decode_group() says
    int2* counts;              // [units][parts]: scores above / at the threshold per slice
    uint32_t* thr;             // [groups]
    int* ties;                 // [units]
    long long cand_per_outer;  // list entries per layer (across heads) or per (layer, head)
    int parts;                 // slices per score vector
    int across;
};
struct MultiSelectLayout {
    size_t off_state, off_cand, off_counts, off_thr, off_ties, total;
    long long cand_per_outer;
};
// Offsets (relative to a 256-byte aligned base) of the scratch for the given problem.
inline MultiSelectLayout multi_select_layout(int layers, int heads, int batch, long long total_tokens, bool across,
                                             int parts) {
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    const size_t outer = across ? (size_t)layers : (size_t)layers * heads;
    const size_t groups = outer * batch, units = (size_t)layers * heads * batch;
    MultiSelectLayout l;
    l.cand_per_outer = (long long)batch * (kSelCandBase + 1) + ((long long)(across ? heads : 1) * total_tokens) / kSelCandDiv + 1;
    size_t off = 0;
    l.off_state = off;  off += up(sizeof(int) * groups * kSelStateInts);
    l.off_cand = off;   off += up(sizeof(uint2) * outer * (size_t)l.cand_per_outer);
    l.off_counts = off; off += up(sizeof(int2) * units * (size_t)parts);
    l.off_thr = off;    off += up(sizeof(uint32_t) * groups);
    l.off_ties = off;   off += up(sizeof(int) * units);
    l.total = off;
    return l;
}
inline MultiSelect multi_select_at(char* base, const MultiSelectLayout& l, int parts, bool across) {
    MultiSelect m;
    m.state = reinterpret_cast<int*>(base + l.off_state);
    m.cand = reinterpret_cast<uint2*>(base + l.off_cand);
    m.counts = reinterpret_cast<int2*>(base + l.off_counts);
    m.thr = reinterpret_cast<uint32_t*>(base + l.off_thr);
    m.ties = reinterpret_cast<int*>(base + l.off_ties);
    m.cand_per_outer = l.cand_per_outer;
    m.parts = parts;
    m.across = across ? 1 : 0;
    return m;
}
cudaError_t launch_select_multi(const Plan& p, const float* scores, int* idx, int* head_offsets, const MultiSelect& m,
                                cudaStream_t stream);
cudaError_t launch_compact_across(const Plan& p, const Mat& k, const Mat& v, const int* idx, const int* head_offsets,
                                  __nv_bfloat16* k_out, __nv_bfloat16* v_out, cudaStream_t stream);
cudaError_t launch_attention(const Plan& p, const Mat& q, const Mat& k, int q_per_kv, float scale, int pool,
                             float* raw, float* out, int* status, cudaStream_t stream);

// Bytes of W (two bf16 terms, [term][mp][128]) per unit.
__host__ __device__ inline size_t w_elems_per_unit(int mp) { return (size_t)2 * mp * kD; }
// doubles per unit between the projection and the factorisation: the parts of A (never less than what one T = C Phi takes,
// which the one-kernel sweep keeps there)
__host__ __device__ inline size_t a_elems_per_unit(int mp) {
    const size_t parts = (size_t)kFactorParts * mp * mp, t = (size_t)kD * mp;
    return parts > t ? parts : t;
}

}  // namespace compactor

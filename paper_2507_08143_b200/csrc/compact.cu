// Compaction (Section 3, Preliminaries: only the selected fraction of the tokens is retained):
// gathers the kept rows of K and V of every unit into dense [total_keep][128] blocks.  Each
// 256-byte row is moved by 16 threads as 128-bit pieces; bit-exact.
#include "common.cuh"

namespace compactor {
namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerIter = kThreads / 16;     // 16 rows in flight per instruction
// One row pair (K and V piece) in flight per thread and step: the loads are kept in flight by
// occupancy (38 registers, eight CTAs per SM) rather than by unrolling, which measured 6 % faster.
constexpr int kUnroll = 1;
constexpr int kSteps = 8;
constexpr int kRowsPerCta = kRowsPerIter * kUnroll * kSteps;   // 128 output rows per CTA

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

__global__ void __launch_bounds__(kThreads)
compact_kernel(Plan p, Mat k, Mat v, const int* __restrict__ idx,
               __nv_bfloat16* __restrict__ k_out, __nv_bfloat16* __restrict__ v_out) {
    pdl_trigger();
    pdl_wait();                                            // the indices are complete
    const int lh = blockIdx.y;
    const int layer = lh / p.heads, head = lh % p.heads;
    const int piece = threadIdx.x & 15, sub = threadIdx.x >> 4;
    const int* idx_lh = idx + (size_t)lh * p.total_keep;
    const __nv_bfloat16* kb = k.ptr + layer * k.stride_layer + head * k.stride_head;
    const __nv_bfloat16* vb = v.ptr + layer * v.stride_layer + head * v.stride_head;
    uint4* ko = reinterpret_cast<uint4*>(k_out + (size_t)lh * p.total_keep * kD);
    uint4* vo = reinterpret_cast<uint4*>(v_out + (size_t)lh * p.total_keep * kD);

    const int row0 = blockIdx.x * kRowsPerCta;
#pragma unroll
    for (int half = 0; half < kSteps; ++half) {
        uint4 kv[kUnroll], vv[kUnroll];
        int rows[kUnroll];
        bool ok[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            int row = row0 + (half * kUnroll + u) * kRowsPerIter + sub;
            rows[u] = row;
            ok[u] = false;
            if (row < p.total_keep) {
                int b = find_segment(p.cu_keep, p.batch, row);
                int n = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
                int local = idx_lh[row];
                if (local >= 0 && local < n) {
                    long long tok = (long long)p.cu_seqlens[b] + local;
                    kv[u] = ld_stream(reinterpret_cast<const uint4*>(kb + tok * k.stride_token) + piece);
                    vv[u] = ld_stream(reinterpret_cast<const uint4*>(vb + tok * v.stride_token) + piece);
                    ok[u] = true;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (ok[u]) {
                st_stream(ko + (size_t)rows[u] * 16 + piece, kv[u]);
                st_stream(vo + (size_t)rows[u] * 16 + piece, vv[u]);
            }
        }
    }
}

// The same gather for selection across heads: the output rows of layer l are laid out sequence
// by sequence, and inside a sequence's block of heads * kk rows head by head at the offsets the
// selection wrote (head_offsets [layer][sequence][heads + 1]).
__global__ void __launch_bounds__(kThreads)
compact_across_kernel(Plan p, Mat k, Mat v, const int* __restrict__ idx, const int* __restrict__ head_offsets,
                      __nv_bfloat16* __restrict__ k_out, __nv_bfloat16* __restrict__ v_out) {
    pdl_trigger();
    pdl_wait();                                            // indices and head offsets are complete
    const int layer = blockIdx.y;
    const int piece = threadIdx.x & 15, sub = threadIdx.x >> 4;
    const long long rows_per_layer = (long long)p.heads * p.total_keep;
    const int* idx_l = idx + (size_t)layer * rows_per_layer;
    uint4* ko = reinterpret_cast<uint4*>(k_out + (size_t)layer * rows_per_layer * kD);
    uint4* vo = reinterpret_cast<uint4*>(v_out + (size_t)layer * rows_per_layer * kD);
    const long long row0 = (long long)blockIdx.x * kRowsPerCta;
#pragma unroll
    for (int half = 0; half < kSteps; ++half) {
        uint4 kv[kUnroll], vv[kUnroll];
        long long rows[kUnroll];
        bool ok[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const long long row = row0 + (half * kUnroll + u) * kRowsPerIter + sub;
            rows[u] = row;
            ok[u] = false;
            if (row < rows_per_layer) {
                const int b = find_segment(p.cu_keep, p.batch, (int)(row / p.heads));   // blocks start at heads * cu_keep[b]
                const int r = (int)(row - (long long)p.heads * p.cu_keep[b]);
                const int* offs = head_offsets + ((size_t)layer * p.batch + b) * (p.heads + 1);
                const int head = find_segment(offs, p.heads, r);
                const int n = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
                const int local = idx_l[row];
                if (local >= 0 && local < n) {
                    const long long tok = (long long)p.cu_seqlens[b] + local;
                    kv[u] = ld_stream(reinterpret_cast<const uint4*>(k.ptr + layer * k.stride_layer + head * k.stride_head +
                                                                     tok * k.stride_token) + piece);
                    vv[u] = ld_stream(reinterpret_cast<const uint4*>(v.ptr + layer * v.stride_layer + head * v.stride_head +
                                                                     tok * v.stride_token) + piece);
                    ok[u] = true;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (ok[u]) {
                st_stream(ko + (size_t)rows[u] * 16 + piece, kv[u]);
                st_stream(vo + (size_t)rows[u] * 16 + piece, vv[u]);
            }
        }
    }
}

}  // namespace

cudaError_t launch_compact_across(const Plan& p, const Mat& k, const Mat& v, const int* idx, const int* head_offsets,
                                  __nv_bfloat16* k_out, __nv_bfloat16* v_out, cudaStream_t stream) {
    const long long rows = (long long)p.heads * p.total_keep;
    if (rows == 0 || p.layers == 0) return cudaSuccess;
    dim3 grid((unsigned)((rows + kRowsPerCta - 1) / kRowsPerCta), p.layers);
    cudaError_t e = launch_chained(kPdlCompact, compact_across_kernel, grid, dim3(kThreads), 0, stream, p, k, v, idx, head_offsets, k_out, v_out);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_compact(const Plan& p, const Mat& k, const Mat& v, const int* idx,
                           __nv_bfloat16* k_out, __nv_bfloat16* v_out, cudaStream_t stream) {
    if (p.total_keep == 0 || p.layers * p.heads == 0) return cudaSuccess;
    dim3 grid((p.total_keep + kRowsPerCta - 1) / kRowsPerCta, p.layers * p.heads);
    cudaError_t e = launch_chained(kPdlCompact, compact_kernel, grid, dim3(kThreads), 0, stream, p, k, v, idx, k_out, v_out);
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace compactor

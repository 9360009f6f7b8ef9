// Small factorisation, one CTA per unit (Algorithm 1, line 4, by the Cholesky route that
// Section 3.2 and Appendix C allow): sum the unit's Gram partials in fp64, project
// G = Phi^T C Phi, factor G = L L^T, and emit the back-projection matrix W = Phi L^-T split
// into two bf16 terms, so that line 5-6's score of a key row k_i is || k_i W ||^2.
//
// Rank handling: a pivot not larger than 2^-20 of its original diagonal entry (the fp32 noise
// floor of the Gram sums) is treated as a direction of the null space and dropped; with the
// remaining pivot set P, W = Phi[:, P] L_PP^-T, which equals the pseudo-inverse reading
// o_i = k^_i G^+ k^_i^T whenever k^_i lies in the range of G.
#include "common.cuh"

namespace compactor {
namespace {

constexpr int kThreads = 512;
constexpr double kPivotFloor = 9.5367431640625e-07;   // 2^-20
// Sequences this short are near the sketch dimension, where G is close to singular and the fp32
// rounding of the Gram partials would dominate the scores; their Gram matrix is summed here in
// fp64 straight from the keys instead (the work is tiny).
constexpr int kExactGramTokens = 256;
constexpr int kStageTokens = 32;

// Dynamic shared memory: C (fp64, 128 KB; its space is reused for G once T exists), T = C Phi,
// Phi (fp32), then the small per-column state.
struct FactorTail {
    double diag0[kMaxM];        // original diagonal of G
    int pivot[kMaxM];           // 1 = column kept
    int flags;
};

__host__ __device__ inline size_t factor_smem_bytes(int mp) {
    return sizeof(double) * kGramElems + sizeof(double) * kD * mp + sizeof(float) * kD * mp + sizeof(FactorTail);
}

__global__ void __launch_bounds__(kThreads, 1)
factor_kernel(Plan p, Mat kmat, const float* __restrict__ partials, const float* __restrict__ phi,
              __nv_bfloat16* __restrict__ w_out, int* __restrict__ status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int m = p.m, mp = p.mp;
    double* s_c = reinterpret_cast<double*>(smem_raw);
    double* s_g = s_c;                                   // valid after T has been formed
    double* s_t = s_c + kGramElems;
    float* s_phi = reinterpret_cast<float*>(s_t + kD * mp);
    FactorTail& s = *reinterpret_cast<FactorTail*>(s_phi + kD * mp);

    const int unit = blockIdx.x;
    const int b = unit % p.batch;
    const int lh = unit / p.batch;
    const int tid = threadIdx.x;
    const int chunk_begin = p.cu_chunks[b], chunk_end = p.cu_chunks[b + 1];
    const float* part = partials + ((size_t)lh * p.total_chunks + chunk_begin) * kGramElems;
    const int n_part = chunk_end - chunk_begin;
    const int n_tok = p.cu_seqlens[b + 1] - p.cu_seqlens[b];

    for (int i = tid; i < kD * mp; i += kThreads) {
        int row = i / mp, col = i % mp;
        s_phi[i] = (col < m) ? phi[row * m + col] : 0.f;
    }
    if (tid == 0) s.flags = 0;

    // C = sum of the unit's fp32 partials, in fp64.
    {
        constexpr int kPer = kGramElems / (kThreads * 4);      // float4 groups per thread
        double acc[kPer][4];
#pragma unroll
        for (int q = 0; q < kPer; ++q) acc[q][0] = acc[q][1] = acc[q][2] = acc[q][3] = 0.0;
        if (n_tok > kExactGramTokens) {
            for (int pp = 0; pp < n_part; ++pp) {
                const float4* src = reinterpret_cast<const float4*>(part + (size_t)pp * kGramElems);
#pragma unroll
                for (int q = 0; q < kPer; ++q) {
                    float4 v = __ldcs(src + tid + q * kThreads);
                    acc[q][0] += (double)v.x; acc[q][1] += (double)v.y;
                    acc[q][2] += (double)v.z; acc[q][3] += (double)v.w;
                }
            }
        } else {
            // fp64 Gram of a short sequence; keys are staged, widened, in the space of T.
            const int layer = lh / p.heads, head = lh % p.heads;
            const __nv_bfloat16* kbase = kmat.ptr + layer * kmat.stride_layer + head * kmat.stride_head +
                                         (long long)p.cu_seqlens[b] * kmat.stride_token;
            for (int t0 = 0; t0 < n_tok; t0 += kStageTokens) {
                const int nt = min(kStageTokens, n_tok - t0);
                __syncthreads();
                for (int i = tid; i < nt * kD; i += kThreads)
                    s_t[i] = (double)__bfloat162float(kbase[(long long)(t0 + i / kD) * kmat.stride_token + (i % kD)]);
                __syncthreads();
                for (int t = 0; t < nt; ++t) {
                    const double* krow = s_t + t * kD;
#pragma unroll
                    for (int q = 0; q < kPer; ++q) {
                        int e = (tid + q * kThreads) * 4;
                        double a = krow[e / kD];
                        const double* kc = krow + (e % kD);
                        acc[q][0] = fma(a, kc[0], acc[q][0]); acc[q][1] = fma(a, kc[1], acc[q][1]);
                        acc[q][2] = fma(a, kc[2], acc[q][2]); acc[q][3] = fma(a, kc[3], acc[q][3]);
                    }
                }
            }
        }
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            int e = (tid + q * kThreads) * 4;
            s_c[e] = acc[q][0]; s_c[e + 1] = acc[q][1]; s_c[e + 2] = acc[q][2]; s_c[e + 3] = acc[q][3];
        }
    }
    __syncthreads();

    // T[i][j] = sum_k C[k][i] Phi[k][j] (C is symmetric; reading it by columns keeps a warp's eight
    // rows on consecutive words).  Four threads share a row i, each owning every fourth column.
    {
        const int row = tid >> 2, q = tid & 3;
        double acc[kMaxM / 4];
#pragma unroll
        for (int c = 0; c < kMaxM / 4; ++c) acc[c] = 0.0;
        for (int k = 0; k < kD; ++k) {
            const double cv = s_c[k * kD + row];
            const float* prow = s_phi + k * mp;
#pragma unroll
            for (int c = 0; c < kMaxM / 4; ++c) {
                int col = q + 4 * c;
                if (col < mp) acc[c] = fma(cv, (double)prow[col], acc[c]);
            }
        }
#pragma unroll
        for (int c = 0; c < kMaxM / 4; ++c) {
            int col = q + 4 * c;
            if (col < mp) s_t[row * mp + col] = acc[c];
        }
    }
    __syncthreads();

    // G = Phi^T T (mp x mp); padded rows/columns are zero.  Overwrites the space of C.
    for (int e = tid; e < mp * mp; e += kThreads) {
        int i = e / mp, j = e % mp;
        double acc = 0.0;
        for (int k = 0; k < kD; ++k) acc = fma((double)s_phi[k * mp + i], s_t[k * mp + j], acc);
        s_g[e] = acc;
        if (!isfinite(acc)) atomicOr(&s.flags, COMPACTOR_STATUS_NONFINITE);
    }
    __syncthreads();
    if (tid < mp) s.diag0[tid] = s_g[tid * mp + tid];
    __syncthreads();

    const bool bad = (s.flags & COMPACTOR_STATUS_NONFINITE) != 0;
    if (!bad) {
        // Right-looking Cholesky on the leading m x m block with dropped (null) pivots.
        for (int j = 0; j < m; ++j) {
            double piv = s_g[j * mp + j];
            bool keep = piv > kPivotFloor * s.diag0[j] && s.diag0[j] > 0.0;   // same value in every thread
            double ljj = keep ? sqrt(piv) : 0.0;
            __syncthreads();
            if (tid == 0) {
                s.pivot[j] = keep ? 1 : 0;
                s_g[j * mp + j] = ljj;
                if (!keep) atomicOr(&s.flags, COMPACTOR_STATUS_RANK);
            }
            if (keep) {
                for (int i = j + 1 + tid; i < m; i += kThreads) s_g[i * mp + j] /= ljj;
            } else {
                for (int i = j + 1 + tid; i < m; i += kThreads) s_g[i * mp + j] = 0.0;
            }
            __syncthreads();
            if (keep) {
                const int rem = m - j - 1;
                for (int e = tid; e < rem * rem; e += kThreads) {
                    int i = j + 1 + e / rem, c = j + 1 + e % rem;
                    if (c <= i) s_g[i * mp + c] = fma(-s_g[i * mp + j], s_g[c * mp + j], s_g[i * mp + c]);
                }
            }
            __syncthreads();
        }
    }

    // W[row][:] solves W_P L_PP^T = Phi[row][P]; one thread per key channel (row of Phi).
    __nv_bfloat16* w_hi = w_out + (size_t)unit * w_elems_per_unit(mp);
    __nv_bfloat16* w_lo = w_hi + (size_t)mp * kD;
    if (tid < kD) {
        double wrow[kMaxM];
#pragma unroll 1
        for (int j = 0; j < mp; ++j) {
            double v = 0.0;
            if (!bad && j < m && s.pivot[j]) {
                v = (double)s_phi[tid * mp + j];
                for (int c = 0; c < j; ++c) v = fma(-wrow[c], s_g[j * mp + c], v);
                v /= s_g[j * mp + j];
            }
            wrow[j] = v;
            __nv_bfloat16 hi = __double2bfloat16(v);
            __nv_bfloat16 lo = __double2bfloat16(v - (double)__bfloat162float(hi));
            w_hi[j * kD + tid] = hi;
            w_lo[j * kD + tid] = lo;
        }
    }
    if (tid == 0 && status != nullptr && s.flags != 0) atomicOr(&status[unit], s.flags);
}

}  // namespace

cudaError_t launch_factor(const Plan& p, const Mat& k, const float* partials, const float* phi, __nv_bfloat16* w,
                          int* status, cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    if (units == 0) return cudaSuccess;
    const int smem = (int)factor_smem_bytes(p.mp);
    cudaError_t e = cudaFuncSetAttribute(factor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    factor_kernel<<<units, kThreads, smem, stream>>>(p, k, partials, phi, w, status);
    return cudaGetLastError();
}

}  // namespace compactor

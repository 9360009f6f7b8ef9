// Small factorisation, one CTA per unit (Algorithm 1, line 4, by the Cholesky route that
// Section 3.2 and Appendix C allow): sum the unit's fp64 Gram partials, project
// G = Phi^T C Phi, factor G = L L^T, and emit the back-projection matrix W = Phi L^-T split
// into two bf16 terms, so that line 5-6's score of a key row k_i is || k_i W ||^2.
//
// Rank handling: a pivot not larger than 2^-20 of its original diagonal entry (the fp32 noise
// floor of the 2048-token Gram sums) is treated as a direction of the null space and dropped; with the
// remaining pivot set P, W = Phi[:, P] L_PP^-T, which equals the pseudo-inverse reading
// o_i = k^_i G^+ k^_i^T whenever k^_i lies in the range of G.
//
// Everything is fp64.  The two projections are register-tiled (shared-memory loads and
// fp32->fp64 conversions are the scarce resources, not the FMAs); the factorisation runs in one
// warp (left-looking, reciprocal square roots, no block-wide barriers); the triangular solve
// uses four threads per row of Phi.
#include <type_traits>

#include "common.cuh"

namespace compactor {
namespace {

constexpr int kThreads = 512;
constexpr double kPivotFloor = 9.5367431640625e-07;   // 2^-20
// Sequences this short are near the sketch dimension, where G is close to singular and the fp32
// rounding of the Gram partials would dominate the scores; their Gram matrix is summed here in
// fp64 straight from the keys instead (the work is tiny).
constexpr int kExactGramTokens = 256;
constexpr int kStageTokens = 8;           // 8 KB of widened keys: fits the space of T for every MP

struct FactorTail {
    double inv_diag[kMaxM];     // 1 / L_jj of kept columns, 0 for dropped ones
    int flags;
};

// Shared memory: C (fp64, 128 x 128; its space is reused for G/L with row stride MP+1 and for
// W^T), T = C Phi (fp64, 128 x MP), Phi (fp64 when it fits, else fp32), tail.
template <int MP>
struct FactorCfg {
    static constexpr bool kPhi64 = MP <= 48;
    static constexpr size_t kPhiBytes = (size_t)kD * MP * (kPhi64 ? 8 : 4);
    static constexpr size_t kBytes =
        sizeof(double) * kGramElems + sizeof(double) * kD * MP + kPhiBytes + sizeof(FactorTail);
    static constexpr int kLd = MP + 1;    // odd row stride: a walk down a column spreads over the banks
};

template <int MP>
__global__ void __launch_bounds__(kThreads, 1)
factor_kernel(Plan p, Mat kmat, const double* __restrict__ partials, const float* __restrict__ phi,
              __nv_bfloat16* __restrict__ w_out, int* __restrict__ status) {
    using Cfg = FactorCfg<MP>;
    using PhiT = typename std::conditional<Cfg::kPhi64, double, float>::type;
    constexpr int LD = Cfg::kLd;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int m = p.m;
    double* s_c = reinterpret_cast<double*>(smem_raw);
    double* s_g = s_c;                                   // valid once T has been formed
    double* s_w = s_c + kMaxM * (kMaxM + 1);             // W^T [MP][128], behind G
    double* s_t = s_c + kGramElems;
    PhiT* s_phi = reinterpret_cast<PhiT*>(s_t + kD * MP);
    FactorTail& s = *reinterpret_cast<FactorTail*>(reinterpret_cast<unsigned char*>(s_phi) + Cfg::kPhiBytes);

    const int unit = blockIdx.x;
    const int b = unit % p.batch;
    const int lh = unit / p.batch;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunk_begin = p.cu_chunks[b], chunk_end = p.cu_chunks[b + 1];
    const double* part = partials + ((size_t)lh * p.total_chunks + chunk_begin) * kGramElems;
    const int n_part = chunk_end - chunk_begin;
    const int n_tok = p.cu_seqlens[b + 1] - p.cu_seqlens[b];

    for (int i = tid; i < kD * MP; i += kThreads) {
        int row = i / MP, col = i % MP;
        s_phi[i] = (col < m) ? (PhiT)phi[row * m + col] : (PhiT)0;
    }
    if (tid == 0) s.flags = 0;

    // ---- C = sum of the unit's fp64 partials (two passes of eight double2 per thread, two
    // partials in flight, to stay within the register budget) --------------------------------------
    {
        constexpr int kPerPass = 8;
        constexpr int kPasses = kGramElems / (kThreads * 2 * kPerPass);
        const int layer = lh / p.heads, head = lh % p.heads;
        const __nv_bfloat16* kbase = kmat.ptr + layer * kmat.stride_layer + head * kmat.stride_head +
                                     (long long)p.cu_seqlens[b] * kmat.stride_token;
#pragma unroll 1
        for (int pass = 0; pass < kPasses; ++pass) {
            const int g0 = tid + pass * kPerPass * kThreads;       // first double2 of this pass
            double acc[kPerPass][2];
#pragma unroll
            for (int q = 0; q < kPerPass; ++q) acc[q][0] = acc[q][1] = 0.0;
            if (n_tok > kExactGramTokens) {
                int pp = 0;
                for (; pp + 2 <= n_part; pp += 2) {
                    double2 v[2][kPerPass];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const double2* src = reinterpret_cast<const double2*>(part + (size_t)(pp + u) * kGramElems);
#pragma unroll
                        for (int q = 0; q < kPerPass; ++q) v[u][q] = __ldcs(src + g0 + q * kThreads);
                    }
#pragma unroll
                    for (int u = 0; u < 2; ++u)
#pragma unroll
                        for (int q = 0; q < kPerPass; ++q) { acc[q][0] += v[u][q].x; acc[q][1] += v[u][q].y; }
                }
                for (; pp < n_part; ++pp) {
                    const double2* src = reinterpret_cast<const double2*>(part + (size_t)pp * kGramElems);
#pragma unroll
                    for (int q = 0; q < kPerPass; ++q) {
                        double2 v = __ldcs(src + g0 + q * kThreads);
                        acc[q][0] += v.x; acc[q][1] += v.y;
                    }
                }
            } else {
                // fp64 Gram of a short sequence; keys are staged, widened, in the space of T.
                for (int t0 = 0; t0 < n_tok; t0 += kStageTokens) {
                    const int nt = min(kStageTokens, n_tok - t0);
                    __syncthreads();
                    for (int i = tid; i < nt * kD; i += kThreads)
                        s_t[i] = (double)__bfloat162float(kbase[(long long)(t0 + i / kD) * kmat.stride_token + (i % kD)]);
                    __syncthreads();
                    for (int t = 0; t < nt; ++t) {
                        const double* krow = s_t + t * kD;
#pragma unroll
                        for (int q = 0; q < kPerPass; ++q) {
                            const int e = (g0 + q * kThreads) * 2;
                            const double a = krow[e / kD];
                            const double* kc = krow + (e % kD);
                            acc[q][0] = fma(a, kc[0], acc[q][0]); acc[q][1] = fma(a, kc[1], acc[q][1]);
                        }
                    }
                }
            }
#pragma unroll
            for (int q = 0; q < kPerPass; ++q) {
                const int e = (g0 + q * kThreads) * 2;
                *reinterpret_cast<double2*>(s_c + e) = make_double2(acc[q][0], acc[q][1]);
            }
        }
    }
    __syncthreads();

    // ---- T = C Phi: 256 threads, each a tile of 4 rows x MP/8 columns.  C is symmetric and is read
    // by columns, so a thread's four rows are 32 contiguous bytes.
    if (tid < 256) {
        constexpr int kCols = MP / 8;
        const int row0 = (tid >> 3) * 4, col0 = (tid & 7) * kCols;
        double acc[4][kCols];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < kCols; ++c) acc[r][c] = 0.0;
#pragma unroll 2
        for (int k = 0; k < kD; ++k) {
            const double2 c01 = *reinterpret_cast<const double2*>(s_c + k * kD + row0);
            const double2 c23 = *reinterpret_cast<const double2*>(s_c + k * kD + row0 + 2);
            double ph[kCols];
#pragma unroll
            for (int c = 0; c < kCols; ++c) ph[c] = (double)s_phi[k * MP + col0 + c];
#pragma unroll
            for (int c = 0; c < kCols; ++c) {
                acc[0][c] = fma(c01.x, ph[c], acc[0][c]);
                acc[1][c] = fma(c01.y, ph[c], acc[1][c]);
                acc[2][c] = fma(c23.x, ph[c], acc[2][c]);
                acc[3][c] = fma(c23.y, ph[c], acc[3][c]);
            }
        }
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < kCols; ++c) s_t[(row0 + r) * MP + col0 + c] = acc[r][c];
    }
    __syncthreads();

    // ---- G = Phi^T T (MP x MP, row stride LD), tiles of 2 rows x MP/16 columns; overwrites C ----
    {
        constexpr int kCols = MP / 16;
        constexpr int kTiles = (MP / 2) * 16;
        if (tid < kTiles) {
            const int i0 = (tid >> 4) * 2, j0 = (tid & 15) * kCols;
            double acc[2][kCols];
#pragma unroll
            for (int c = 0; c < kCols; ++c) acc[0][c] = acc[1][c] = 0.0;
#pragma unroll 2
            for (int k = 0; k < kD; ++k) {
                const double p0 = (double)s_phi[k * MP + i0], p1 = (double)s_phi[k * MP + i0 + 1];
#pragma unroll
                for (int c = 0; c < kCols; ++c) {
                    const double tv = s_t[k * MP + j0 + c];
                    acc[0][c] = fma(p0, tv, acc[0][c]);
                    acc[1][c] = fma(p1, tv, acc[1][c]);
                }
            }
            bool finite = true;
#pragma unroll
            for (int c = 0; c < kCols; ++c) {
                s_g[i0 * LD + j0 + c] = acc[0][c];
                s_g[(i0 + 1) * LD + j0 + c] = acc[1][c];
                finite = finite && isfinite(acc[0][c]) && isfinite(acc[1][c]);
            }
            if (!finite) atomicOr(&s.flags, COMPACTOR_STATUS_NONFINITE);
        }
    }
    __syncthreads();
    const bool bad = (s.flags & COMPACTOR_STATUS_NONFINITE) != 0;

    // ---- Cholesky, left-looking, one warp: at column j lane l owns rows j+l and j+l+32 ----------
    if (warp == 0 && !bad) {
        int rank_flag = 0;
        for (int j = 0; j < m; ++j) {
            double v[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int i = j + lane + 32 * h;
                double a0 = 0.0, a1 = 0.0;
                if (i < m) {
                    a0 = s_g[i * LD + j];
                    int c = 0;
                    for (; c + 2 <= j; c += 2) {
                        a0 = fma(-s_g[i * LD + c], s_g[j * LD + c], a0);
                        a1 = fma(-s_g[i * LD + c + 1], s_g[j * LD + c + 1], a1);
                    }
                    if (c < j) a0 = fma(-s_g[i * LD + c], s_g[j * LD + c], a0);
                }
                v[h] = a0 + a1;
            }
            const double piv = __shfl_sync(0xffffffffu, v[0], 0);
            const double d0 = s_g[j * LD + j];              // still the original diagonal entry
            const bool keep = piv > kPivotFloor * d0 && d0 > 0.0;
            const double inv = keep ? rsqrt(piv) : 0.0;
            if (!keep) rank_flag = 1;
            __syncwarp();
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int i = j + lane + 32 * h;
                if (i < m) s_g[i * LD + j] = (i == j) ? piv * inv : v[h] * inv;
            }
            if (lane == 0) s.inv_diag[j] = inv;
            __syncwarp();
        }
        if (lane == 0 && rank_flag) s.flags |= COMPACTOR_STATUS_RANK;
    }
    __syncthreads();

    // ---- W = Phi L^-T: four threads per row of Phi walk the columns together ---------------------
    {
        const int row = tid >> 2, q = tid & 3;
        for (int j = 0; j < MP; ++j) {
            double part_sum = 0.0;
            if (!bad && j < m)
                for (int c = q; c < j; c += 4) part_sum = fma(s_w[c * kD + row], s_g[j * LD + c], part_sum);
            part_sum += __shfl_xor_sync(0xffffffffu, part_sum, 1);
            part_sum += __shfl_xor_sync(0xffffffffu, part_sum, 2);
            if (q == 0) {
                double wv = 0.0;
                if (!bad && j < m) wv = ((double)s_phi[row * MP + j] - part_sum) * s.inv_diag[j];
                s_w[j * kD + row] = wv;
            }
            __syncwarp();
        }
    }
    __syncthreads();

    __nv_bfloat16* w_hi = w_out + (size_t)unit * w_elems_per_unit(MP);
    __nv_bfloat16* w_lo = w_hi + (size_t)MP * kD;
    for (int i = tid; i < MP * kD; i += kThreads) {
        const double v = s_w[i];
        const __nv_bfloat16 hi = __double2bfloat16(v);
        w_hi[i] = hi;
        w_lo[i] = __double2bfloat16(v - (double)__bfloat162float(hi));
    }
    if (tid == 0 && status != nullptr && s.flags != 0) atomicOr(&status[unit], s.flags);
}

template <int MP>
cudaError_t launch_factor_mp(const Plan& p, const Mat& k, const double* partials, const float* phi, __nv_bfloat16* w,
                             int* status, cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    const int smem = (int)FactorCfg<MP>::kBytes;
    cudaError_t e = cudaFuncSetAttribute(factor_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    factor_kernel<MP><<<units, kThreads, smem, stream>>>(p, k, partials, phi, w, status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_factor(const Plan& p, const Mat& k, const double* partials, const float* phi, __nv_bfloat16* w,
                          int* status, cudaStream_t stream) {
    if (p.layers * p.heads * p.batch == 0) return cudaSuccess;
    switch (p.mp) {
        case 16: return launch_factor_mp<16>(p, k, partials, phi, w, status, stream);
        case 32: return launch_factor_mp<32>(p, k, partials, phi, w, status, stream);
        case 48: return launch_factor_mp<48>(p, k, partials, phi, w, status, stream);
        case 64: return launch_factor_mp<64>(p, k, partials, phi, w, status, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace compactor

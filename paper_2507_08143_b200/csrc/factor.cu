// Small factorisation (Algorithm 1, line 4, by the Cholesky route that Section 3.2 and
// Appendix C allow), in two kernels, all fp64:
//
//   project_kernel   eight CTAs per unit, each owning 16 rows of C = sum of the unit's Gram
//                    partials: T_r = C[rows,:] Phi and the partial projection
//                    G_r = Phi[rows,:]^T T_r, so that G = Phi^T C Phi = sum_r G_r.  This is where
//                    the fp64 FMAs are (1.1 M per unit), spread over the whole device.
//   cholesky_kernel  one small CTA per unit (four fit on an SM, so all units of a large batch are
//                    resident at once): G = sum_r G_r, G = L L^T in one warp (left-looking,
//                    reciprocal square roots), then W = Phi L^-T with one thread per row of Phi
//                    holding the row in registers, split into two bf16 terms.  The score of a key
//                    row k_i is then || k_i W ||^2 (Algorithm 1, lines 5-6).
//
// Rank handling: a pivot not larger than 2^-20 of its original diagonal entry (the fp32 noise
// floor of the 2048-token Gram sums) is treated as a direction of the null space and dropped;
// with the remaining pivot set P, W = Phi[:, P] L_PP^-T, which equals the pseudo-inverse reading
// o_i = k^_i G^+ k^_i^T whenever k^_i lies in the range of G.
#include "common.cuh"

namespace compactor {
namespace {

constexpr double kPivotFloor = 9.5367431640625e-07;   // 2^-20
// Sequences this short are near the sketch dimension, where G is close to singular and the fp32
// rounding inside the Gram partials would dominate the scores; their Gram matrix is summed in
// fp64 straight from the keys instead (the work is tiny).
constexpr int kExactGramTokens = 256;
constexpr int kStageTokens = 8;

constexpr int kSlices = kFactorSlices;     // CTAs per unit in the projection
constexpr int kRows = kD / kSlices;        // rows of C per CTA
constexpr int kProjThreads = 256;

template <int MP>
struct ProjectSmem {
    double phi[kD * MP];           // Phi widened, [channel][column]
    double c[kD * kRows];          // C[k][row0 + i] at [k * kRows + i]  (C is symmetric)
    double t[kRows * MP];          // T_r
    double keys[kStageTokens * kD];
};

template <int MP>
__global__ void __launch_bounds__(kProjThreads)
project_kernel(Plan p, Mat kmat, const double* __restrict__ partials, const float* __restrict__ phi,
               double* __restrict__ g_partials) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ProjectSmem<MP>& s = *reinterpret_cast<ProjectSmem<MP>*>(smem_raw);
    const int unit = blockIdx.x, slice = blockIdx.y;
    const int b = unit % p.batch, lh = unit / p.batch;
    const int m = p.m, tid = threadIdx.x;
    const int row0 = slice * kRows;
    const int chunk_begin = p.cu_chunks[b], n_part = p.cu_chunks[b + 1] - chunk_begin;
    const double* part = partials + ((size_t)lh * p.total_chunks + chunk_begin) * kGramElems;
    const int n_tok = p.cu_seqlens[b + 1] - p.cu_seqlens[b];

    for (int i = tid; i < kD * MP; i += kProjThreads) {
        int row = i / MP, col = i % MP;
        s.phi[i] = (col < m) ? (double)phi[row * m + col] : 0.0;
    }

    // ---- the CTA's 16 columns of C (= 16 rows, by symmetry), summed over the partials ----------
    {
        constexpr int kPer = kD * kRows / kProjThreads;     // 8 elements per thread: e = tid + 256 q
        double acc[kPer];
#pragma unroll
        for (int q = 0; q < kPer; ++q) acc[q] = 0.0;
        if (n_tok > kExactGramTokens) {
            int pp = 0;
            for (; pp + 2 <= n_part; pp += 2) {
                double v[2][kPer];
#pragma unroll
                for (int u = 0; u < 2; ++u)
#pragma unroll
                    for (int q = 0; q < kPer; ++q) {
                        const int e = tid + q * kProjThreads;
                        v[u][q] = __ldcs(part + (size_t)(pp + u) * kGramElems + (e / kRows) * kD + row0 + (e % kRows));
                    }
#pragma unroll
                for (int q = 0; q < kPer; ++q) acc[q] += v[0][q] + v[1][q];
            }
            if (pp < n_part) {
#pragma unroll
                for (int q = 0; q < kPer; ++q) {
                    const int e = tid + q * kProjThreads;
                    acc[q] += __ldcs(part + (size_t)pp * kGramElems + (e / kRows) * kD + row0 + (e % kRows));
                }
            }
        } else {
            const int layer = lh / p.heads, head = lh % p.heads;
            const __nv_bfloat16* kbase = kmat.ptr + layer * kmat.stride_layer + head * kmat.stride_head +
                                         (long long)p.cu_seqlens[b] * kmat.stride_token;
            for (int t0 = 0; t0 < n_tok; t0 += kStageTokens) {
                const int nt = min(kStageTokens, n_tok - t0);
                __syncthreads();
                for (int i = tid; i < nt * kD; i += kProjThreads)
                    s.keys[i] = (double)__bfloat162float(kbase[(long long)(t0 + i / kD) * kmat.stride_token + (i % kD)]);
                __syncthreads();
                for (int t = 0; t < nt; ++t) {
                    const double* krow = s.keys + t * kD;
#pragma unroll
                    for (int q = 0; q < kPer; ++q) {
                        const int e = tid + q * kProjThreads;
                        acc[q] = fma(krow[e / kRows], krow[row0 + (e % kRows)], acc[q]);
                    }
                }
            }
        }
#pragma unroll
        for (int q = 0; q < kPer; ++q) s.c[tid + q * kProjThreads] = acc[q];
    }
    __syncthreads();

    // ---- T_r[i][j] = sum_k C[k][row0+i] Phi[k][j]: thread = (row i, MP/16 columns) ---------------
    {
        constexpr int kCols = MP / 16;
        const int i = tid >> 4, col0 = (tid & 15) * kCols;
        double acc[kCols];
#pragma unroll
        for (int c = 0; c < kCols; ++c) acc[c] = 0.0;
#pragma unroll 4
        for (int k = 0; k < kD; ++k) {
            const double cv = s.c[k * kRows + i];
#pragma unroll
            for (int c = 0; c < kCols; ++c) acc[c] = fma(cv, s.phi[k * MP + col0 + c], acc[c]);
        }
#pragma unroll
        for (int c = 0; c < kCols; ++c) s.t[i * MP + col0 + c] = acc[c];
    }
    __syncthreads();

    // ---- G_r[a][b] = sum_i Phi[row0+i][a] T_r[i][b]: thread = (MP/16 rows a) x (MP/16 columns b) --
    {
        constexpr int kT = MP / 16;
        const int a0 = (tid >> 4) * kT, b0 = (tid & 15) * kT;
        double acc[kT][kT];
#pragma unroll
        for (int x = 0; x < kT; ++x)
#pragma unroll
            for (int y = 0; y < kT; ++y) acc[x][y] = 0.0;
#pragma unroll 4
        for (int i = 0; i < kRows; ++i) {
            double pa[kT], tb[kT];
#pragma unroll
            for (int x = 0; x < kT; ++x) { pa[x] = s.phi[(row0 + i) * MP + a0 + x]; tb[x] = s.t[i * MP + b0 + x]; }
#pragma unroll
            for (int x = 0; x < kT; ++x)
#pragma unroll
                for (int y = 0; y < kT; ++y) acc[x][y] = fma(pa[x], tb[y], acc[x][y]);
        }
        double* out = g_partials + ((size_t)unit * kSlices + slice) * (MP * MP);
#pragma unroll
        for (int x = 0; x < kT; ++x)
#pragma unroll
            for (int y = 0; y < kT; ++y) out[(a0 + x) * MP + b0 + y] = acc[x][y];
    }
}

constexpr int kCholThreads = kD;           // one thread per row of Phi

template <int MP>
struct CholSmem {
    double g[MP * (MP + 1)];     // G, then L in the lower triangle; odd row stride spreads a column over the banks
    double inv_diag[MP];         // 1 / L_jj of kept columns, 0 for dropped or padded ones
    int flags;
};

template <int MP>
__global__ void __launch_bounds__(kCholThreads, 4)
cholesky_kernel(Plan p, const double* __restrict__ g_partials, const float* __restrict__ phi,
                __nv_bfloat16* __restrict__ w_out, int* __restrict__ status) {
    __shared__ CholSmem<MP> s;
    constexpr int LD = MP + 1;
    const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m = p.m;

    if (tid == 0) s.flags = 0;
    if (tid < MP) s.inv_diag[tid] = 0.0;
    __syncthreads();
    {   // G = sum of the partial projections
        const double* src = g_partials + (size_t)unit * kSlices * (MP * MP);
        bool finite = true;
        for (int e = tid; e < MP * MP; e += kCholThreads) {
            double v = 0.0;
#pragma unroll
            for (int r = 0; r < kSlices; ++r) v += src[(size_t)r * (MP * MP) + e];
            s.g[(e / MP) * LD + (e % MP)] = v;
            finite = finite && isfinite(v);
        }
        if (!finite) atomicOr(&s.flags, COMPACTOR_STATUS_NONFINITE);
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
                    a0 = s.g[i * LD + j];
                    int c = 0;
                    for (; c + 2 <= j; c += 2) {
                        a0 = fma(-s.g[i * LD + c], s.g[j * LD + c], a0);
                        a1 = fma(-s.g[i * LD + c + 1], s.g[j * LD + c + 1], a1);
                    }
                    if (c < j) a0 = fma(-s.g[i * LD + c], s.g[j * LD + c], a0);
                }
                v[h] = a0 + a1;
            }
            const double piv = __shfl_sync(0xffffffffu, v[0], 0);
            const double d0 = s.g[j * LD + j];              // still the original diagonal entry
            const bool keep = piv > kPivotFloor * d0 && d0 > 0.0;
            const double inv = keep ? rsqrt(piv) : 0.0;
            if (!keep) rank_flag = 1;
            __syncwarp();
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int i = j + lane + 32 * h;
                if (i < m) s.g[i * LD + j] = (i == j) ? piv * inv : v[h] * inv;
            }
            if (lane == 0) s.inv_diag[j] = inv;
            __syncwarp();
        }
        if (lane == 0 && rank_flag) s.flags |= COMPACTOR_STATUS_RANK;
    }
    __syncthreads();

    // ---- W = Phi L^-T: forward substitution along the row, which is held in registers ------------
    {
        const int row = tid;
        double r[MP];
#pragma unroll
        for (int c = 0; c < MP; ++c) r[c] = (c < m && !bad) ? (double)phi[row * m + c] : 0.0;
#pragma unroll
        for (int j = 0; j < MP; ++j) {
            const double wj = r[j] * s.inv_diag[j];
            r[j] = wj;
#pragma unroll
            for (int c = j + 1; c < MP; ++c) r[c] = fma(-wj, s.g[c * LD + j], r[c]);
        }
        __nv_bfloat16* w_hi = w_out + (size_t)unit * w_elems_per_unit(MP);
        __nv_bfloat16* w_lo = w_hi + (size_t)MP * kD;
#pragma unroll
        for (int j = 0; j < MP; ++j) {
            const __nv_bfloat16 hi = __double2bfloat16(r[j]);
            w_hi[j * kD + row] = hi;
            w_lo[j * kD + row] = __double2bfloat16(r[j] - (double)__bfloat162float(hi));
        }
    }
    if (tid == 0 && status != nullptr && s.flags != 0) atomicOr(&status[unit], s.flags);
}

template <int MP>
cudaError_t launch_factor_mp(const Plan& p, const Mat& k, const double* partials, const float* phi,
                             double* g_partials, __nv_bfloat16* w, int* status, cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    const int smem = (int)sizeof(ProjectSmem<MP>);
    cudaError_t e = cudaFuncSetAttribute(project_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    project_kernel<MP><<<dim3(units, kSlices), kProjThreads, smem, stream>>>(p, k, partials, phi, g_partials);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    cholesky_kernel<MP><<<units, kCholThreads, 0, stream>>>(p, g_partials, phi, w, status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_factor(const Plan& p, const Mat& k, const double* partials, const float* phi, double* g_partials,
                          __nv_bfloat16* w, int* status, cudaStream_t stream) {
    if (p.layers * p.heads * p.batch == 0) return cudaSuccess;
    switch (p.mp) {
        case 16: return launch_factor_mp<16>(p, k, partials, phi, g_partials, w, status, stream);
        case 32: return launch_factor_mp<32>(p, k, partials, phi, g_partials, w, status, stream);
        case 48: return launch_factor_mp<48>(p, k, partials, phi, g_partials, w, status, stream);
        case 64: return launch_factor_mp<64>(p, k, partials, phi, g_partials, w, status, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace compactor

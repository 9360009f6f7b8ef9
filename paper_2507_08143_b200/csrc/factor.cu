// Small factorisation (Algorithm 1, line 4, by the Cholesky route that Section 3.2 and
// Appendix C allow), in two kernels, all fp64:
//
//   project_kernel   two work items per unit.  C = sum of the unit's Gram partials is symmetric, so
//                    G = Phi^T C Phi = A + A^T with A = Phi^T M Phi, M the half of C below the
//                    diagonal (plus half the diagonal).  An item takes two of the four 32-row
//                    slices of M, forms their rows of M Phi and then their share of A on fp64
//                    mma.m8n8k4 (this is where the fp64 work is: 0.8 M multiply-adds per unit,
//                    spread over the whole device) and writes an m x m part of A.
//   cholesky_kernel  one small CTA per unit, several per SM: G = sum of the parts and their
//                    transposes, G = L L^T by panels of eight columns (the 8 x 8 diagonal blocks
//                    are factored redundantly by every lane of a warp, so no pivot has to travel),
//                    then W = Phi L^-T as a blocked substitution on fp64 mma, split into two bf16
//                    terms.  The score of a key row k_i is then || k_i W ||^2 (Algorithm 1, lines
//                    5-6), which the scoring sweep computes.  A unit about as short as the sketch
//                    is wide (n <= m + 16) has a G too close to singular for that: it is factored
//                    with diagonal pivoting and its scores are written here, in fp64.
//
// Rank handling: a pivot not larger than 2^-20 of its original diagonal entry (the fp32 noise
// floor of the fp32 Gram runs) is treated as a direction of the null space and dropped;
// with the remaining pivot set P, W = Phi[:, P] L_PP^-T, which equals the pseudo-inverse reading
// o_i = k^_i G^+ k^_i^T whenever k^_i lies in the range of G.
#include "common.cuh"
#include "factor_math.cuh"

namespace compactor {
namespace {

using namespace factor_math;

// Sequences this short are near the sketch dimension, where G is close to singular and the fp32
// rounding inside the Gram partials would dominate the scores; their Gram matrix is summed in
// fp64 straight from the keys instead (the work is tiny).
constexpr int kExactGramTokens = 256;
constexpr int kStageTokens = 16;

// The sketch [128][m] from global memory into shared memory as [128][MP] with row stride LD (columns from m on are
// zero), eight loads per thread in flight at a time (a plain copy loop waits for every load in turn).
template <int MP, int LD, int NTHREADS, class T>
__device__ __forceinline__ void load_sketch(T* dst, const float* __restrict__ phi, int m, int tid) {
    constexpr int kBatch = 8;
    static_assert(kD * MP % (kBatch * NTHREADS) == 0, "whole batches");
    for (int i0 = tid; i0 < kD * MP; i0 += kBatch * NTHREADS) {
        float v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int i = i0 + u * NTHREADS, row = i / MP, col = i - row * MP;
            v[u] = __ldg(phi + row * m + min(col, m - 1));          // unconditional, masked below
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int i = i0 + u * NTHREADS, row = i / MP, col = i - row * MP;
            dst[row * LD + col] = col < m ? (T)v[u] : (T)0;
        }
    }
}

constexpr int kSlices = kFactorSlices;     // 32-row slices of C per unit
constexpr int kRows = kD / kSlices;        // rows of C per slice
constexpr int kPairs = kFactorParts;       // work items per unit: slices s and kSlices-1-s together cost the same for every s
constexpr int kProjThreads = 256;
static_assert(kSlices == 2 * kPairs, "slices are paired");

template <int MP>
struct ProjectSmem {
    static constexpr int kLd = MP + 4;     // row stride (doubles): the four k-rows of a B fragment land in distinct banks
    double phi[kD * kLd];                  // Phi widened, [channel][column]
    static constexpr int kLdc = kRows + 4; // stride of a k-row of c: the four k-rows of an A fragment land in distinct banks
    double c[kD * kLdc];                   // the slice of the triangular half of C, [k][row0 + i] at [k * kLdc + i]
    union {
        double keys[kStageTokens * kD];    // short sequences: staged key rows
        double t[kRows * kLd];             // the slice's rows of the half product, until they are multiplied by Phi^T
    } u;
};

// C is symmetric, so G = Phi^T C Phi = A + A^T with A = Phi^T M Phi, where M is the part of C below the diagonal plus half of
// the diagonal.  Only that half is read (the Gram pass writes only the blocks it needs) and multiplied:
// a slice of 32 rows of M has non-zeros in its first 32 (s + 1) columns only.  Each item takes two slices of a unit
// (s and 3 - s: five blocks of 32 x 32 whatever s is), forms their rows of M Phi, multiplies them by the matching rows of
// Phi^T and writes the sum, an MP x MP part of A; the factor kernel adds the parts of a unit and their transposes.
// Persistent: each CTA loads Phi once and then walks the items with a grid stride.
template <int MP>
__global__ void __launch_bounds__(kProjThreads, 2)
project_kernel(Plan p, Mat kmat, const double* __restrict__ partials, const float* __restrict__ phi,
               double* __restrict__ a_parts, int n_items) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using Smem = ProjectSmem<MP>;
    Smem& s = *reinterpret_cast<Smem*>(smem_raw);
    constexpr int LD = Smem::kLd;
    constexpr int LDC = Smem::kLdc;
    constexpr int kWarps = kProjThreads / 32;
    const int m = p.m, tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int fr = lane >> 2, fk = lane & 3;            // fragment coordinates: A[fr][fk], B[fk][fr], C[fr][2 fk, 2 fk + 1]
    constexpr int kNT = MP / 8;                         // 8-column tiles
    constexpr int kATiles = kNT * kNT;                  // 8 x 8 tiles of a part of A
    constexpr int kAGroup = 8;                          // tiles of A a warp holds in registers at a time
    constexpr int kAPer = (kATiles + kWarps - 1) / kWarps;
    constexpr bool kKeepA = kAPer <= kAGroup;           // a part of A stays in registers over both slices (else: added up in global memory)
    constexpr int kAHeld = kKeepA ? kAPer : kAGroup;

    pdl_trigger();
    load_sketch<MP, LD, kProjThreads>(s.phi, phi, m, tid);   // Phi, widened
    pdl_wait();                                           // the Gram partials are complete

    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int unit = item / kPairs, pair = item % kPairs;
        const int b = unit % p.batch, lh = unit / p.batch;
        const int chunk_begin = p.cu_chunks[b];
        const int n_part = p.cu_chunks[b + 1] - chunk_begin;
        const int n_tok = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
        const double* part = partials + ((size_t)lh * p.total_chunks + chunk_begin) * kGramElems;
        double* a_out = a_parts + (size_t)unit * a_elems_per_unit(MP) + (size_t)pair * MP * MP;
        double a[kAHeld][2];
#pragma unroll
        for (int si = 0; si < kAHeld; ++si) a[si][0] = a[si][1] = 0.0;

        // One slice: kS is its number as a type, so that every loop below has constant bounds.
        auto do_slice = [&](auto slice_tag, bool second) {
            constexpr int kS = decltype(slice_tag)::value;
            constexpr int kmax = kRows * (kS + 1);                   // columns of M that this slice can have non-zeros in
            constexpr int kPer = kmax * kRows / kProjThreads;        // elements of the slice per thread: e = tid + 256 q
            constexpr int kInFlight = kPer <= 4 ? 4 : (kPer <= 8 ? 2 : 1);   // partials loaded together
            const int row0 = kS * kRows;
            // element (k, i) of the slice is M[row0 + i][k] = C[k][row0 + i] below the diagonal, half of it on the diagonal
            auto masked = [&](int k, int i, double v) {
                const int kk = k - row0;
                return kk < i ? v : (kk == i ? 0.5 * v : 0.0);
            };
            if (n_tok > kExactGramTokens) {
                double acc[kPer];
#pragma unroll
                for (int q = 0; q < kPer; ++q) acc[q] = 0.0;
                for (int pp = 0; pp < n_part; pp += kInFlight) {
                    double v[kInFlight][kPer];
#pragma unroll
                    for (int u = 0; u < kInFlight; ++u) {
                        // unconditional loads (a partial past the last one re-reads the last and is not added): loads under
                        // a per-load condition are issued one after the other instead of together
                        const int uu = pp + u < n_part ? pp + u : n_part - 1;
#pragma unroll
                        for (int q = 0; q < kPer; ++q) {
                            const int e = tid + q * kProjThreads;
                            v[u][q] = __ldcs(part + (size_t)uu * kGramElems + (e / kRows) * kD + row0 + (e % kRows));
                        }
                    }
#pragma unroll
                    for (int u = 0; u < kInFlight; ++u)
                        if (pp + u < n_part) {
#pragma unroll
                            for (int q = 0; q < kPer; ++q) acc[q] += v[u][q];
                        }
                }
                __syncthreads();                              // the previous slice's products are done with c
#pragma unroll
                for (int q = 0; q < kPer; ++q) {
                    const int e = tid + q * kProjThreads;
                    s.c[(e / kRows) * LDC + (e % kRows)] = masked(e / kRows, e % kRows, acc[q]);
                }
            } else {
                // short sequence: fp64 Gram straight from the keys, C[:, rows] = K^T K[:, rows], as fp64 mma.m8n8k4
                // over four tokens at a time (only the 8-row tiles that the slice needs)
                const int layer = lh / p.heads, head = lh % p.heads;
                const __nv_bfloat16* kbase = kmat.ptr + layer * kmat.stride_layer + head * kmat.stride_head +
                                             (long long)p.cu_seqlens[b] * kmat.stride_token;
                constexpr int kTilesPerWarp = (kD / 8) * (kRows / 8) / kWarps;
                double d[kTilesPerWarp][2];
#pragma unroll
                for (int j = 0; j < kTilesPerWarp; ++j) d[j][0] = d[j][1] = 0.0;
                // the keys of the next stage are on their way while the current stage is multiplied
                constexpr int kLoads = kStageTokens * kD / kProjThreads;
                float nxt[kLoads];
                auto fetch = [&](int t0) {                    // missing tokens of the last stage are zeros
#pragma unroll
                    for (int u = 0; u < kLoads; ++u) {
                        const int i = tid + u * kProjThreads, t = min(t0 + i / kD, n_tok - 1);
                        nxt[u] = __bfloat162float(kbase[(long long)t * kmat.stride_token + (i % kD)]);
                        if (t0 + i / kD >= n_tok) nxt[u] = 0.f;
                    }
                };
                if (n_tok > 0) fetch(0);
                for (int t0 = 0; t0 < n_tok; t0 += kStageTokens) {
                    __syncthreads();                          // the previous stage, and the previous slice's products, are done
#pragma unroll
                    for (int u = 0; u < kLoads; ++u) s.u.keys[tid + u * kProjThreads] = (double)nxt[u];
                    __syncthreads();
                    if (t0 + kStageTokens < n_tok) fetch(t0 + kStageTokens);
#pragma unroll
                    for (int ks = 0; ks < kStageTokens / 4; ++ks) {
                        const double* krow = s.u.keys + (ks * 4 + fk) * kD;        // token ks*4 + fk of the stage
#pragma unroll
                        for (int j = 0; j < kTilesPerWarp; ++j) {
                            const int tile = warp + j * kWarps;
                            const int mt = tile / (kRows / 8), nt8 = tile % (kRows / 8);
                            if (mt * 8 < kmax)
                                mma_f64(d[j], krow[mt * 8 + fr], krow[row0 + nt8 * 8 + fr]);   // A[channel][token], B[token][channel of the slice]
                        }
                    }
                }
                __syncthreads();                              // the previous slice's products are done with c
#pragma unroll
                for (int j = 0; j < kTilesPerWarp; ++j) {
                    const int tile = warp + j * kWarps;
                    const int mt = tile / (kRows / 8), nt8 = tile % (kRows / 8);
                    if (mt * 8 < kmax) {
                        s.c[(mt * 8 + fr) * LDC + nt8 * 8 + 2 * fk] = masked(mt * 8 + fr, nt8 * 8 + 2 * fk, d[j][0]);
                        s.c[(mt * 8 + fr) * LDC + nt8 * 8 + 2 * fk + 1] = masked(mt * 8 + fr, nt8 * 8 + 2 * fk + 1, d[j][1]);
                    }
                }
            }
            __syncthreads();

            // ---- (M Phi)[rows] (32 x MP) = M[rows, :kmax] Phi[:kmax] : a warp-wide fp64 mma does 256 multiply-adds for two
            // 8-byte shared-memory loads per lane; the contraction is cut into four independent chains --------------------
            for (int tile = warp; tile < (kRows / 8) * kNT; tile += kWarps) {
                const int mt = tile / kNT, nt = tile % kNT;
                double d[4][2];
#pragma unroll
                for (int g = 0; g < 4; ++g) d[g][0] = d[g][1] = 0.0;
#pragma unroll
                for (int k0 = 0; k0 < kmax / 4; k0 += 4) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const int k = g * (kmax / 4) + k0 + fk;
                        mma_f64(d[g], s.c[k * LDC + mt * 8 + fr], s.phi[k * LD + nt * 8 + fr]);   // A[row][k] = M[row0 + row][k], B[k][col]
                    }
                }
                *reinterpret_cast<double2*>(&s.u.t[(mt * 8 + fr) * LD + nt * 8 + 2 * fk]) =
                    make_double2((d[0][0] + d[1][0]) + (d[2][0] + d[3][0]), (d[0][1] + d[1][1]) + (d[2][1] + d[3][1]));
            }
            __syncthreads();

            // ---- the slice's share of the part of A: Phi[rows]^T (MP x 32) times those rows (32 x MP) ---------------------
            if constexpr (kKeepA) {
#pragma unroll
                for (int si = 0; si < kAPer; ++si) {
                    const int tile = warp + si * kWarps;
                    if (tile < kATiles) {
                        const int mt = tile / kNT, nt = tile % kNT;
#pragma unroll
                        for (int k0 = 0; k0 < kRows; k0 += 4)
                            mma_f64(a[si], s.phi[(row0 + k0 + fk) * LD + mt * 8 + fr], s.u.t[(k0 + fk) * LD + nt * 8 + fr]);
                    }
                }
            } else {
                for (int g0 = 0; g0 < kAPer; g0 += kAGroup) {
#pragma unroll
                    for (int si = 0; si < kAGroup; ++si) {
                        const int tile = warp + (g0 + si) * kWarps;
                        if (tile >= kATiles) continue;
                        const int mt = tile / kNT, nt = tile % kNT;
                        double* out = a_out + (size_t)(mt * 8 + fr) * MP + nt * 8 + 2 * fk;
                        double2 sum = make_double2(0.0, 0.0);
                        if (second) sum = __ldcg(reinterpret_cast<const double2*>(out));     // what this thread wrote for the first slice
                        a[si][0] = sum.x; a[si][1] = sum.y;
#pragma unroll
                        for (int k0 = 0; k0 < kRows; k0 += 4)
                            mma_f64(a[si], s.phi[(row0 + k0 + fk) * LD + mt * 8 + fr], s.u.t[(k0 + fk) * LD + nt * 8 + fr]);
                        __stcg(reinterpret_cast<double2*>(out), make_double2(a[si][0], a[si][1]));
                    }
                }
            }
        };
        if (pair == 0) {
            do_slice(std::integral_constant<int, 0>{}, false);
            do_slice(std::integral_constant<int, kSlices - 1>{}, true);
        } else {
            do_slice(std::integral_constant<int, 1>{}, false);
            do_slice(std::integral_constant<int, kSlices - 2>{}, true);
        }
        if constexpr (kKeepA) {
#pragma unroll
            for (int si = 0; si < kAPer; ++si) {
                const int tile = warp + si * kWarps;
                if (tile < kATiles) {
                    const int mt = tile / kNT, nt = tile % kNT;
                    __stcg(reinterpret_cast<double2*>(a_out + (size_t)(mt * 8 + fr) * MP + nt * 8 + 2 * fk), make_double2(a[si][0], a[si][1]));
                }
            }
        }
    }
}

// G = sum over the unit's parts of (A + A^T), the 8 x 8 tiles on and below the diagonal, by columns
// (g[c * MP + i] = G[i][c]); the loads of four elements per thread are in flight together.  Returns false in a
// thread that met an entry that is not finite.
template <int MP, int NTHREADS>
__device__ __forceinline__ bool gram_from_parts(const double* __restrict__ a_unit, double* g, int tid) {
    constexpr int kNT = MP / 8, kElems = kNT * (kNT + 1) / 2 * 64, kBatch = 4;
    bool finite = true;
    for (int e0 = tid; e0 < kElems; e0 += kBatch * NTHREADS) {
        double v[kBatch][2 * kPairs];
        int at[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int e = min(e0 + u * NTHREADS, kElems - 1);       // unconditional loads; the surplus is not stored
            int rem = e >> 6, mt = 0;
            while (rem > mt) { rem -= mt + 1; ++mt; }                // tile number -> (mt, nt = rem), mt >= nt
            const int i = mt * 8 + (e & 7), c = rem * 8 + ((e >> 3) & 7);
            at[u] = c * MP + i;
#pragma unroll
            for (int part = 0; part < kPairs; ++part) {
                v[u][2 * part] = __ldcg(a_unit + (size_t)part * MP * MP + i * MP + c);
                v[u][2 * part + 1] = __ldcg(a_unit + (size_t)part * MP * MP + c * MP + i);
            }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            double sum = 0.0;
#pragma unroll
            for (int j = 0; j < 2 * kPairs; ++j) sum += v[u][j];
            if (e0 + u * NTHREADS < kElems) {
                g[at[u]] = sum;
                finite = finite && isfinite(sum);
            }
        }
    }
    return finite;
}

constexpr int kCholThreads = 128;
constexpr int kCholWarps = kCholThreads / 32;

template <int MP>
struct CholSmem {
    float phi[kD * MP];                    // the sketch, zero in the padded columns
    double g[MP * MP];                     // G, then L by columns (and the inverses of its diagonal blocks)
    double diag0[MP], inv_diag[MP];
    int perm[2 * MP];                      // pivot order and "already a pivot" marks of the pivoted factorisation
    int flags;
};

// Sequences about as short as the sketch is wide: G = (K Phi)^T (K Phi) has rank n or is nearly singular, and a
// Cholesky factorisation in the given column order meets pivots that are small differences of large numbers.  Here
// the factorisation takes the largest remaining diagonal entry as its next pivot (which is stable for positive
// semi-definite matrices and reveals the rank: it stops at `rank_bound` pivots or when what remains is below 2^-40 of
// the largest original entry), one CTA per unit, a step at a time: the work is tiny and such units are rare.
// `a` holds G by columns (lower triangle valid on entry, the whole square is used); W = Phi[:, P] L^-T comes out in
// pivot order (the order of its columns does not matter to the scores), zero beyond the rank.  Returns the rank.
// With `scores_unit` the unit's scores are written too, in fp64 arithmetic: o_i = || y_i ||^2, y_i the same
// substitution applied to k^_i = Phi^T k_i (W in two bf16 terms resolves 2^-17 of its largest entries, and
// with a G this close to singular the products k_i W cancel far below that).  `keys`: the unit's first key row.
template <int MP>
__device__ int pivoted_factor_and_solve(double* a, const float* phi, int m, int rank_bound, int tid, int* perm, double* red,
                                        __nv_bfloat16* w_hi, const __nv_bfloat16* keys, long long stride_token, int n_tok,
                                        float* scores_unit) {
    constexpr int LD = MP;
    const int lane = tid & 31, warp = tid >> 5;
    for (int idx = tid; idx < m * m; idx += kCholThreads) {            // both triangles
        const int i = idx % m, c = idx / m;
        if (i < c) a[c * LD + i] = a[i * LD + c];
    }
    __syncthreads();
    // block-wide maximum of the remaining diagonal with its index (ties: lower index); perm[MP + i] = 1 once i is a pivot
    auto arg_max = [&](double& best, int& where) {
        double v = -1.0; int at = 0x7fffffff;
        for (int i = tid; i < m; i += kCholThreads)
            if (perm[MP + i] == 0) { const double d = a[i * LD + i]; if (d > v || (d == v && i < at)) { v = d; at = i; } }
#pragma unroll
        for (int dlt = 16; dlt > 0; dlt >>= 1) {
            const double ov = __shfl_xor_sync(0xffffffffu, v, dlt);
            const int oa = __shfl_xor_sync(0xffffffffu, at, dlt);
            if (ov > v || (ov == v && oa < at)) { v = ov; at = oa; }
        }
        __syncthreads();                                                 // earlier readers of red are done
        if (lane == 0) { red[warp] = v; red[kCholWarps + warp] = (double)at; }
        __syncthreads();
        best = red[0]; where = (int)red[kCholWarps];
        for (int w = 1; w < kCholWarps; ++w)
            if (red[w] > best || (red[w] == best && (int)red[kCholWarps + w] < where)) { best = red[w]; where = (int)red[kCholWarps + w]; }
    };
    for (int i = tid; i < m; i += kCholThreads) perm[MP + i] = 0;
    __syncthreads();
    double d_first; int at;
    arg_max(d_first, at);
    const double floor_abs = d_first * 9.094947017729282e-13;           // 2^-40 of the largest diagonal entry
    int rank = 0;
    const int max_rank = min(m, rank_bound);
    while (rank < max_rank) {
        double piv; int pj;
        arg_max(piv, pj);
        if (!(piv > floor_abs) || !(piv > 0.0)) break;
        const double ljj = sqrt(piv), inv = 1.0 / ljj;
        __syncthreads();
        for (int i = tid; i < m; i += kCholThreads)                     // column pj becomes column `rank` of L (by original row)
            if (perm[MP + i] == 0) a[pj * LD + i] = (i == pj) ? ljj : a[pj * LD + i] * inv;
        __syncthreads();
        if (tid == 0) { perm[rank] = pj; perm[MP + pj] = 1; }
        __syncthreads();
        for (int idx = tid; idx < m * m; idx += kCholThreads) {        // what remains: A_ik -= L_i L_k
            const int i = idx % m, k = idx / m;
            if (perm[MP + i] == 0 && perm[MP + k] == 0) a[k * LD + i] = fma(-a[pj * LD + i], a[pj * LD + k], a[k * LD + i]);
        }
        __syncthreads();
        ++rank;
    }
    // forward substitution, one row of Phi per thread: w_j = (phi[perm j] - sum_{t<j} w_t L[perm j][t]) / L[perm j][j]
    __nv_bfloat16* w_lo = w_hi + (size_t)MP * kD;
    for (int row = tid; row < kD; row += kCholThreads) {
        double w[MP];
        for (int j = 0; j < rank; ++j) {
            const int pj = perm[j];
            double acc = (double)phi[row * MP + pj];
            for (int t = 0; t < j; ++t) acc = fma(-w[t], a[perm[t] * LD + pj], acc);
            w[j] = acc / a[pj * LD + pj];
        }
        for (int j = 0; j < MP; ++j) {
            const double v = j < rank ? w[j] : 0.0;
            const __nv_bfloat16 hi = __double2bfloat16(v);
            w_hi[j * kD + row] = hi;
            w_lo[j * kD + row] = __double2bfloat16(v - (double)__bfloat162float(hi));
        }
    }
    if (scores_unit != nullptr) {
        for (int tok = tid; tok < n_tok; tok += kCholThreads) {
            double kh[MP], y[MP];
            for (int j = 0; j < m; ++j) kh[j] = 0.0;
            const __nv_bfloat16* krow = keys + (long long)tok * stride_token;
            for (int c = 0; c < kD; ++c) {
                const double kv = (double)__bfloat162float(krow[c]);
                for (int j = 0; j < m; ++j) kh[j] = fma(kv, (double)phi[c * MP + j], kh[j]);
            }
            double o = 0.0;
            for (int j = 0; j < rank; ++j) {
                const int pj = perm[j];
                double acc = kh[pj];
                for (int t = 0; t < j; ++t) acc = fma(-y[t], a[perm[t] * LD + pj], acc);
                y[j] = acc / a[pj * LD + pj];
                o = fma(y[j], y[j], o);
            }
            scores_unit[tok] = (float)o;
        }
    }
    return rank;
}

template <int MP>
__global__ void __launch_bounds__(kCholThreads, MP <= 48 ? 4 : (MP <= 64 ? 2 : 1))
cholesky_kernel(Plan p, Mat kmat, const double* __restrict__ a_parts, const float* __restrict__ phi,
                __nv_bfloat16* __restrict__ w_out, float* __restrict__ scores, int* __restrict__ status) {
    extern __shared__ __align__(16) unsigned char chol_smem_raw[];
    CholSmem<MP>& s = *reinterpret_cast<CholSmem<MP>*>(chol_smem_raw);
    const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m = p.m;

    pdl_trigger();
    if (tid == 0) s.flags = 0;
    load_sketch<MP, MP, kCholThreads>(s.phi, phi, m, tid);
    if (tid < MP) s.inv_diag[tid] = 0.0;
    pdl_wait();                                           // the parts of A of every unit are complete
    __syncthreads();
    auto sync = [] { __syncthreads(); };
    const bool finite = gram_from_parts<MP, kCholThreads>(a_parts + (size_t)unit * a_elems_per_unit(MP), s.g, tid);
    if (!finite) atomicOr(&s.flags, COMPACTOR_STATUS_NONFINITE);
    __syncthreads();
    const bool bad = (s.flags & COMPACTOR_STATUS_NONFINITE) != 0;
    // The pivot floor (2^-20 of the original diagonal) is the noise floor of the fp32 Gram sums.  A short sequence's
    // Gram matrix was summed in fp64 from the keys and has no such noise, while its pivots are legitimately small
    // (few rows, nearly dependent columns): there the floor is 2^-40 (the reference diagonal is scaled down instead).
    // What that floor lets through once the rank is used up is rounding amplified by the conditioning of the leading
    // block; a sequence of n < m tokens has rank n at most, so no more than n pivots are kept.
    const int n_unit = p.cu_seqlens[unit % p.batch + 1] - p.cu_seqlens[unit % p.batch];
    const bool exact_gram = n_unit <= kExactGramTokens;
    __nv_bfloat16* w_unit = w_out + (size_t)unit * w_elems_per_unit(MP);
    // about as many tokens as sketch columns: G is singular or nearly so; only a pivoted factorisation is accurate, and the
    // scores are worked out here as well (the scoring sweep leaves such units alone)
    const bool tiny = n_unit <= m + kTinyExtra;
    const int b_unit = unit % p.batch, lh_unit = unit / p.batch;
    float* scores_unit = scores == nullptr ? nullptr : scores + (size_t)lh_unit * p.total_tokens + p.cu_seqlens[b_unit];
    if (!bad && tiny) {
        const int layer = lh_unit / p.heads, head = lh_unit % p.heads;
        const __nv_bfloat16* keys = kmat.ptr + layer * kmat.stride_layer + head * kmat.stride_head +
                                    (long long)p.cu_seqlens[b_unit] * kmat.stride_token;
        const int rank = pivoted_factor_and_solve<MP>(s.g, s.phi, m, n_unit, tid, s.perm, s.diag0, w_unit, keys,
                                                      kmat.stride_token, n_unit, scores_unit);
        if (tid == 0 && status != nullptr && rank < m) atomicOr(&status[unit], COMPACTOR_STATUS_RANK);
        return;
    }
    if (bad && tiny && scores_unit != nullptr)              // non-finite keys: W = 0 below, and so are the scores
        for (int tok = tid; tok < n_unit; tok += kCholThreads) scores_unit[tok] = 0.f;
    if (tid < MP) s.diag0[tid] = s.g[tid * MP + tid] * (exact_gram ? 9.5367431640625e-07 : 1.0);
    __syncthreads();
    if (!bad) cholesky_panels<MP, kCholWarps>(s.g, s.diag0, s.inv_diag, m, tid, &s.flags, sync, exact_gram ? n_unit : (1 << 30));
    __syncthreads();
    if (!bad) {
        for (int rb = warp * 16; rb < kD; rb += kCholWarps * 16) solve_w_tiles<MP>(s.phi, s.g, s.inv_diag, rb, lane, w_unit);
    } else {                                              // a unit with non-finite keys gets W = 0
        for (int e = tid; e < (int)w_elems_per_unit(MP); e += kCholThreads) w_unit[e] = __float2bfloat16(0.f);
    }
    if (tid == 0 && status != nullptr && s.flags != 0) atomicOr(&status[unit], s.flags);
}

// ---------------------------------------------------------------------------------------------
// Appendix C, eigendecomposition route: G = V Lambda V^T by cyclic two-sided Jacobi rotations in
// fp64 (all disjoint index pairs of a round-robin step are rotated at once), every eigenvalue
// raised to at least `floor`, W = Phi V Lambda^-1/2 split into two bf16 terms.  One CTA per unit.
constexpr int kEigThreads = kD;
constexpr int kEigMaxSweeps = 16;

template <int MP>
struct EigSmem {
    static constexpr int kLd = MP + 1;
    double a[MP * kLd];          // G, driven to diagonal form
    double v[MP * kLd];          // accumulated rotations: columns are the eigenvectors (first: G by columns, as it is formed)
    float phi[kD * MP];
    double rot_c[MP / 2], rot_s[MP / 2];
    int rot_p[MP / 2], rot_q[MP / 2];
    double inv_sqrt[MP];
    double red[kEigThreads / 32][2];
    int flags;
};

template <int MP>
__global__ void __launch_bounds__(kEigThreads, 3)
eig_kernel(Plan p, const double* __restrict__ a_parts, const float* __restrict__ phi, double floor,
           __nv_bfloat16* __restrict__ w_out, int* __restrict__ status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using Smem = EigSmem<MP>;
    Smem& s = *reinterpret_cast<Smem*>(smem_raw);
    constexpr int LD = Smem::kLd;
    const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m = p.m;
    const int n = (m + 1) & ~1;                 // an even number of indices to pair; the padding row is zero
    const int half = n >> 1;

    if (tid == 0) s.flags = 0;
    __syncthreads();
    {
        // G from its parts into `v` (by columns, lower triangle), then mirrored into `a`
        load_sketch<MP, MP, kEigThreads>(s.phi, phi, m, tid);
        __syncthreads();
        const bool finite = gram_from_parts<MP, kEigThreads>(a_parts + (size_t)unit * a_elems_per_unit(MP), s.v, tid);
        if (!finite) atomicOr(&s.flags, COMPACTOR_STATUS_NONFINITE);
        __syncthreads();
        for (int e = tid; e < MP * MP; e += kEigThreads) {
            const int i = e / MP, j = e % MP;
            s.a[i * LD + j] = i >= j ? s.v[j * MP + i] : s.v[i * MP + j];
        }
        __syncthreads();
        for (int e = tid; e < MP * MP; e += kEigThreads) {
            const int i = e / MP, j = e % MP;
            s.v[i * LD + j] = (i == j) ? 1.0 : 0.0;
        }
    }
    __syncthreads();
    const bool bad = (s.flags & COMPACTOR_STATUS_NONFINITE) != 0;

    // G is scaled by a power of two (exactly) so that its largest diagonal entry lies in [1/2, 1): the rotation
    // angles can then be worked out in fp32 without overflow; the eigenvalues are scaled back at the end.
    int scale_exp = 0;
    if (!bad) {
        double dmax = 0.0;
        for (int i = 0; i < m; ++i) dmax = fmax(dmax, fabs(s.a[i * LD + i]));      // the same in every thread
        if (dmax > 0.0) (void)frexp(dmax, &scale_exp);
        __syncthreads();
        for (int e = tid; e < MP * MP; e += kEigThreads) {
            const int i = e / MP, j = e % MP;
            s.a[i * LD + j] = ldexp(s.a[i * LD + j], -scale_exp);
        }
        __syncthreads();
    }

    for (int sweep = 0; sweep < kEigMaxSweeps && !bad; ++sweep) {
        // off-diagonal mass against the whole: the same value in every thread, so all leave together
        double off = 0.0, all = 0.0;
        for (int e = tid; e < n * n; e += kEigThreads) {
            const int i = e / n, j = e % n;
            const double x = s.a[i * LD + j];
            all = fma(x, x, all);
            if (i != j) off = fma(x, x, off);
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            off += __shfl_xor_sync(0xffffffffu, off, d);
            all += __shfl_xor_sync(0xffffffffu, all, d);
        }
        if (lane == 0) { s.red[warp][0] = off; s.red[warp][1] = all; }
        __syncthreads();
        off = 0.0; all = 0.0;
#pragma unroll
        for (int w = 0; w < kEigThreads / 32; ++w) { off += s.red[w][0]; all += s.red[w][1]; }
        __syncthreads();
        if (!(off > 1e-26 * all)) break;

        for (int step = 0; step < n - 1; ++step) {
            if (tid < half) {
                // round-robin pairing: index n-1 stays, the others move round a ring of n-1 seats
                int a0, a1;
                if (tid == 0) { a0 = n - 1; a1 = step % (n - 1); }
                else { a0 = (step + tid) % (n - 1); a1 = (step - tid + (n - 1)) % (n - 1); }
                const int pp = min(a0, a1), qq = max(a0, a1);
                const double apq = s.a[pp * LD + qq], app = s.a[pp * LD + pp], aqq = s.a[qq * LD + qq];
                double c = 1.0, sn = 0.0;
                if (fabs(apq) > 1e-300) {
                    // tan of the rotation angle to fp32 accuracy (a rotation by a slightly different angle still
                    // is an exact similarity; it leaves 1e-7 of the pivot instead of nothing), then cos and
                    // sin to fp64 accuracy from it, so that the rotation stays orthogonal: the cosine by two
                    // Newton steps on a single-precision reciprocal square root
                    const float theta = (float)(aqq - app) / (2.0f * (float)apq);    // inf when apq underflows: t = 0
                    const float tf = copysignf(1.0f, theta) / (fabsf(theta) + sqrtf(fmaf(theta, theta, 1.0f)));
                    const double t = (double)tf;
                    const double x = fma(t, t, 1.0);                                 // in [1, 2]
                    double r = (double)rsqrtf((float)x);
                    r = r * fma(-0.5 * x, r * r, 1.5);
                    r = r * fma(-0.5 * x, r * r, 1.5);
                    c = r;
                    sn = t * r;
                }
                s.rot_c[tid] = c; s.rot_s[tid] = sn; s.rot_p[tid] = pp; s.rot_q[tid] = qq;
            }
            __syncthreads();
            // columns: A <- A J and V <- V J.  A lane owns one index pair (there are at most 32), a warp takes
            // every fourth row: no index arithmetic beyond additions, and the rotation stays in registers.
            if (lane < half) {
                const int pp = s.rot_p[lane], qq = s.rot_q[lane];
                const double c = s.rot_c[lane], sn = s.rot_s[lane];
                for (int i = warp; i < n; i += kEigThreads / 32) {
                    double* ra = s.a + i * LD;
                    double* rv = s.v + i * LD;
                    const double x = ra[pp], y = ra[qq], u = rv[pp], w = rv[qq];
                    ra[pp] = fma(c, x, -sn * y);
                    ra[qq] = fma(sn, x, c * y);
                    rv[pp] = fma(c, u, -sn * w);
                    rv[qq] = fma(sn, u, c * w);
                }
            }
            __syncthreads();
            // rows: A <- J^T A.  A warp takes every fourth pair, its lanes the columns.
            for (int k = warp; k < half; k += kEigThreads / 32) {
                const int pp = s.rot_p[k], qq = s.rot_q[k];
                const double c = s.rot_c[k], sn = s.rot_s[k];
                for (int i = lane; i < n; i += 32) {
                    const double x = s.a[pp * LD + i], y = s.a[qq * LD + i];
                    s.a[pp * LD + i] = fma(c, x, -sn * y);
                    s.a[qq * LD + i] = fma(sn, x, c * y);
                }
            }
            __syncthreads();
        }
    }

    if (tid < MP) {
        double inv = 0.0;
        if (tid < m && !bad) {
            const double lam = ldexp(s.a[tid * LD + tid], scale_exp);
            if (lam < floor) atomicOr(&s.flags, COMPACTOR_STATUS_RANK);
            inv = rsqrt(fmax(lam, floor));
        }
        s.inv_sqrt[tid] = inv;
    }
    __syncthreads();

    {   // W = Phi V Lambda^-1/2: one thread per row of Phi
        const int row = tid;
        double r[MP];
#pragma unroll
        for (int c = 0; c < MP; ++c) r[c] = (c < m && !bad) ? (double)phi[row * m + c] : 0.0;
        __nv_bfloat16* w_hi = w_out + (size_t)unit * w_elems_per_unit(MP);
        __nv_bfloat16* w_lo = w_hi + (size_t)MP * kD;
        for (int j = 0; j < MP; ++j) {
            double acc0 = 0.0, acc1 = 0.0;
#pragma unroll
            for (int c = 0; c < MP; c += 2) {
                acc0 = fma(r[c], s.v[c * LD + j], acc0);
                acc1 = fma(r[c + 1], s.v[(c + 1) * LD + j], acc1);
            }
            const double wj = (j < m) ? (acc0 + acc1) * s.inv_sqrt[j] : 0.0;
            const __nv_bfloat16 hi = __double2bfloat16(wj);
            w_hi[j * kD + row] = hi;
            w_lo[j * kD + row] = __double2bfloat16(wj - (double)__bfloat162float(hi));
        }
    }
    if (tid == 0 && status != nullptr && s.flags != 0) atomicOr(&status[unit], s.flags);
}

template <int MP>
cudaError_t launch_factor_mp(const Plan& p, const Mat& k, const double* partials, const float* phi,
                             double* a_parts, __nv_bfloat16* w, float* scores, int* status, int factorization, double eig_floor,
                             int sm_count, cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    const int smem = (int)sizeof(ProjectSmem<MP>);
    cudaError_t e = cudaFuncSetAttribute(project_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    const int n_items = units * kPairs;
    const int resident = 2 * sm_count;                            // two CTAs fit on an SM
    const int grid = n_items < resident ? n_items : resident;
    e = launch_chained(kPdlProject, project_kernel<MP>, dim3(grid), dim3(kProjThreads), smem, stream, p, k, partials, phi, a_parts, n_items);
    if (e != cudaSuccess) return e;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (factorization == COMPACTOR_FACTOR_EIG) {
        if constexpr (MP <= 64) {
            const int esmem = (int)sizeof(EigSmem<MP>);
            e = cudaFuncSetAttribute(eig_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, esmem);
            if (e != cudaSuccess) return e;
            eig_kernel<MP><<<units, kEigThreads, esmem, stream>>>(p, a_parts, phi, eig_floor, w, status);
        } else {
            return cudaErrorInvalidValue;        // two m x m fp64 matrices no longer fit in shared memory
        }
    } else {
        const int csmem = (int)sizeof(CholSmem<MP>);
        e = cudaFuncSetAttribute(cholesky_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, csmem);
        if (e != cudaSuccess) return e;
        e = launch_chained(kPdlCholesky, cholesky_kernel<MP>, dim3(units), dim3(kCholThreads), csmem, stream, p, k, (const double*)a_parts, phi, w, scores, status);
        if (e != cudaSuccess) return e;
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_factor(const Plan& p, const Mat& k, const double* partials, const float* phi, double* a_parts,
                          __nv_bfloat16* w, float* scores, int* status, int factorization, double eig_floor, int sm_count,
                          cudaStream_t stream) {
    if (p.layers * p.heads * p.batch == 0) return cudaSuccess;
    switch (p.mp) {
        case 16: return launch_factor_mp<16>(p, k, partials, phi, a_parts, w, scores, status, factorization, eig_floor, sm_count, stream);
        case 32: return launch_factor_mp<32>(p, k, partials, phi, a_parts, w, scores, status, factorization, eig_floor, sm_count, stream);
        case 48: return launch_factor_mp<48>(p, k, partials, phi, a_parts, w, scores, status, factorization, eig_floor, sm_count, stream);
        case 64: return launch_factor_mp<64>(p, k, partials, phi, a_parts, w, scores, status, factorization, eig_floor, sm_count, stream);
        case 128: return launch_factor_mp<128>(p, k, partials, phi, a_parts, w, scores, status, factorization, eig_floor, sm_count, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace compactor

// Double-precision building blocks of the small factorisation (Algorithm 1, line 4, by the Cholesky route that
// Section 3.2 and Appendix C allow): fp64 tensor-core products, a panel Cholesky factorisation and the blocked
// solve W = Phi L^-T.  Shared by the factor kernels and the one-kernel sweep.
//
// On this part only the fp64 mma path has throughput; ordinary double-precision instructions have about 50 cycles
// of latency, so everything here is arranged to keep dependency chains short and loads unconditional.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "common.cuh"

namespace compactor {
namespace factor_math {

constexpr double kPivotFloor = 9.5367431640625e-07;   // 2^-20: the fp32 noise floor of the Gram sums
constexpr int kPanel = 8;                             // columns per panel of the Cholesky factorisation
constexpr int kTRows = 32;                            // rows of T staged at a time for G = Phi^T T

// D (8 x 8) += A (8 x 4) B (4 x 8): lane (fr = lane / 4, fk = lane % 4) holds A[fr][fk], B[fk][fr] and
// D[fr][2 fk], D[fr][2 fk + 1].
__device__ __forceinline__ void mma_f64(double (&d)[2], double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(d[0]), "+d"(d[1]) : "d"(a), "d"(b));
}

// 1 / sqrt(x) for a positive, finite, normal x: single-precision seed on x scaled by an even power of two
// into [1, 4), one Newton step in double precision (relative error of the order of 1e-13: the factor it
// scales stays consistent, L L^T = G to that accuracy, far below what the scores resolve), scaled back.
// The chain of 48 dependent pivots is what the factorisation's latency consists of, so the conversions
// between the two formats are done on the bit patterns (integer instructions have a fraction of the
// latency of the conversion instructions).
__device__ __forceinline__ double fast_rsqrt(double x) {
    const int hi = __double2hiint(x), lo = __double2loint(x);
    const int eh = (((hi >> 20) & 0x7ff) - 1023) >> 1;
    const int hs = hi - ((2 * eh) << 20);                                   // x * 2^(-2 eh), in [1, 4)
    const double xs = __hiloint2double(hs, lo);
    const float xf = __int_as_float(((hs - ((1023 - 127) << 20)) << 3) | (int)((unsigned)lo >> 29));   // xs truncated to fp32
    const int yb = __float_as_int(rsqrtf(xf));                              // in (0.5, 1]
    double y = __hiloint2double((int)((unsigned)yb >> 3) + ((1023 - 127) << 20), yb << 29);
    const double h = 0.5 * xs;
    y = y * fma(-h * y, y, 1.5);
    return __hiloint2double(__double2hiint(y) - (eh << 20), __double2loint(y));
}

// One panel (columns j0 .. j1-1, at most eight) of the right-looking Cholesky factorisation, by one warp.
// `g` holds the lower triangle by columns, g[c * LD + i] = A[i][c] for i >= c.  Every lane factors the
// panel's 8 x 8 diagonal block itself (the same arithmetic in all lanes: no pivot has to travel), then
// solves the panel entries of its own rows (lane, lane + 32, ...) against it.  Also leaves the inverse of
// the diagonal block's factor, X = L_JJ^-1, below the diagonal in the free triangle of `g`
// (g[(j0 + n) * LD + j0 + k] = X[n][k], k < n; the diagonal of X is inv_diag).  Pivots not larger than
// 2^-20 of their original diagonal entry are dropped (their column of L and of X is zero), and so is every pivot
// once `budget` of them have been kept in this panel (the caller knows an upper bound of the rank).
// Returns (pivots kept in this panel) * 2 + (1 if a pivot was dropped).
template <int LD>
__device__ __noinline__ int factor_panel(double* g, const double* diag0, double* inv_diag, int j0, int j1, int m, int lane,
                                         int budget) {
    constexpr int kOwn = (LD + 31) / 32;          // rows per lane: lane, lane + 32, ...
    double dd[kPanel][kPanel];                    // lower triangle of the diagonal block
#pragma unroll
    for (int r = 0; r < kPanel; ++r)
#pragma unroll
        for (int c = 0; c <= r; ++c) {               // loads are unconditional (they then travel together); masked afterwards
            const double v = g[(j0 + c) * LD + j0 + r];
            dd[r][c] = (j0 + r < j1) ? v : 0.0;
        }
    double a[kOwn][kPanel];
#pragma unroll
    for (int o = 0; o < kOwn; ++o)
#pragma unroll
        for (int c = 0; c < kPanel; ++c) {
            const int r = lane + 32 * o;
            const double v = g[(j0 + c) * LD + min(r, LD - 1)];
            a[o][c] = (r < m && j0 + c < j1) ? v : 0.0;
        }
    // One straight line of code (no branches): the pivot chain, the solves of the lane's rows and the inverse of the
    // diagonal block are independent chains of double-precision operations, and the compiler interleaves them.
    // Columns past j1 (a short last panel) have a zero pivot: they are "dropped" (zero column) without being counted.
    double inv[kPanel];
    bool dropped = false;
    int kept = 0;
#pragma unroll
    for (int c = 0; c < kPanel; ++c) {
        const double piv = dd[c][c], d0 = diag0[min(j0 + c, LD - 1)];
        const bool keep = piv > kPivotFloor * d0 && d0 > 0.0 && kept < budget;
        kept += keep;
        inv[c] = keep ? fast_rsqrt(keep ? piv : 1.0) : 0.0;
        dropped = dropped || (!keep && j0 + c < j1);
        dd[c][c] = piv * inv[c];
#pragma unroll
        for (int r = c + 1; r < kPanel; ++r) dd[r][c] *= inv[c];
#pragma unroll
        for (int r = c + 1; r < kPanel; ++r)
#pragma unroll
            for (int c2 = c + 1; c2 <= r; ++c2) dd[r][c2] = fma(-dd[r][c], dd[c2][c], dd[r][c2]);
        // the lane's rows: l[c] = (a[c] - sum_{c' < c} l[c'] L_JJ[c][c']) / L_JJ[c][c], right-looking
#pragma unroll
        for (int o = 0; o < kOwn; ++o) {
            a[o][c] *= inv[c];
#pragma unroll
            for (int c2 = c + 1; c2 < kPanel; ++c2) a[o][c2] = fma(-a[o][c], dd[c2][c], a[o][c2]);
        }
    }
#pragma unroll
    for (int o = 0; o < kOwn; ++o)
#pragma unroll
        for (int c = 0; c < kPanel; ++c) {
            const int r = lane + 32 * o;
            if (j0 + c < j1 && r < m && r >= j0 + c) g[(j0 + c) * LD + r] = a[o][c];
        }
    // X = L_JJ^-1 by forward substitution (every lane computes it, lane k stores column k):
    // x[k] = inv[k], x[n] = -inv[n] sum_{t=k}^{n-1} L_JJ[n][t] x[t], right-looking
#pragma unroll
    for (int k = 0; k < kPanel; ++k) {
        double x[kPanel];
#pragma unroll
        for (int n = k + 1; n < kPanel; ++n) x[n] = 0.0;
        x[k] = inv[k];
#pragma unroll
        for (int t = k; t < kPanel; ++t) {
            if (t > k) x[t] *= inv[t];
#pragma unroll
            for (int n = t + 1; n < kPanel; ++n) x[n] = fma(-dd[n][t], x[t], x[n]);
        }
        if (lane == k) {
            if (j0 + k < j1) inv_diag[j0 + k] = inv[k];
#pragma unroll
            for (int n = k + 1; n < kPanel; ++n)
                if (j0 + n < j1) g[(j0 + n) * LD + j0 + k] = x[n];
        }
    }
    return kept * 2 + (dropped ? 1 : 0);
}

// W = Phi L^-T for the 16 rows of Phi that one warp owns, as a blocked forward substitution on fp64
// mma.m8n8k4: W_J = (Phi_J - sum_{I<J} W_I L_JI^T) X_JJ^T, the blocks of W kept in registers as A
// fragments.  Each 8 x 8 block of the result is split into two bf16 terms and stored at
// w_hi[col * 128 + row] and w_hi[(MP + col) * 128 + row].
template <int MP>
__device__ __noinline__ void solve_w_tiles(const float* phi, const double* g, const double* inv_diag, int row_base,
                                           int lane, __nv_bfloat16* w_hi) {
    constexpr int LD = MP, kNB = MP / 8;
    const int fr = lane >> 2, fk = lane & 3;
    __nv_bfloat16* w_lo = w_hi + (size_t)MP * kD;
    double wa[2][kNB][2];                         // [m-tile][block][k-step]: A fragments of the finished blocks
#pragma unroll
    for (int J = 0; J < kNB; ++J) {
        double d[2][2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const int row = row_base + mt * 8 + fr;
            d[mt][0] = (double)phi[row * MP + J * 8 + 2 * fk];
            d[mt][1] = (double)phi[row * MP + J * 8 + 2 * fk + 1];
        }
#pragma unroll
        for (int I = 0; I < J; ++I)
#pragma unroll
            for (int sk = 0; sk < 2; ++sk) {
                const double b = -g[(I * 8 + 4 * sk + fk) * LD + J * 8 + fr];       // -(L_JI^T)[k][n] = -L[J*8+n][I*8+k]
                mma_f64(d[0], wa[0][I][sk], b);
                mma_f64(d[1], wa[1][I][sk], b);
            }
        // right-hand block times X_JJ^T: fragments of the left operand come from the accumulator by quad shuffles
        double e[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
#pragma unroll
        for (int sk = 0; sk < 2; ++sk) {
            const int k = 4 * sk + fk, n = fr;                                        // B[k][n] = X[n][k]
            const double xg = g[(J * 8 + n) * LD + J * 8 + k], xd = inv_diag[J * 8 + n];    // both loaded, one chosen
            const double b = k < n ? xg : (k == n ? xd : 0.0);
            const int src = (lane & ~3) | (2 * sk + (fk >> 1));
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                const double v0 = __shfl_sync(0xffffffffu, d[mt][0], src), v1 = __shfl_sync(0xffffffffu, d[mt][1], src);
                mma_f64(e[mt], (fk & 1) ? v1 : v0, b);
            }
        }
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const int row = row_base + mt * 8 + fr;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int col = J * 8 + 2 * fk + q;
                const __nv_bfloat16 hi = __double2bfloat16(e[mt][q]);
                w_hi[col * kD + row] = hi;
                w_lo[col * kD + row] = __double2bfloat16(e[mt][q] - (double)__bfloat162float(hi));
            }
#pragma unroll
            for (int sk = 0; sk < 2; ++sk) {
                const int src = (lane & ~3) | (2 * sk + (fk >> 1));
                const double v0 = __shfl_sync(0xffffffffu, e[mt][0], src), v1 = __shfl_sync(0xffffffffu, e[mt][1], src);
                wa[mt][J][sk] = (fk & 1) ? v1 : v0;
            }
        }
    }
}


// G = Phi^T T (lower-triangular 8 x 8 tiles only) for one unit, by NWARPS warps.  `t_unit` is T [128][MP] in
// global memory (read past L1), `phi` the sketch [128][MP] fp32 in shared memory, `tstage` shared scratch of
// kTRows * (MP + 4) doubles, `g` the result by columns (g[c * MP + i] = G[i][c], i >= c); `g` may overlap `tstage`.
// Returns false (in every thread of a warp that saw it) if an entry of G is not finite.
template <int MP, int NWARPS, class Sync>
__device__ __forceinline__ bool gram_of_sketch(const double* __restrict__ t_unit, const float* phi, double* g, double* tstage,
                                               int tid, Sync sync) {
    constexpr int LD = MP, LDT = MP + 4, kNT = MP / 8, kThreadsHere = 32 * NWARPS;
    constexpr int kLower = kNT * (kNT + 1) / 2;
    constexpr int kMaxTiles = (kLower + NWARPS - 1) / NWARPS;
    constexpr int kPerChunk = kTRows * MP / kThreadsHere;
    constexpr bool kPreload = (kD / kTRows) * kPerChunk <= 24;           // all of T in flight at once if it fits the registers
    const int warp = tid >> 5, lane = tid & 31, fr = lane >> 2, fk = lane & 3;
    double d[kMaxTiles][2];
    int tmt[kMaxTiles], tnt[kMaxTiles];
#pragma unroll
    for (int si = 0; si < kMaxTiles; ++si) {
        d[si][0] = d[si][1] = 0.0;
        int rem = warp + NWARPS * si, mt = 0;
        while (rem > mt) { rem -= mt + 1; ++mt; }
        tmt[si] = mt; tnt[si] = rem;
    }
    double tv[kPreload ? kD / kTRows : 1][kPerChunk];
    if constexpr (kPreload) {
#pragma unroll
        for (int chunk = 0; chunk < kD / kTRows; ++chunk)
#pragma unroll
            for (int u = 0; u < kPerChunk; ++u) tv[chunk][u] = __ldcg(t_unit + (size_t)chunk * kTRows * MP + tid + u * kThreadsHere);
    }
#pragma unroll
    for (int chunk = 0; chunk < kD / kTRows; ++chunk) {
        if constexpr (!kPreload) {
#pragma unroll
            for (int u = 0; u < kPerChunk; ++u) tv[0][u] = __ldcg(t_unit + (size_t)chunk * kTRows * MP + tid + u * kThreadsHere);
        }
        if (chunk > 0) sync();
#pragma unroll
        for (int u = 0; u < kPerChunk; ++u) {
            const int e = tid + u * kThreadsHere, rr = e / MP, cc = e - rr * MP;
            tstage[rr * LDT + cc] = tv[kPreload ? chunk : 0][u];
        }
        sync();
#pragma unroll
        for (int si = 0; si < kMaxTiles; ++si) {
            if (warp + NWARPS * si >= kLower) continue;
#pragma unroll
            for (int k0 = 0; k0 < kTRows; k0 += 4)
                mma_f64(d[si], (double)phi[(chunk * kTRows + k0 + fk) * MP + tmt[si] * 8 + fr],
                        tstage[(k0 + fk) * LDT + tnt[si] * 8 + fr]);
        }
    }
    sync();
    bool finite = true;
#pragma unroll
    for (int si = 0; si < kMaxTiles; ++si) {
        if (warp + NWARPS * si >= kLower) continue;
        // fragment (row mt*8 + fr, columns nt*8 + 2 fk, + 1), stored by column
        g[(tnt[si] * 8 + 2 * fk) * LD + tmt[si] * 8 + fr] = d[si][0];
        g[(tnt[si] * 8 + 2 * fk + 1) * LD + tmt[si] * 8 + fr] = d[si][1];
        finite = finite && isfinite(d[si][0]) && isfinite(d[si][1]);
    }
    return finite;
}

// In-place Cholesky factorisation G = L L^T of the m leading rows and columns of `g` (by columns, stride MP),
// right-looking by panels of eight columns: warp 0 factors the panel (factor_panel), all warps update what
// follows on fp64 mma.  `diag0` must hold the original diagonal and `inv_diag` zeros on entry; on return
// inv_diag[j] = 1 / L[j][j] (0 for a dropped pivot) and the inverses of the diagonal blocks lie in the free
// triangle of `g`.  COMPACTOR_STATUS_RANK is or-ed into *flags (shared memory) if a pivot was dropped.  `rank_bound`: at
// most this many pivots are kept (a sequence of fewer tokens than sketch columns cannot have more).
template <int MP, int NWARPS, class Sync>
__device__ __forceinline__ void cholesky_panels(double* g, const double* diag0, double* inv_diag, int m, int tid, int* flags, Sync sync,
                                                int rank_bound = 1 << 30) {
    constexpr int LD = MP;
    const int warp = tid >> 5, lane = tid & 31, fr = lane >> 2, fk = lane & 3;
    int kept = 0;                                         // pivots kept so far (only warp 0 counts)
    for (int j0 = 0; j0 < m; j0 += kPanel) {
        const int j1 = min(j0 + kPanel, m);
        if (warp == 0) {
            const int res = factor_panel<LD>(g, diag0, inv_diag, j0, j1, m, lane, rank_bound - kept);
            kept += res >> 1;
            if (lane == 0 && (res & 1)) atomicOr(flags, COMPACTOR_STATUS_RANK);
        }
        sync();
        // trailing block, rows and columns j1 .. : A_ij -= L_i L_j^T by 8 x 8 tiles (lower tiles only; rows and
        // columns past m hold zeros)
        const int nb = (MP - j1) / 8;
        if (j1 < m && nb > 0) {
            for (int tile = warp; tile < nb * (nb + 1) / 2; tile += NWARPS) {
                int rem = tile, bi = 0;
                while (rem > bi) { rem -= bi + 1; ++bi; }
                const int bj = rem;
                double* cp = g + (j1 + 8 * bj + 2 * fk) * LD + j1 + 8 * bi + fr;      // fragment (row fr, columns 2 fk, + 1)
                double d[2] = {cp[0], cp[LD]};
#pragma unroll
                for (int sk = 0; sk < 2; ++sk) {
                    const double av = g[(j0 + 4 * sk + fk) * LD + j1 + 8 * bi + fr];   // L[j1 + 8 bi + fr][j0 + k]
                    const double bv = g[(j0 + 4 * sk + fk) * LD + j1 + 8 * bj + fr];   // (L_j^T)[k][n] = L[j1 + 8 bj + n][j0 + k]
                    mma_f64(d, -av, bv);
                }
                cp[0] = d[0];
                cp[LD] = d[1];
            }
            sync();
        }
    }
}

}  // namespace factor_math
}  // namespace compactor

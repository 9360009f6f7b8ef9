// Per-unit top-k (Section 3.4: keep the ceil(r N) highest-scoring tokens of a head) and the
// blend of Eq. 6.  Selection is an exact radix select on the order-preserving integer image of
// the fp32 scores (three passes: 11 + 11 + 10 bits) followed by one ordered compaction pass;
// equal scores go to the lower index and indices come out ascending.
#include "common.cuh"

namespace compactor {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kBins = 2048;

// Monotone map float -> uint32: larger float <=> larger key; -0 and +0 share a key (adding +0
// turns -0 into +0) and a NaN with the sign bit clear ranks highest.
__device__ __forceinline__ uint32_t order_key(float f) {
    uint32_t u = __float_as_uint(f + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SelectSmem {
    int hist[kBins];
    int warp_sums[kWarps];
    int warp_sums2[kWarps];
    int bin;          // chosen bin of the current pass
    int remaining;    // how many elements are still to be taken from the chosen bin
};

// Finds, scanning from the highest bin down, the bin where the running count reaches `want`.
// Returns (via smem) that bin and want - (count in higher bins).
__device__ void pick_bin(SelectSmem& s, int nbins, int want) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // thread t owns bins nbins-1-2t and nbins-2-2t (descending order)
    int b0 = nbins - 1 - 2 * tid, b1 = b0 - 1;
    int c0 = (b0 >= 0) ? s.hist[b0] : 0;
    int c1 = (b1 >= 0) ? s.hist[b1] : 0;
    int mine = c0 + c1;
    int incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += v;
    }
    if (lane == 31) s.warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int v = s.warp_sums[lane];
        int sc = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            int u = __shfl_up_sync(0xffffffffu, sc, off);
            if (lane >= off) sc += u;
        }
        s.warp_sums[lane] = sc - v;   // exclusive prefix of warp totals
    }
    __syncthreads();
    int before = s.warp_sums[warp] + incl - mine;   // elements in bins above mine
    if (before < want && want <= before + mine) {   // exactly one thread satisfies this
        if (want <= before + c0) { s.bin = b0; s.remaining = want - before; }
        else { s.bin = b1; s.remaining = want - before - c0; }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kThreads, 1)
select_kernel(Plan p, const float* __restrict__ scores, int* __restrict__ idx_out) {
    __shared__ SelectSmem s;
    const int unit = blockIdx.x;
    const int b = unit % p.batch, lh = unit / p.batch;
    const int n = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
    const int kk = p.cu_keep[b + 1] - p.cu_keep[b];
    if (kk <= 0 || n <= 0) return;
    const float* sc = scores + (size_t)lh * p.total_tokens + p.cu_seqlens[b];
    int* out = idx_out + (size_t)lh * p.total_keep + p.cu_keep[b];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (kk >= n) {
        for (int i = tid; i < n; i += kThreads) out[i] = i;
        return;
    }

    // --- radix select of the kk-th largest key -------------------------------------------
    uint32_t prefix = 0;      // high bits fixed so far
    int want = kk;
    const int shifts[3] = {21, 10, 0};
    const int widths[3] = {11, 11, 10};
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = shifts[pass], nb = 1 << widths[pass];
        for (int i = tid; i < kBins; i += kThreads) s.hist[i] = 0;
        __syncthreads();
        const int hi_shift = shift + widths[pass];     // bits above the current digit
        for (int i = tid; i < n; i += kThreads) {
            uint32_t key = order_key(sc[i]);
            bool match = (pass == 0) || ((key >> hi_shift) == (prefix >> hi_shift));
            if (match) atomicAdd(&s.hist[(key >> shift) & (nb - 1)], 1);
        }
        __syncthreads();
        pick_bin(s, nb, want);
        prefix |= (uint32_t)s.bin << shift;
        want = s.remaining;
        __syncthreads();
    }
    const uint32_t thr = prefix;   // key of the kk-th largest element
    const int ties = want;         // how many elements equal to it are kept (lowest indices first)

    // --- ordered compaction -----------------------------------------------------------------
    int base_gt = 0, base_eq = 0;          // counts over the elements before this block-iteration
    for (int start = 0; start < n; start += kThreads * 4) {
        const int i0 = start + tid * 4;
        uint32_t keys[4];
        int gt = 0, eq = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int i = i0 + e;
            keys[e] = (i < n) ? order_key(sc[i]) : 0u;
            if (i < n) { gt += keys[e] > thr; eq += keys[e] == thr; }
        }
        int packed = gt | (eq << 16);
        int incl = packed;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            int v = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += v;
        }
        if (lane == 31) s.warp_sums2[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int v = s.warp_sums2[lane];
            int scn = v;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                int u = __shfl_up_sync(0xffffffffu, scn, off);
                if (lane >= off) scn += u;
            }
            s.warp_sums[lane] = scn - v;
            if (lane == 31) s.bin = scn;      // block total (packed)
        }
        __syncthreads();
        int excl = s.warp_sums[warp] + incl - packed;
        int gt_before = base_gt + (excl & 0xffff);
        int eq_before = base_eq + (excl >> 16);
        int total = s.bin;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int i = i0 + e;
            if (i < n) {
                if (keys[e] > thr) {
                    out[gt_before + min(eq_before, ties)] = i;
                    ++gt_before;
                } else if (keys[e] == thr) {
                    if (eq_before < ties) out[gt_before + eq_before] = i;
                    ++eq_before;
                }
            }
        }
        base_gt += total & 0xffff;
        base_eq += total >> 16;
        __syncthreads();
    }
}

// Eq. 6: s = z(a) + lambda z(o), population standard deviation, per unit.  Overwrites the
// outlier scores in place.
__global__ void __launch_bounds__(kThreads, 1)
blend_kernel(Plan p, const float* __restrict__ attn, float lambda, float* __restrict__ scores) {
    __shared__ double red[4][kWarps];
    __shared__ double stats[4];
    const int unit = blockIdx.x;
    const int b = unit % p.batch, lh = unit / p.batch;
    const int n = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
    if (n <= 0) return;
    const size_t off = (size_t)lh * p.total_tokens + p.cu_seqlens[b];
    const float* a = attn + off;
    float* o = scores + off;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    auto block_sum2 = [&](double x, double y, int slot) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            x += __shfl_xor_sync(0xffffffffu, x, d);
            y += __shfl_xor_sync(0xffffffffu, y, d);
        }
        if (lane == 0) { red[slot][warp] = x; red[slot + 1][warp] = y; }
        __syncthreads();
        if (warp == 0) {
            double u = red[slot][lane], v = red[slot + 1][lane];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                u += __shfl_xor_sync(0xffffffffu, u, d);
                v += __shfl_xor_sync(0xffffffffu, v, d);
            }
            if (lane == 0) { stats[slot] = u; stats[slot + 1] = v; }
        }
        __syncthreads();
    };

    double sa = 0.0, so = 0.0;
    for (int i = tid; i < n; i += kThreads) { sa += (double)a[i]; so += (double)o[i]; }
    block_sum2(sa, so, 0);
    const double mean_a = stats[0] / n, mean_o = stats[1] / n;
    double va = 0.0, vo = 0.0;
    for (int i = tid; i < n; i += kThreads) {
        double da = (double)a[i] - mean_a, d_o = (double)o[i] - mean_o;
        va = fma(da, da, va); vo = fma(d_o, d_o, vo);
    }
    block_sum2(va, vo, 2);
    const double sd_a = sqrt(stats[2] / n), sd_o = sqrt(stats[3] / n);
    const double inv_a = sd_a > 0.0 ? 1.0 / sd_a : 0.0;
    const double inv_o = sd_o > 0.0 ? (double)lambda / sd_o : 0.0;
    for (int i = tid; i < n; i += kThreads)
        o[i] = (float)(((double)a[i] - mean_a) * inv_a + ((double)o[i] - mean_o) * inv_o);
}

}  // namespace

cudaError_t launch_select(const Plan& p, const float* scores, int* idx, cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    if (units == 0 || p.total_keep == 0) return cudaSuccess;
    select_kernel<<<units, kThreads, 0, stream>>>(p, scores, idx);
    return cudaGetLastError();
}

cudaError_t launch_blend(const Plan& p, const float* attn, float lambda, float* scores, cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    if (units == 0 || p.total_tokens == 0) return cudaSuccess;
    blend_kernel<<<units, kThreads, 0, stream>>>(p, attn, lambda, scores);
    return cudaGetLastError();
}

}  // namespace compactor

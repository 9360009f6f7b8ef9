// Per-unit top-k (Section 3.4: keep the ceil(r N) highest-scoring tokens of a head) and the
// blend of Eq. 6.  Selection is exact: it finds the key of the kk-th largest score (keys are the
// order-preserving integer image of the fp32 scores), then one ordered pass emits the indices of
// all larger scores plus the lowest-indexed ties, ascending.
//
// Finding the threshold.  Leverage scores of one head are spread over a narrow range, so a radix
// histogram on the leading float bits would pile everything into a dozen bins.  Instead the range
// is estimated from the first few thousand scores, a 2048-bin histogram linear in the score value
// is taken over all of them (values outside the estimate fall into the end bins; the binning is
// monotone, so it orders exactly), the bin holding the kk-th largest is found, its members are
// collected in shared memory and the exact key is found there by a three-pass radix select.
// Inputs that defeat this (non-finite values, a constant score, more members than fit) take the
// same three-pass radix select over global memory.
#include "common.cuh"

namespace compactor {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kBins = 2048;
constexpr int kSample = 4096;          // scores used to estimate the value range
constexpr int kCand = 8192;            // capacity of the candidate list
constexpr int kSub = 8;                // rows of the small shared count table

// Monotone map float -> uint32: larger float <=> larger key; -0 and +0 share a key (adding +0
// turns -0 into +0) and a NaN with the sign bit clear ranks highest.
__device__ __forceinline__ uint32_t order_key(float f) {
    uint32_t u = __float_as_uint(f + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SelectSmem {
    int hist[kBins];
    uint32_t cand[kCand];
    int cnt[2][kSub][kWarps];      // per-warp packed counts of the ordered pass, double buffered
    int row_total[2][kSub];
    int warp_sums[kWarps];
    float red[2][kWarps];
    int bin;          // chosen bin of the current pass
    int remaining;    // how many elements are still to be taken from the chosen bin
    int n_cand;
    float lo, scale;
    int fallback;
};

// Finds, scanning from the highest bin down, the bin where the running count reaches `want`.
// Leaves that bin and want - (count in higher bins) in shared memory.
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

// Calls f(value) for every score of the unit: unaligned head, 16-byte body with four vectors in
// flight per thread, tail.  The visiting order is unspecified.
template <class F>
__device__ __forceinline__ void for_each_score(const float* __restrict__ sc, int n, F f) {
    const int tid = threadIdx.x;
    const int head = min(n, (int)((4 - ((reinterpret_cast<uintptr_t>(sc) >> 2) & 3)) & 3));
    const int n_vec = (n - head) >> 2;
    const float4* body = reinterpret_cast<const float4*>(sc + head);
    if (tid < head) f(sc[tid]);
    for (int v0 = 0; v0 < n_vec; v0 += 4 * kThreads) {
        float4 q[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int vi = v0 + u * kThreads + tid;
            q[u] = vi < n_vec ? __ldg(body + vi) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (v0 + u * kThreads + tid < n_vec) { f(q[u].x); f(q[u].y); f(q[u].z); f(q[u].w); }
    }
    for (int i = head + 4 * n_vec + tid; i < n; i += kThreads) f(sc[i]);
}

// Three-pass radix select (11 + 11 + 10 bits) of the `want`-th largest key among the keys produced
// by `visit(tally)`; returns the key and, through *ties, how many keys equal to it are wanted.
template <class Visit>
__device__ uint32_t radix_select(SelectSmem& s, int want, int* ties, Visit visit) {
    const int tid = threadIdx.x;
    uint32_t prefix = 0;
    const int shifts[3] = {21, 10, 0};
    const int widths[3] = {11, 11, 10};
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = shifts[pass], nb = 1 << widths[pass];
        for (int i = tid; i < kBins; i += kThreads) s.hist[i] = 0;
        __syncthreads();
        const int hi_shift = shift + widths[pass];
        const uint32_t want_hi = prefix >> hi_shift;
        visit([&](uint32_t key) {
            if (pass == 0 || (key >> hi_shift) == want_hi) atomicAdd(&s.hist[(key >> shift) & (nb - 1)], 1);
        });
        __syncthreads();
        pick_bin(s, nb, want);
        prefix |= (uint32_t)s.bin << shift;
        want = s.remaining;
        __syncthreads();
    }
    *ties = want;
    return prefix;
}

// Key of the `want`-th largest of the values that `visit(f)` enumerates (f(value) is called once per
// value, in any order, by any thread), and through *ties how many values equal to that key belong
// to the top `want`.  `sample` / `n_sample` are some of the values, used to guess their range.
template <class Visit>
__device__ uint32_t find_threshold(SelectSmem& s, Visit visit, const float* __restrict__ sample, int n_sample,
                                   int want_total, int* ties, bool* all_finite_out = nullptr) {
    if (all_finite_out != nullptr) *all_finite_out = false;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // ---- value range from a sample ------------------------------------------------------------
    {
        float lo = INFINITY, hi = -INFINITY;
        bool finite = true;
        float smp[kSample / kThreads];
#pragma unroll
        for (int u = 0; u < kSample / kThreads; ++u) {
            const int i = u * kThreads + tid;
            smp[u] = sample[i < n_sample ? i : 0];
        }
#pragma unroll
        for (int u = 0; u < kSample / kThreads; ++u) {
            finite = finite && isfinite(smp[u]);
            lo = fminf(lo, smp[u]); hi = fmaxf(hi, smp[u]);
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, d));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, d));
        }
        const int all_finite = __syncthreads_and(finite ? 1 : 0);
        if (lane == 0) { s.red[0][warp] = lo; s.red[1][warp] = hi; }
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < kWarps; ++w) { lo = fminf(lo, s.red[0][w]); hi = fmaxf(hi, s.red[1][w]); }
            const float width = hi - lo;
            const float scale = (float)(kBins - 2) / width;              // sampled range -> bins 1 .. kBins-2
            s.fallback = !(all_finite && width > 0.f && isfinite(width) && isfinite(scale));
            s.lo = lo;
            s.scale = s.fallback ? 0.f : scale;
            s.n_cand = 0;
        }
        __syncthreads();
    }

    if (!s.fallback) {
        const float lo = s.lo, scale = s.scale;
        // monotone in v: subtraction, multiplication by a positive constant, clamping and truncation all are
        auto bin_of = [&](float v) {
            const float x = fminf(fmaxf((v - lo) * scale + 1.0f, 0.0f), (float)(kBins - 1));
            return (int)x;
        };
        for (int i = tid; i < kBins; i += kThreads) s.hist[i] = 0;
        __syncthreads();
        int nonfinite = 0;
        visit([&](float v) {
            if (!isfinite(v)) nonfinite = 1;
            atomicAdd(&s.hist[bin_of(v)], 1);
        });
        const int any_nonfinite = __syncthreads_or(nonfinite);
        pick_bin(s, kBins, want_total);
        const int tbin = s.bin, want = s.remaining;
        const int members = s.hist[tbin];
        __syncthreads();
        if (!any_nonfinite && members <= kCand) {
            if (all_finite_out != nullptr) *all_finite_out = true;       // every value has been seen and is finite
            visit([&](float v) {
                if (bin_of(v) == tbin) s.cand[atomicAdd(&s.n_cand, 1)] = order_key(v);
            });
            __syncthreads();
            const int nc = s.n_cand;
            return radix_select(s, want, ties, [&](auto tally) {
                for (int i = tid; i < nc; i += kThreads) tally(s.cand[i]);
            });
        }
    }
    return radix_select(s, want_total, ties, [&](auto tally) {
        visit([&](float v) { tally(order_key(v)); });
    });
}

// Ordered pass over one score vector: writes, ascending, the indices of the scores whose key exceeds
// `thr` and of the first `ties` scores whose key equals it.  The vector is cut into an unaligned
// head (0-3 scores), a 16-byte aligned body and a tail (0-3 scores).  Every warp owns a contiguous
// stretch of the body, read as float4 (four consecutive scores per lane): it first counts its
// scores above and at the threshold, one block-wide scan turns the counts into output offsets, and
// then each warp emits its stretch on its own (a shuffle scan of per-lane counts per 128 scores).
// The pass is bound by instruction issue, hence four scores per load and per scan.
// kPlain: every score is known to be finite, so that comparing the floats themselves orders them as the
// keys do (and -0 == +0 either way); that saves the key mapping, which is most of the work per score.
template <bool kPlain>
__device__ void emit_ordered(SelectSmem& s, const float* __restrict__ sc, int n, uint32_t thr, int ties,
                             int* __restrict__ out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int head = min(n, (int)((4 - ((reinterpret_cast<uintptr_t>(sc) >> 2) & 3)) & 3));
    const int n_vec = (n - head) >> 2;
    const int tail_begin = head + 4 * n_vec;
    const float4* body = reinterpret_cast<const float4*>(sc + head);
    const int per_warp = (((n_vec + kWarps - 1) / kWarps) + 31) & ~31;   // vectors per stretch, a multiple of 32
    const int vbegin = min(n_vec, warp * per_warp), vend = min(n_vec, vbegin + per_warp);
    constexpr int kAhead = 4;                                             // vector steps loaded together

    const float thr_f = __uint_as_float((thr & 0x80000000u) ? (thr & 0x7fffffffu) : ~thr);   // the float behind the key
    auto flags = [&](const float4& q, int& g, int& e) {                   // 4-bit masks: above / at the threshold
        if (kPlain) {
            g = (q.x > thr_f) | ((q.y > thr_f) << 1) | ((q.z > thr_f) << 2) | ((q.w > thr_f) << 3);
            e = (q.x == thr_f) | ((q.y == thr_f) << 1) | ((q.z == thr_f) << 2) | ((q.w == thr_f) << 3);
        } else {
            const uint32_t k0 = order_key(q.x), k1 = order_key(q.y), k2 = order_key(q.z), k3 = order_key(q.w);
            g = (k0 > thr) | ((k1 > thr) << 1) | ((k2 > thr) << 2) | ((k3 > thr) << 3);
            e = (k0 == thr) | ((k1 == thr) << 1) | ((k2 == thr) << 2) | ((k3 == thr) << 3);
        }
    };

    // ---- counts: head (warp 0), the warp's stretch, tail (last warp) ----------------------------
    int head_gt = 0, head_eq = 0;                       // head scores precede everything; every thread counts them
    for (int i = 0; i < head; ++i) {
        const uint32_t key = order_key(sc[i]);
        head_gt += key > thr; head_eq += key == thr;
    }
    int cnt_gt = 0, cnt_eq = 0;                         // full-width counters: a stretch may hold more than 2^16 scores
    for (int v0 = vbegin; v0 < vend; v0 += 32 * kAhead) {
        float4 q[kAhead];
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
            const int vi = v0 + u * 32 + lane;
            q[u] = vi < vend ? __ldg(body + vi) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
            int g, e;
            flags(q[u], g, e);
            if (v0 + u * 32 + lane < vend) { cnt_gt += __popc(g); cnt_eq += __popc(e); }
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        cnt_gt += __shfl_xor_sync(0xffffffffu, cnt_gt, d);
        cnt_eq += __shfl_xor_sync(0xffffffffu, cnt_eq, d);
    }
    __syncthreads();                                    // earlier users of the shared arrays are done
    if (lane == 0) { s.cnt[0][0][warp] = cnt_gt; s.cnt[1][0][warp] = cnt_eq; }
    __syncthreads();
    int base_gt, base_eq;
    {
        const int c_gt = s.cnt[0][0][lane], c_eq = s.cnt[1][0][lane];       // kWarps == 32: one pair of counts per lane
        int incl_gt = c_gt, incl_eq = c_eq;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t_gt = __shfl_up_sync(0xffffffffu, incl_gt, off);
            const int t_eq = __shfl_up_sync(0xffffffffu, incl_eq, off);
            if (lane >= off) { incl_gt += t_gt; incl_eq += t_eq; }
        }
        base_gt = head_gt + __shfl_sync(0xffffffffu, incl_gt - c_gt, warp);  // exclusive prefixes of this warp
        base_eq = head_eq + __shfl_sync(0xffffffffu, incl_eq - c_eq, warp);
    }

    // ---- emission: head, stretches, tail ----------------------------------------------------------
    if (tid == 0) {
        int g = 0, e = 0;
        for (int i = 0; i < head; ++i) {
            const uint32_t key = order_key(sc[i]);
            if (key > thr) out[g + min(e, ties)] = i;
            else if (key == thr && e < ties) out[g + e] = i;
            g += key > thr; e += key == thr;
        }
    }
    for (int v0 = vbegin; v0 < vend; v0 += 32 * kAhead) {
        float4 q[kAhead];
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
            const int vi = v0 + u * 32 + lane;
            q[u] = vi < vend ? __ldg(body + vi) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
            const int vi = v0 + u * 32 + lane;
            int g, e;
            flags(q[u], g, e);
            if (vi >= vend) { g = 0; e = 0; }
            const int mine = __popc(g) | (__popc(e) << 16);
            int incl = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += t;
            }
            int gt_before = base_gt + ((incl - mine) & 0xffff);
            int eq_before = base_eq + ((incl - mine) >> 16);
            const int i0 = head + 4 * vi;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if ((g >> j) & 1) { out[gt_before + min(eq_before, ties)] = i0 + j; ++gt_before; }
                else if ((e >> j) & 1) { if (eq_before < ties) out[gt_before + eq_before] = i0 + j; ++eq_before; }
            }
            const int total = __shfl_sync(0xffffffffu, incl, 31);
            base_gt += total & 0xffff;
            base_eq += total >> 16;
        }
    }
    if (warp == kWarps - 1 && lane == 0) {                // the tail follows the last stretch
        for (int i = tail_begin; i < n; ++i) {
            const uint32_t key = order_key(sc[i]);
            if (key > thr) out[base_gt + min(base_eq, ties)] = i;
            else if (key == thr && base_eq < ties) out[base_gt + base_eq] = i;
            base_gt += key > thr; base_eq += key == thr;
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
select_kernel(Plan p, const float* __restrict__ scores, int* __restrict__ idx_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SelectSmem& s = *reinterpret_cast<SelectSmem*>(smem_raw);
    const int unit = blockIdx.x;
    const int b = unit % p.batch, lh = unit / p.batch;
    const int n = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
    const int kk = p.cu_keep[b + 1] - p.cu_keep[b];
    if (kk <= 0 || n <= 0) return;
    const float* sc = scores + (size_t)lh * p.total_tokens + p.cu_seqlens[b];
    int* out = idx_out + (size_t)lh * p.total_keep + p.cu_keep[b];
    if (kk >= n) {
        for (int i = threadIdx.x; i < n; i += kThreads) out[i] = i;
        return;
    }
    int ties = 0;
    bool all_finite = false;
    const uint32_t thr = find_threshold(s, [&](auto f) { for_each_score(sc, n, f); }, sc, n, kk, &ties, &all_finite);
    if (all_finite) emit_ordered<true>(s, sc, n, thr, ties, out);
    else emit_ordered<false>(s, sc, n, thr, ties, out);
}

// ---- selection across the heads of a layer (Section 3.4's alternative) -------------------------
// Step 1, one CTA per (layer, sequence): the key of the (heads * kk)-th largest score over all heads,
// how many scores each head keeps (ties go to the lower head first, then to the lower index), and
// the heads' offsets inside the sequence's block of the output.
__global__ void __launch_bounds__(kThreads, 1)
across_threshold_kernel(Plan p, const float* __restrict__ scores, uint32_t* __restrict__ thr_out,
                        int* __restrict__ ties_out, int* __restrict__ head_offsets) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SelectSmem& s = *reinterpret_cast<SelectSmem*>(smem_raw);
    __shared__ int head_gt[64], head_eq[64];
    const int layer = blockIdx.x / p.batch, b = blockIdx.x % p.batch;
    const int n = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
    const int kk = p.cu_keep[b + 1] - p.cu_keep[b];
    const int H = p.heads, tid = threadIdx.x;
    int* offs = head_offsets + ((size_t)layer * p.batch + b) * (H + 1);
    int* ties_h = ties_out + ((size_t)layer * p.batch + b) * H;
    const float* base = scores + (size_t)layer * H * p.total_tokens + p.cu_seqlens[b];
    if (kk <= 0 || n <= 0) {
        for (int h = tid; h <= H; h += kThreads) offs[h] = 0;
        return;
    }
    if (kk >= n) {                                         // everything is kept
        for (int h = tid; h <= H; h += kThreads) offs[h] = h * n;
        for (int h = tid; h < H; h += kThreads) ties_h[h] = n;
        if (tid == 0) thr_out[blockIdx.x] = 0u;           // every key is >= 0: all scores count as ties or above
        return;
    }
    auto visit_all = [&](auto f) {
        for (int h = 0; h < H; ++h) for_each_score(base + (size_t)h * p.total_tokens, n, f);
    };
    int ties = 0;
    const uint32_t thr = find_threshold(s, visit_all, base, n, H * kk, &ties);
    // per-head counts above and at the threshold
    for (int h = tid; h < H; h += kThreads) { head_gt[h] = 0; head_eq[h] = 0; }
    __syncthreads();
    for (int h = 0; h < H; ++h) {
        int gt = 0, eq = 0;
        for_each_score(base + (size_t)h * p.total_tokens, n, [&](float v) {
            const uint32_t key = order_key(v);
            gt += key > thr; eq += key == thr;
        });
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            gt += __shfl_xor_sync(0xffffffffu, gt, d);
            eq += __shfl_xor_sync(0xffffffffu, eq, d);
        }
        if ((tid & 31) == 0) { atomicAdd(&head_gt[h], gt); atomicAdd(&head_eq[h], eq); }
    }
    __syncthreads();
    if (tid == 0) {
        int left = ties, off = 0;
        for (int h = 0; h < H; ++h) {
            const int take = min(left, head_eq[h]);
            left -= take;
            ties_h[h] = take;
            offs[h] = off;
            off += head_gt[h] + take;
        }
        offs[H] = off;
        thr_out[blockIdx.x] = thr;
    }
}

// Step 2, one CTA per (layer, head, sequence): the head's kept indices, ascending.
__global__ void __launch_bounds__(kThreads, 1)
across_emit_kernel(Plan p, const float* __restrict__ scores, const uint32_t* __restrict__ thr_in,
                   const int* __restrict__ ties_in, const int* __restrict__ head_offsets, int* __restrict__ idx_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SelectSmem& s = *reinterpret_cast<SelectSmem*>(smem_raw);
    const int unit = blockIdx.x;
    const int b = unit % p.batch, lh = unit / p.batch;
    const int layer = lh / p.heads, head = lh % p.heads;
    const int n = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
    const int kk = p.cu_keep[b + 1] - p.cu_keep[b];
    if (kk <= 0 || n <= 0) return;
    const size_t lb = (size_t)layer * p.batch + b;
    const int off = head_offsets[lb * (p.heads + 1) + head];
    const int count = head_offsets[lb * (p.heads + 1) + head + 1] - off;
    if (count <= 0) return;
    const float* sc = scores + (size_t)lh * p.total_tokens + p.cu_seqlens[b];
    int* out = idx_out + (size_t)layer * p.heads * p.total_keep + (size_t)p.heads * p.cu_keep[b] + off;
    if (kk >= n) {
        for (int i = threadIdx.x; i < n; i += kThreads) out[i] = i;
        return;
    }
    emit_ordered<false>(s, sc, n, thr_in[lb], ties_in[lb * p.heads + head], out);
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
    const int smem = (int)sizeof(SelectSmem);
    cudaError_t e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    select_kernel<<<units, kThreads, smem, stream>>>(p, scores, idx);
    return cudaGetLastError();
}

cudaError_t launch_select_across(const Plan& p, const float* scores, int* idx, int* head_offsets, uint32_t* thr,
                                 int* ties, cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    if (units == 0 || p.heads > 64) return units == 0 ? cudaSuccess : cudaErrorInvalidValue;
    const int smem = (int)sizeof(SelectSmem);
    cudaError_t e = cudaFuncSetAttribute(across_threshold_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(across_emit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    across_threshold_kernel<<<p.layers * p.batch, kThreads, smem, stream>>>(p, scores, thr, ties, head_offsets);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    across_emit_kernel<<<units, kThreads, smem, stream>>>(p, scores, thr, ties, head_offsets, idx);
    return cudaGetLastError();
}

cudaError_t launch_blend(const Plan& p, const float* attn, float lambda, float* scores, cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    if (units == 0 || p.total_tokens == 0) return cudaSuccess;
    blend_kernel<<<units, kThreads, 0, stream>>>(p, attn, lambda, scores);
    return cudaGetLastError();
}

}  // namespace compactor

// Per-unit top-k (Section 3.4: keep the ceil(r N) highest-scoring tokens of a head) and the
// blend of Eq. 6.  Selection is exact: it finds the key of the kk-th largest score (keys are the
// order-preserving integer image of the fp32 scores), then one ordered pass emits the indices of
// all larger scores plus the lowest-indexed ties, ascending.
//
// Finding the threshold.  Leverage scores of one head are spread over a narrow range, so a radix
// histogram on the leading float bits would pile everything into a dozen bins.  Instead the range
// is estimated from the first few thousand scores, a 2048-bin histogram linear in the score value
// is taken over all of them (values outside the estimate fall into the end bins; the binning is
// monotone, so it orders exactly) and the bin holding the kk-th largest is found.  A second pass, cut
// the way the ordered pass is, counts per warp the scores in higher bins and lists the members of that
// bin; the exact key is found among them (a few hundred) and they are added to their warps' counts, so
// the ordered pass starts from finished counts.  Inputs that defeat this (non-finite values, a constant
// score, more members than fit) take a three-pass radix select over global memory and an ordered pass
// that counts for itself.  Where one CTA per score vector would leave most SMs idle, the vectors are cut
// into slices over many CTAs (the multi_* kernels below).
#include <type_traits>

#include "common.cuh"

namespace compactor {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kBins = 2048;
constexpr int kSample = 4096;          // scores used to estimate the value range
constexpr int kCand = 8192;            // capacity of the candidate list

// Monotone map float -> uint32: larger float <=> larger key; -0 and +0 share a key (adding +0
// turns -0 into +0) and a NaN with the sign bit clear ranks highest.
__device__ __forceinline__ uint32_t order_key(float f) {
    uint32_t u = __float_as_uint(f + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SelectSmem {
    int hist[kBins];
    uint32_t cand[kCand];
    unsigned char cand_warp[kCand];   // which warp's stretch a candidate lies in (255: the unaligned head or tail)
    int warp_gt[kWarps], warp_eq[kWarps];   // per warp stretch: scores above / at the threshold (ordered pass)
    int stage[kWarps][512];        // kept indices of 4 x 128 scores per warp, in output order
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
        {   // the next round's lines (128 bytes = 8 vectors each) are asked into L2 while this round is consumed
            const int vi = v0 + 4 * kThreads + tid * 8;
            if (tid < kThreads / 2 && vi < n_vec) asm volatile("prefetch.global.L2 [%0];" ::"l"(body + vi));
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

// Value range of a score vector from its first kSample entries: leaves in shared memory the lower end,
// the scale that maps the sampled range onto bins 1 .. kBins-2, and `fallback` when the sample is not
// finite or has no width.  Every CTA that is given the same sample arrives at the same numbers.
// *lopsided (optional): nine tenths of the sample lie in a sixteenth of its range, at either end.
__device__ void compute_range(SelectSmem& s, const float* __restrict__ sample, int n_sample, bool* lopsided = nullptr) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
    if (warp == 0) {                                                   // kWarps == 32: one pair per lane
        lo = s.red[0][lane]; hi = s.red[1][lane];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, d));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, d));
        }
    }
    if (tid == 0) {
        const float width = hi - lo;
        const float scale = (float)(kBins - 2) / width;              // sampled range -> bins 1 .. kBins-2
        s.fallback = !(all_finite && width > 0.f && isfinite(width) && isfinite(scale));
        s.lo = lo;
        s.scale = s.fallback ? 0.f : scale;
        s.n_cand = 0;
    }
    __syncthreads();
    if (lopsided != nullptr) {
        *lopsided = false;
        if (!s.fallback && n_sample >= 512) {
            const float lo1 = s.lo, sixteenth = (float)(kBins - 2) / s.scale * 0.0625f;
            int both = 0;                                               // low in bits 0-15, high in bits 16-31
#pragma unroll
            for (int u = 0; u < kSample / kThreads; ++u)
                if (u * kThreads + tid < n_sample)
                    both += (smp[u] < lo1 + sixteenth ? 1 : 0) + (smp[u] > lo1 + 15.f * sixteenth ? 1 << 16 : 0);
            both = __reduce_add_sync(0xffffffffu, both);
            if (lane == 0) s.warp_sums[warp] = both;
            __syncthreads();
            both = __reduce_add_sync(0xffffffffu, s.warp_sums[lane]);   // kWarps == 32: one sum per lane
            const int low = both & 0xffff, high = both >> 16;
            const int n_smp = min(n_sample, kSample);
            *lopsided = 10 * low > 9 * n_smp || 10 * high > 9 * n_smp;
        }
    }
}

// Bin of a score: monotone in v (subtraction, multiplication by a positive constant, clamping and
// rounding all are; the rounding is an addition, cheaper than a float-to-int conversion), so the bins order the scores exactly; values outside the sampled range land in
// the end bins.
__device__ __forceinline__ int bin_of(float v, float lo, float scale) {
    const float x = fminf(fmaxf((v - lo) * scale + 1.0f, 0.0f), (float)(kBins - 1));
    return __float_as_int(x + 8388608.0f) & (2 * kBins - 1);   // round to nearest: at 2^23 the integer sits in the low mantissa bits
}

// Key of the `want`-th largest of the values that `visit(f)` enumerates (f(value) is called once per
// value, in any order, by any thread), and through *ties how many values equal to that key belong
// to the top `want`.  `sample` / `n_sample` are some of the values, used to guess their range.
template <class Visit>
__device__ uint32_t find_threshold(SelectSmem& s, Visit visit, const float* __restrict__ sample, int n_sample,
                                   int want_total, int* ties, bool* all_finite_out = nullptr) {
    if (all_finite_out != nullptr) *all_finite_out = false;
    const int tid = threadIdx.x;
    compute_range(s, sample, n_sample);

    if (!s.fallback) {
        const float lo = s.lo, scale = s.scale;
        auto bin_of = [&](float v) { return compactor::bin_of(v, lo, scale); };
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

// Narrows the range left by compute_range() to the bins that hold 99 % of the sample (values outside fall into
// the end bins, as before), as long as those are less than half of all bins (three times at most).  Every CTA that
// is given the same sample arrives at the same range.
__device__ __noinline__ void narrow_range(SelectSmem& s, const float* __restrict__ sc, int n_smp) {
    const int tid = threadIdx.x;
    for (int round = 0; round < 3; ++round) {
        const float lo0 = s.lo, scale0 = s.scale;
        for (int i = tid; i < kBins; i += kThreads) s.hist[i] = 0;
        __syncthreads();
        for (int i = tid; i < n_smp; i += kThreads) atomicAdd(&s.hist[bin_of(sc[i], lo0, scale0)], 1);
        __syncthreads();
        pick_bin(s, kBins, n_smp / 200 + 1);
        const int b_hi = s.bin;
        __syncthreads();
        pick_bin(s, kBins, n_smp - n_smp / 200);
        const int b_lo = s.bin;
        __syncthreads();
        if (b_hi - b_lo + 1 >= kBins / 2) break;
        const float new_lo = lo0 + (float)(b_lo - 1) / scale0;
        const float new_scale = (float)(kBins - 2) * scale0 / (float)(b_hi - b_lo + 1);
        if (!(isfinite(new_lo) && isfinite(new_scale) && new_scale > 0.f)) break;
        if (tid == 0) { s.lo = new_lo; s.scale = new_scale; }
        __syncthreads();
    }
}

// The threshold of one finite score vector together with what the ordered pass needs to start: per warp
// stretch (the same cut as emit_ordered's) the number of scores above and at the threshold.  First pass:
// the value-linear histogram (this is the pass that brings the scores in from HBM).  Second pass: a warp
// counts the scores of its stretch in bins above the threshold bin and lists the members of that bin
// with its own number; once the exact key is known among the listed ones, they are added to the counts
// of their warps, so the ordered pass need not count again.  Returns false (and has written nothing that
// matters) when the histogram route does not apply: the caller then takes find_threshold and the
// counting emit_ordered.
__device__ bool threshold_with_counts(SelectSmem& s, const float* __restrict__ sc, int n, int want_total,
                                      uint32_t* thr_out, int* ties_out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    bool lopsided = false;
    compute_range(s, sc, n, &lopsided);
    if (s.fallback) return false;
    // A few extreme scores among the sampled ones (the first token of a real context is one) stretch the range so
    // that the bulk lands in a handful of bins: all atomics of the histogram pass would then hit the same words.
    // So if nine tenths of the sample lie in a sixteenth of its range, the sample is binned, and if 99 % of it sit in
    // less than an eighth of the bins the range is narrowed to them (values outside fall into the end bins, as before);
    // the check is repeated once.
    if (lopsided) narrow_range(s, sc, min(n, kSample));
    const float lo = s.lo, scale = s.scale;
    for (int i = tid; i < kBins; i += kThreads) s.hist[i] = 0;
    __syncthreads();
    int nonfinite = 0;
    for_each_score(sc, n, [&](float v) {
        if (!isfinite(v)) nonfinite = 1;
        atomicAdd(&s.hist[bin_of(v, lo, scale)], 1);
    });
    const int any_nonfinite = __syncthreads_or(nonfinite);
    pick_bin(s, kBins, want_total);
    const int tbin = s.bin;
    int want = s.remaining;
    int members = s.hist[tbin];
    __syncthreads();
    // A few extreme scores among the sampled ones (the first token of a real context is one) stretch the range so that
    // the bulk lands in a handful of bins, too crowded for the list: then a second histogram over the threshold bin
    // alone, 2046 times finer, and the threshold bin of that.
    bool refined = false;
    float lo2 = 0.f, scale2 = 0.f;
    int tbin2 = 0;
    if (!any_nonfinite && members > kCand && tbin > 0 && tbin < kBins - 1) {
        lo2 = lo + (float)(tbin - 1) / scale;
        scale2 = scale * (float)(kBins - 2);
        if (isfinite(lo2) && isfinite(scale2)) {
            for (int i = tid; i < kBins; i += kThreads) s.hist[i] = 0;
            __syncthreads();
            for_each_score(sc, n, [&](float v) {
                if (bin_of(v, lo, scale) == tbin) atomicAdd(&s.hist[bin_of(v, lo2, scale2)], 1);
            });
            __syncthreads();
            pick_bin(s, kBins, want);
            tbin2 = s.bin;
            want = s.remaining;
            members = s.hist[tbin2];
            __syncthreads();
            refined = true;
        }
    }
    if (any_nonfinite || members > kCand) return false;
    // rank of a score: its bin, and inside the threshold bin its finer bin (both maps are monotone in the score);
    // 2 = above the threshold's bin, 1 = in it, 0 = below
    const bool fine = refined;
    const float f_lo = lo2, f_scale = scale2;
    const int f_bin = tbin2;
    auto placed = [=](float x) -> int {
        const int bin = bin_of(x, lo, scale);
        int code = bin > tbin ? 2 : (bin == tbin ? 1 : 0);
        if (fine && code == 1) {
            const int bin2 = bin_of(x, f_lo, f_scale);
            code = bin2 > f_bin ? 2 : (bin2 == f_bin ? 1 : 0);
        }
        return code;
    };

    const int head = min(n, (int)((4 - ((reinterpret_cast<uintptr_t>(sc) >> 2) & 3)) & 3));
    const int n_vec = (n - head) >> 2;
    const float4* body = reinterpret_cast<const float4*>(sc + head);
    const int per_warp = (((n_vec + kWarps - 1) / kWarps) + 31) & ~31;
    const int vbegin = min(n_vec, warp * per_warp), vend = min(n_vec, vbegin + per_warp);
    auto candidate = [&](float v, int tag) {
        const int pos = atomicAdd(&s.n_cand, 1);
        s.cand[pos] = order_key(v);
        s.cand_warp[pos] = (unsigned char)tag;
    };
    int above = 0;
    constexpr int kAhead = 4;
    auto stretch = [&](auto fine_tag) {                    // the warp's stretch; the refined test only where it is needed
        constexpr bool kFine = decltype(fine_tag)::value;
        for (int v0 = vbegin; v0 < vend; v0 += 32 * kAhead) {
            float4 q[kAhead];
#pragma unroll
            for (int u = 0; u < kAhead; ++u) {
                const int vi = v0 + u * 32 + lane;
                q[u] = vi < vend ? __ldg(body + vi) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < kAhead; ++u) {
                if (v0 + u * 32 + lane < vend) {
                    const float x[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (kFine) {
                            const int code = placed(x[j]);
                            above += code >> 1;
                            if (code == 1) candidate(x[j], warp);
                        } else {
                            const int bin = bin_of(x[j], lo, scale);
                            above += bin > tbin;
                            if (bin == tbin) candidate(x[j], warp);
                        }
                    }
                }
            }
        }
    };
    if (fine) stretch(std::true_type{}); else stretch(std::false_type{});
    auto loose = [&](float x) {                           // the few scores outside the 16-byte aligned body
        if (placed(x) == 1) candidate(x, 255);
    };
    if (tid < head) loose(sc[tid]);
    for (int i = head + 4 * n_vec + tid; i < n; i += kThreads) loose(sc[i]);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) above += __shfl_xor_sync(0xffffffffu, above, d);
    if (lane == 0) { s.warp_gt[warp] = above; s.warp_eq[warp] = 0; }
    __syncthreads();
    const int nc = s.n_cand;
    uint32_t thr;
    int ties;
    if (nc <= 64) {
        // few candidates: every one of them counts the others above and equal to itself
        if (tid < nc) {
            const uint32_t mine = s.cand[tid];
            int gt = 0, eq = 0;
            for (int j = 0; j < nc; ++j) { const uint32_t o = s.cand[j]; gt += o > mine; eq += o == mine; }
            if (gt < want && want <= gt + eq) { s.bin = (int)mine; s.remaining = want - gt; }   // the same pair from every holder of that key
        }
        __syncthreads();
        thr = (uint32_t)s.bin;
        ties = s.remaining;
    } else {
        thr = radix_select(s, want, &ties, [&](auto tally) {
            for (int i = tid; i < nc; i += kThreads) tally(s.cand[i]);
        });
    }
    for (int i = tid; i < nc; i += kThreads) {
        const int w = s.cand_warp[i];
        if (w < kWarps) {
            if (s.cand[i] > thr) atomicAdd(&s.warp_gt[w], 1);
            else if (s.cand[i] == thr) atomicAdd(&s.warp_eq[w], 1);
        }
    }
    *thr_out = thr;
    *ties_out = ties;
    return true;                                           // emit_ordered synchronises before it reads the counts
}

// Ordered pass over one score vector: writes, ascending, the indices of the scores whose key exceeds
// `thr` and of the first `ties` scores whose key equals it.  The vector is cut into an unaligned
// head (0-3 scores), a 16-byte aligned body and a tail (0-3 scores).  Every warp owns a contiguous
// stretch of the body, read as float4 (four consecutive scores per lane): it first counts its
// scores above and at the threshold (unless the caller has them already), one block-wide scan turns
// the counts into output offsets, and then each warp emits its stretch on its own, 512 scores at a
// time (see the loop).
// kPlain: every score is known to be finite, so that comparing the floats themselves orders them as the
// keys do (and -0 == +0 either way); that saves the key mapping, which is most of the work per score.
// A CTA may be given a slice of the vector: `index_base` is the index of sc[0] in the whole vector and
// gt0 / eq0 count the scores above / at the threshold that precede the slice.
// kCounted: the per-warp counts of the body are already in shared memory (threshold_with_counts left them).
template <bool kPlain, bool kCounted = false>
__device__ void emit_ordered(SelectSmem& s, const float* __restrict__ sc, int n, uint32_t thr, int ties,
                             int* __restrict__ out, int index_base = 0, int gt0 = 0, int eq0 = 0) {
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
    if (!kCounted) {
        int cnt_gt = 0, cnt_eq = 0;                     // full-width counters: a stretch may hold more than 2^16 scores
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
        __syncthreads();                                // earlier users of the shared arrays are done
        if (lane == 0) { s.warp_gt[warp] = cnt_gt; s.warp_eq[warp] = cnt_eq; }
    }
    __syncthreads();
    int base_gt, base_eq;
    {
        const int c_gt = s.warp_gt[lane], c_eq = s.warp_eq[lane];       // kWarps == 32: one pair of counts per lane
        int incl_gt = c_gt, incl_eq = c_eq;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t_gt = __shfl_up_sync(0xffffffffu, incl_gt, off);
            const int t_eq = __shfl_up_sync(0xffffffffu, incl_eq, off);
            if (lane >= off) { incl_gt += t_gt; incl_eq += t_eq; }
        }
        base_gt = gt0 + head_gt + __shfl_sync(0xffffffffu, incl_gt - c_gt, warp);  // exclusive prefixes of this warp
        base_eq = eq0 + head_eq + __shfl_sync(0xffffffffu, incl_eq - c_eq, warp);
    }

    // ---- emission: head, stretches, tail ----------------------------------------------------------
    if (tid == 0) {
        int g = gt0, e = eq0;
        for (int i = 0; i < head; ++i) {
            const uint32_t key = order_key(sc[i]);
            if (key > thr) out[g + min(e, ties)] = index_base + i;
            else if (key == thr && e < ties) out[g + e] = index_base + i;
            g += key > thr; e += key == thr;
        }
    }
    // A warp takes 512 scores at a time, 16 consecutive ones per lane: one packed shuffle scan of the lanes' counts
    // gives every lane its place (population counts and votes per score were the bottleneck before), the kept
    // indices go to the warp's staging buffer in output order and leave through coalesced stores.
    int* stage = s.stage[warp];
    auto above = [&](float x) { return kPlain ? x > thr_f : order_key(x) > thr; };
    auto equal = [&](float x) { return kPlain ? x == thr_f : order_key(x) == thr; };
    auto load4 = [&](int v0, float4 (&q)[kAhead]) {
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
            const int vi = v0 + kAhead * lane + u;
            q[u] = vi < vend ? __ldg(body + vi) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    float4 q[kAhead];
    load4(vbegin, q);
    for (int v0 = vbegin; v0 < vend; v0 += 32 * kAhead) {
        float4 nx[kAhead];
        load4(v0 + 32 * kAhead, nx);                     // the next 512 scores are on their way while these are placed
        const int ties_before = min(base_eq, ties);      // ties already emitted
        uint32_t gbits = 0, ebits = 0;                   // this lane's 16 scores: above / at the threshold
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
            if (v0 + kAhead * lane + u < vend) {
                const float x[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (above(x[j])) gbits |= 1u << (4 * u + j);
                    else if (equal(x[j])) ebits |= 1u << (4 * u + j);
                }
            }
        }
        const int mine = __popc(gbits) | (__popc(ebits) << 16);
        int incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += t;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        const int mgt = total & 0xffff, meq = total >> 16;
        int g_loc = (incl - mine) & 0xffff, q_loc = (incl - mine) >> 16;
        const int i0 = index_base + head + 4 * (v0 + kAhead * lane);
        if (meq == 0) {                                  // the common case: no score of these 512 equals the threshold
            const int shift = min(base_eq, ties) - ties_before;      // zero; kept for symmetry with the general case
            int* dst = stage + g_loc + shift;
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if ((gbits >> j) & 1) *dst++ = i0 + j;
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if ((gbits >> j) & 1) { stage[g_loc + min(base_eq + q_loc, ties) - ties_before] = i0 + j; ++g_loc; }
                else if ((ebits >> j) & 1) { if (base_eq + q_loc < ties) stage[g_loc + q_loc] = i0 + j; ++q_loc; }
            }
        }
        __syncwarp();
        const int count = mgt + min(base_eq + meq, ties) - ties_before;
        int* dst = out + base_gt + ties_before;
        for (int i = lane; i < count; i += 32) dst[i] = stage[i];
        __syncwarp();
        base_gt += mgt;
        base_eq += meq;
#pragma unroll
        for (int u = 0; u < kAhead; ++u) q[u] = nx[u];
    }
    if (warp == kWarps - 1 && lane == 0) {                // the tail follows the last stretch
        for (int i = tail_begin; i < n; ++i) {
            const uint32_t key = order_key(sc[i]);
            if (key > thr) out[base_gt + min(base_eq, ties)] = index_base + i;
            else if (key == thr && base_eq < ties) out[base_gt + base_eq] = index_base + i;
            base_gt += key > thr; base_eq += key == thr;
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
select_kernel(Plan p, const float* __restrict__ scores, int* __restrict__ idx_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SelectSmem& s = *reinterpret_cast<SelectSmem*>(smem_raw);
    pdl_trigger();
    const int unit = blockIdx.x;
    const int b = unit % p.batch, lh = unit / p.batch;
    const int n = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
    const int kk = p.cu_keep[b + 1] - p.cu_keep[b];
    pdl_wait();                                            // the scores are complete
    if (kk <= 0 || n <= 0) return;
    const float* sc = scores + (size_t)lh * p.total_tokens + p.cu_seqlens[b];
    int* out = idx_out + (size_t)lh * p.total_keep + p.cu_keep[b];
    if (kk >= n) {
        for (int i = threadIdx.x; i < n; i += kThreads) out[i] = i;
        return;
    }
    int ties = 0;
    uint32_t thr;
    if (threshold_with_counts(s, sc, n, kk, &thr, &ties)) {
        emit_ordered<true, true>(s, sc, n, thr, ties, out);
        return;
    }
    bool all_finite = false;
    thr = find_threshold(s, [&](auto f) { for_each_score(sc, n, f); }, sc, n, kk, &ties, &all_finite);
    if (all_finite) emit_ordered<true>(s, sc, n, thr, ties, out);
    else emit_ordered<false>(s, sc, n, thr, ties, out);
}

// ---- selection spread over several CTAs -----------------------------------------------------------
// Used where one CTA per score vector leaves most of the GPU idle: selection across the heads of a
// layer (Section 3.4's alternative: one threshold per layer and sequence over heads * n scores) and
// per-head selection of a few long sequences.  A "group" is what shares a threshold: a (layer,
// sequence) pair with all its heads, or one unit.  Every head's vector is cut into `parts` slices,
// one CTA each:
//   1. histogram: the group's value range from the first scores of its first head (every CTA arrives
//      at the same numbers), a value-linear histogram of the slice in shared memory, added into the
//      group's histogram in global memory;
//   2. candidates: every CTA finds the threshold bin in the finished histogram, appends the slice's
//      members of that bin as (key, head) pairs to the group's list and counts, per head, the scores in
//      higher bins;
//   3. finalize, one CTA per group: exact radix select among the candidates, per-head counts above
//      and at the threshold (ties go to the lower head first, then to the lower index), the heads'
//      offsets.  Groups whose scores defeat the histogram (non-finite values, no spread, an overfull
//      bin) are redone here by one CTA over all scores, as the single-CTA selection would;
//      it also turns the candidates into per-slice counts of scores above / at the threshold;
//   4. ordered emission of every slice at its offset.
// Per-group scratch words: histogram, range, candidate counter, flags, per-head counts.
constexpr int kStLo = kBins, kStScale = kBins + 1, kStCand = kBins + 2, kStFlags = kBins + 3, kStAbove = kBins + 4;
static_assert(kWarps == 32, "block-wide sums take one warp, one partial per lane");
static_assert(kStAbove + 64 <= kSelStateInts, "per-group scratch too small");
static_assert(kCand / 2 >= 64 * 64, "per-slice counts of a group live in the candidate array");

struct Slice {
    int part, unit, b, lh, layer, head;
    int group, hg, hi;         // group index, heads per group, this head's index inside the group
    int n, kk, begin, end;     // the slice is [begin, end) of the unit's n scores
    long long cand_begin;      // the group's candidate list
    int cand_cap;
};

__device__ __forceinline__ Slice decode_group(const Plan& p, const MultiSelect& m, int group) {
    Slice c;
    c.b = group % p.batch;
    const int outer = group / p.batch;
    c.group = group;
    c.hg = m.across ? p.heads : 1;
    c.layer = m.across ? outer : outer / p.heads;
    c.head = m.across ? 0 : outer % p.heads;
    c.lh = c.layer * p.heads + c.head;
    c.hi = 0;
    c.unit = c.lh * p.batch + c.b;
    c.n = p.cu_seqlens[c.b + 1] - p.cu_seqlens[c.b];
    c.kk = p.cu_keep[c.b + 1] - p.cu_keep[c.b];
    c.part = 0; c.begin = 0; c.end = c.n;
    c.cand_begin = (long long)outer * m.cand_per_outer + (long long)c.b * (kSelCandBase + 1) +
                   ((long long)c.hg * p.cu_seqlens[c.b]) / kSelCandDiv;
    c.cand_cap = kSelCandBase + (int)(((long long)c.hg * c.n) / kSelCandDiv);
    return c;
}

__device__ __forceinline__ Slice decode_slice(const Plan& p, const MultiSelect& m, int block) {
    const int part = block % m.parts, unit = block / m.parts;
    const int b = unit % p.batch, lh = unit / p.batch;
    const int layer = lh / p.heads, head = lh % p.heads;
    Slice c = decode_group(p, m, m.across ? layer * p.batch + b : unit);
    c.part = part; c.unit = unit; c.lh = lh; c.head = head;
    c.hi = m.across ? head : 0;
    const int len = (((c.n + m.parts - 1) / m.parts) + 3) & ~3;
    c.begin = min(c.n, part * len);
    c.end = min(c.n, c.begin + len);
    return c;
}

__global__ void __launch_bounds__(kThreads, 1)
multi_hist_kernel(Plan p, const float* __restrict__ scores, MultiSelect m) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SelectSmem& s = *reinterpret_cast<SelectSmem*>(smem_raw);
    pdl_trigger();
    const Slice c = decode_slice(p, m, blockIdx.x);
    if (c.kk <= 0 || c.n <= 0 || c.kk >= c.n) return;
    const int tid = threadIdx.x;
    int* st = m.state + (size_t)c.group * kSelStateInts;
    const float* first = scores + (size_t)(c.lh - c.hi) * p.total_tokens + p.cu_seqlens[c.b];   // the group's first head
    bool lopsided = false;
    compute_range(s, first, c.n, &lopsided);
    if (s.fallback) {
        if (tid == 0) atomicOr(&st[kStFlags], 1);
        return;
    }
    if (lopsided) narrow_range(s, first, min(c.n, kSample));
    const float lo = s.lo, scale = s.scale;
    if (c.part == 0 && c.hi == 0 && tid == 0) { st[kStLo] = __float_as_int(lo); st[kStScale] = __float_as_int(scale); }
    for (int i = tid; i < kBins; i += kThreads) s.hist[i] = 0;
    __syncthreads();
    int nonfinite = 0;
    for_each_score(first + (size_t)c.hi * p.total_tokens + c.begin, c.end - c.begin, [&](float v) {
        if (!isfinite(v)) nonfinite = 1;
        atomicAdd(&s.hist[bin_of(v, lo, scale)], 1);
    });
    const int any_nonfinite = __syncthreads_or(nonfinite);
    for (int i = tid; i < kBins; i += kThreads)
        if (s.hist[i] != 0) atomicAdd(&st[i], s.hist[i]);
    if (any_nonfinite && tid == 0) atomicOr(&st[kStFlags], 1);
}

__global__ void __launch_bounds__(kThreads, 1)
multi_candidates_kernel(Plan p, const float* __restrict__ scores, MultiSelect m) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SelectSmem& s = *reinterpret_cast<SelectSmem*>(smem_raw);
    pdl_trigger();
    const Slice c = decode_slice(p, m, blockIdx.x);
    pdl_wait();                                            // the groups' histograms are complete
    if (c.kk <= 0 || c.n <= 0 || c.kk >= c.n) return;
    const int tid = threadIdx.x, lane = tid & 31;
    int* st = m.state + (size_t)c.group * kSelStateInts;
    if ((st[kStFlags] & 1) != 0) return;                  // set by the histogram pass: the same for every CTA of the group
    const float lo = __int_as_float(st[kStLo]), scale = __int_as_float(st[kStScale]);
    for (int i = tid; i < kBins; i += kThreads) s.hist[i] = st[i];
    if (tid == 0) s.n_cand = 0;                           // here: the slice's scores in bins above the threshold bin
    __syncthreads();
    pick_bin(s, kBins, c.hg * c.kk);
    const int tbin = s.bin;
    if (s.hist[tbin] > c.cand_cap) {                      // every CTA of the group sees the same histogram
        if (tid == 0) atomicOr(&st[kStFlags], 2);
        return;
    }
    uint2* cand = m.cand + c.cand_begin;
    int above = 0;
    for_each_score(scores + (size_t)c.lh * p.total_tokens + p.cu_seqlens[c.b] + c.begin, c.end - c.begin, [&](float v) {
        const int bin = bin_of(v, lo, scale);
        above += bin > tbin;
        if (bin == tbin) {
            const int pos = atomicAdd(&st[kStCand], 1);
            if (pos < c.cand_cap) cand[pos] = make_uint2(order_key(v), (uint32_t)(c.hi * m.parts + c.part));
        }
    });
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) above += __shfl_xor_sync(0xffffffffu, above, d);
    if (lane == 0 && above != 0) atomicAdd(&s.n_cand, above);       // zeroed by pick_bin's caller below
    __syncthreads();
    if (tid == 0) {
        m.counts[blockIdx.x] = make_int2(s.n_cand, 0);
        if (s.n_cand != 0) atomicAdd(&st[kStAbove + c.hi], s.n_cand);
    }
}

// One CTA per group.  Writes the group's threshold key, every head's share of the ties and, when
// selecting across heads, the heads' offsets inside the sequence's block of the output.
__global__ void __launch_bounds__(kThreads, 1)
multi_finalize_kernel(Plan p, const float* __restrict__ scores, MultiSelect m, int* __restrict__ head_offsets) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SelectSmem& s = *reinterpret_cast<SelectSmem*>(smem_raw);
    __shared__ int head_gt[64], head_eq[64];
    pdl_trigger();
    const Slice c = decode_group(p, m, blockIdx.x);
    pdl_wait();                                            // the candidate lists are complete
    const int H = c.hg, n = c.n, kk = c.kk, tid = threadIdx.x;
    int* offs = head_offsets != nullptr ? head_offsets + (size_t)c.group * (H + 1) : nullptr;
    auto unit_of = [&](int h) { return (c.lh + h) * p.batch + c.b; };
    if (kk <= 0 || n <= 0) {
        if (offs != nullptr) for (int h = tid; h <= H; h += kThreads) offs[h] = 0;
        return;
    }
    if (kk >= n) {                                         // everything is kept
        if (offs != nullptr) for (int h = tid; h <= H; h += kThreads) offs[h] = h * n;
        for (int h = tid; h < H; h += kThreads) m.ties[unit_of(h)] = n;
        if (tid == 0) m.thr[c.group] = 0u;                 // every key is >= 0: all scores count as ties or above
        return;
    }
    int* st = m.state + (size_t)c.group * kSelStateInts;
    const float* base = scores + (size_t)c.lh * p.total_tokens + p.cu_seqlens[c.b];
    // scores above / at the threshold per slice of the group (head-major), so that a slice can be emitted on its own;
    // they live where the single-CTA route keeps its candidates (at most 64 heads x 64 slices)
    int* slice_gt = reinterpret_cast<int*>(s.cand);
    int* slice_eq = slice_gt + kCand / 2;
    const int n_slices = H * m.parts;
    const bool fast = st[kStFlags] == 0;
    int ties = 0;
    uint32_t thr;
    if (fast) {
        for (int i = tid; i < kBins; i += kThreads) s.hist[i] = st[i];
        for (int i = tid; i < n_slices; i += kThreads) { slice_gt[i] = 0; slice_eq[i] = 0; }
        __syncthreads();
        pick_bin(s, kBins, H * kk);
        const int want = s.remaining;
        const int nc = min(st[kStCand], c.cand_cap);
        const uint2* cand = m.cand + c.cand_begin;
        __syncthreads();
        thr = radix_select(s, want, &ties, [&](auto tally) {
            for (int i = tid; i < nc; i += kThreads) tally(cand[i].x);
        });
        for (int i = tid; i < nc; i += kThreads) {
            const uint2 e = cand[i];
            if (e.x > thr) atomicAdd(&slice_gt[e.y], 1);
            else if (e.x == thr) atomicAdd(&slice_eq[e.y], 1);
        }
        __syncthreads();
    } else {
        auto visit_all = [&](auto f) {
            for (int h = 0; h < H; ++h) for_each_score(base + (size_t)h * p.total_tokens, n, f);
        };
        thr = find_threshold(s, visit_all, base, n, H * kk, &ties);
        __syncthreads();
        for (int i = tid; i < n_slices; i += kThreads) { slice_gt[i] = 0; slice_eq[i] = 0; }
        __syncthreads();
        const int len = (((n + m.parts - 1) / m.parts) + 3) & ~3;
        for (int i = 0; i < n_slices; ++i) {
            const int h = i / m.parts, part = i % m.parts;
            const int begin = min(n, part * len), end = min(n, begin + len);
            int gt = 0, eq = 0;
            for_each_score(base + (size_t)h * p.total_tokens + begin, end - begin, [&](float v) {
                const uint32_t key = order_key(v);
                gt += key > thr; eq += key == thr;
            });
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                gt += __shfl_xor_sync(0xffffffffu, gt, d);
                eq += __shfl_xor_sync(0xffffffffu, eq, d);
            }
            if ((tid & 31) == 0) { atomicAdd(&slice_gt[i], gt); atomicAdd(&slice_eq[i], eq); }
        }
        __syncthreads();
    }
    for (int i = tid; i < n_slices; i += kThreads) {
        int2* dst = &m.counts[(size_t)unit_of(i / m.parts) * m.parts + i % m.parts];
        const int above = fast ? dst->x : 0;               // left there by the candidates pass
        *dst = make_int2(above + slice_gt[i], slice_eq[i]);
    }
    for (int h = tid; h < H; h += kThreads) {
        int gt = fast ? st[kStAbove + h] : 0, eq = 0;
        for (int q = 0; q < m.parts; ++q) { gt += slice_gt[h * m.parts + q]; eq += slice_eq[h * m.parts + q]; }
        head_gt[h] = gt; head_eq[h] = eq;
    }
    __syncthreads();
    if (tid == 0) {
        int left = ties, off = 0;
        for (int h = 0; h < H; ++h) {
            const int take = min(left, head_eq[h]);
            left -= take;
            m.ties[unit_of(h)] = take;
            if (offs != nullptr) offs[h] = off;
            off += head_gt[h] + take;
        }
        if (offs != nullptr) offs[H] = off;
        m.thr[c.group] = thr;
    }
}

// One CTA per slice: the slice's kept indices, ascending, at their place in the head's output.
__global__ void __launch_bounds__(kThreads, 1)
multi_emit_kernel(Plan p, const float* __restrict__ scores, MultiSelect m, const int* __restrict__ head_offsets,
                  int* __restrict__ idx_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SelectSmem& s = *reinterpret_cast<SelectSmem*>(smem_raw);
    pdl_trigger();
    const Slice c = decode_slice(p, m, blockIdx.x);
    pdl_wait();                                            // thresholds, offsets and slice counts are complete
    if (c.kk <= 0 || c.n <= 0) return;
    int* out;
    if (m.across) {
        const int* offs = head_offsets + (size_t)c.group * (p.heads + 1);
        if (offs[c.head + 1] - offs[c.head] <= 0) return;
        out = idx_out + (size_t)c.layer * p.heads * p.total_keep + (size_t)p.heads * p.cu_keep[c.b] + offs[c.head];
    } else {
        out = idx_out + (size_t)c.lh * p.total_keep + p.cu_keep[c.b];
    }
    if (c.kk >= c.n) {
        for (int i = c.begin + threadIdx.x; i < c.end; i += kThreads) out[i] = i;
        return;
    }
    int gt0 = 0, eq0 = 0;
    for (int q = 0; q < c.part; ++q) {
        const int2 v = m.counts[(size_t)c.unit * m.parts + q];
        gt0 += v.x; eq0 += v.y;
    }
    const float* sc = scores + (size_t)c.lh * p.total_tokens + p.cu_seqlens[c.b] + c.begin;
    const bool plain = m.state[(size_t)c.group * kSelStateInts + kStFlags] == 0;     // every score was seen and is finite
    if (plain) emit_ordered<true>(s, sc, c.end - c.begin, m.thr[c.group], m.ties[c.unit], out, c.begin, gt0, eq0);
    else emit_ordered<false>(s, sc, c.end - c.begin, m.thr[c.group], m.ties[c.unit], out, c.begin, gt0, eq0);
}

// Eq. 6: s = z(a) + lambda z(o), population standard deviation, per unit.  Overwrites the
// outlier scores in place.
__global__ void __launch_bounds__(kThreads, 1)
blend_kernel(Plan p, const float* __restrict__ attn, float lambda, float* __restrict__ scores) {
    __shared__ double red[4][kWarps];
    __shared__ double stats[4];
    pdl_trigger();
    pdl_wait();                                            // the leverage scores are complete
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
    // a term without spread contributes nothing; "without spread" is a standard deviation of at most 1e-3 of |mean|,
    // below what the scores resolve (the leverage scores of a sequence no longer than the sketch are all one)
    const double sd_a = sqrt(stats[2] / n), sd_o = sqrt(stats[3] / n);
    const double inv_a = sd_a > 1e-3 * fabs(mean_a) ? 1.0 / sd_a : 0.0;
    const double inv_o = sd_o > 1e-3 * fabs(mean_o) ? (double)lambda / sd_o : 0.0;
    for (int i = tid; i < n; i += kThreads)
        o[i] = (float)(((double)a[i] - mean_a) * inv_a + ((double)o[i] - mean_o) * inv_o);
}

// The blend for a few long units: every unit's vectors are cut into `parts` slices.  First kernel: mean and
// sum of squared deviations of a and o per slice; second kernel: every CTA merges its unit's slices in a
// fixed order (pairwise update of count, mean and squared deviations), then rewrites its own slice.
__device__ __forceinline__ void block_sum2(double x, double y, double (*red)[kWarps], double* out) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        x += __shfl_xor_sync(0xffffffffu, x, d);
        y += __shfl_xor_sync(0xffffffffu, y, d);
    }
    __syncthreads();                                      // earlier readers of red / out are done
    if (lane == 0) { red[0][warp] = x; red[1][warp] = y; }
    __syncthreads();
    if (warp == 0) {
        double u = red[0][lane], v = red[1][lane];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            u += __shfl_xor_sync(0xffffffffu, u, d);
            v += __shfl_xor_sync(0xffffffffu, v, d);
        }
        if (lane == 0) { out[0] = u; out[1] = v; }
    }
    __syncthreads();
}

__device__ __forceinline__ void blend_slice(int n, int parts, int part, int* begin, int* end) {
    const int len = (n + parts - 1) / parts;
    *begin = min(n, part * len);
    *end = min(n, *begin + len);
}

__global__ void __launch_bounds__(kThreads, 1)
blend_stats_kernel(Plan p, const float* __restrict__ attn, const float* __restrict__ scores, int parts,
                   double* __restrict__ stats) {
    __shared__ double red[2][kWarps];
    __shared__ double tot[2];
    pdl_trigger();
    pdl_wait();                                            // the leverage scores are complete
    const int part = blockIdx.x % parts, unit = blockIdx.x / parts;
    const int b = unit % p.batch, lh = unit / p.batch;
    const int n = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
    int begin, end;
    blend_slice(n, parts, part, &begin, &end);
    const int cnt = end - begin;
    double* out = stats + (size_t)blockIdx.x * 4;
    if (cnt <= 0) {
        if (threadIdx.x < 4) out[threadIdx.x] = 0.0;
        return;
    }
    const size_t off = (size_t)lh * p.total_tokens + p.cu_seqlens[b] + begin;
    const float* a = attn + off;
    const float* o = scores + off;
    double sa = 0.0, so = 0.0;
    for (int i = threadIdx.x; i < cnt; i += kThreads) { sa += (double)a[i]; so += (double)o[i]; }
    block_sum2(sa, so, red, tot);
    const double mean_a = tot[0] / cnt, mean_o = tot[1] / cnt;
    double va = 0.0, vo = 0.0;
    for (int i = threadIdx.x; i < cnt; i += kThreads) {
        const double da = (double)a[i] - mean_a, d_o = (double)o[i] - mean_o;
        va = fma(da, da, va); vo = fma(d_o, d_o, vo);
    }
    block_sum2(va, vo, red, tot);
    if (threadIdx.x == 0) { out[0] = mean_a; out[1] = tot[0]; out[2] = mean_o; out[3] = tot[1]; }
}

__global__ void __launch_bounds__(kThreads, 1)
blend_apply_kernel(Plan p, const float* __restrict__ attn, float lambda, float* __restrict__ scores, int parts,
                   const double* __restrict__ stats) {
    pdl_trigger();
    pdl_wait();                                            // the slices' statistics are complete
    const int part = blockIdx.x % parts, unit = blockIdx.x / parts;
    const int b = unit % p.batch, lh = unit / p.batch;
    const int n = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
    int begin, end;
    blend_slice(n, parts, part, &begin, &end);
    if (end <= begin) return;
    // every thread of every CTA of the unit merges the slices in the same order: the same statistics everywhere
    double cnt = 0.0, mean_a = 0.0, m2_a = 0.0, mean_o = 0.0, m2_o = 0.0;
    for (int q = 0; q < parts; ++q) {
        int qb, qe;
        blend_slice(n, parts, q, &qb, &qe);
        const double c = (double)(qe - qb);
        if (c <= 0.0) continue;
        const double* st = stats + ((size_t)unit * parts + q) * 4;
        const double tot = cnt + c;
        const double da = st[0] - mean_a, d_o = st[2] - mean_o;
        mean_a += da * (c / tot);  m2_a += st[1] + da * da * (cnt * c / tot);
        mean_o += d_o * (c / tot); m2_o += st[3] + d_o * d_o * (cnt * c / tot);
        cnt = tot;
    }
    const double sd_a = sqrt(m2_a / n), sd_o = sqrt(m2_o / n);
    const double inv_a = sd_a > 1e-3 * fabs(mean_a) ? 1.0 / sd_a : 0.0;          // as in blend_kernel
    const double inv_o = sd_o > 1e-3 * fabs(mean_o) ? (double)lambda / sd_o : 0.0;
    const size_t off = (size_t)lh * p.total_tokens + p.cu_seqlens[b];
    const float* a = attn + off;
    float* o = scores + off;
    for (int i = begin + threadIdx.x; i < end; i += kThreads)
        o[i] = (float)(((double)a[i] - mean_a) * inv_a + ((double)o[i] - mean_o) * inv_o);
}

}  // namespace

cudaError_t launch_select(const Plan& p, const float* scores, int* idx, cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    if (units == 0 || p.total_keep == 0) return cudaSuccess;
    const int smem = (int)sizeof(SelectSmem);
    cudaError_t e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = launch_chained(kPdlSelect, select_kernel, dim3(units), dim3(kThreads), smem, stream, p, scores, idx);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_select_multi(const Plan& p, const float* scores, int* idx, int* head_offsets, const MultiSelect& m,
                                cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    if (units == 0) return cudaSuccess;
    if (m.parts < 1 || (m.across && (p.heads > 64 || head_offsets == nullptr))) return cudaErrorInvalidValue;
    const int groups = m.across ? p.layers * p.batch : units;
    const int smem = (int)sizeof(SelectSmem);
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(multi_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(multi_candidates_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(multi_finalize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(multi_emit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(m.state, 0, sizeof(int) * (size_t)groups * kSelStateInts, stream)) != cudaSuccess) return e;
    const unsigned slices = (unsigned)units * (unsigned)m.parts;
    multi_hist_kernel<<<slices, kThreads, smem, stream>>>(p, scores, m);
    if ((e = launch_chained(kPdlOther, multi_candidates_kernel, dim3(slices), dim3(kThreads), smem, stream, p, scores, m)) != cudaSuccess) return e;
    if ((e = launch_chained(kPdlOther, multi_finalize_kernel, dim3(groups), dim3(kThreads), smem, stream, p, scores, m,
                            m.across ? head_offsets : (int*)nullptr)) != cudaSuccess) return e;
    if (p.total_keep > 0) {
        if ((e = launch_chained(kPdlOther, multi_emit_kernel, dim3(slices), dim3(kThreads), smem, stream, p, scores, m,
                                (const int*)head_offsets, idx)) != cudaSuccess) return e;
    }
    return cudaGetLastError();
}

cudaError_t launch_blend(const Plan& p, const float* attn, float lambda, float* scores, int parts, double* stats,
                         cudaStream_t stream) {
    const int units = p.layers * p.heads * p.batch;
    if (units == 0 || p.total_tokens == 0) return cudaSuccess;
    if (parts > 1 && stats != nullptr) {
        cudaError_t e = launch_chained(kPdlOther, blend_stats_kernel, dim3(units * parts), dim3(kThreads), 0, stream, p, attn,
                                       (const float*)scores, parts, stats);
        if (e != cudaSuccess) return e;
        e = launch_chained(kPdlOther, blend_apply_kernel, dim3(units * parts), dim3(kThreads), 0, stream, p, attn, lambda, scores, parts,
                           (const double*)stats);
        if (e != cudaSuccess) return e;
    } else {
        cudaError_t e = launch_chained(kPdlOther, blend_kernel, dim3(units), dim3(kThreads), 0, stream, p, attn, lambda, scores);
        if (e != cudaSuccess) return e;
    }
    return cudaGetLastError();
}

}  // namespace compactor

// Attention term of the score (Eq. 5): a = concat_i 1^T softmax(Q[i] K[i]^T) over chunks of 256
// consecutive tokens, no causal mask, summed over the query heads that share a KV head, then
// mean-pooled.  Readings where the paper is silent: logits are multiplied by a caller-given scale,
// the last, shorter chunk is a softmax over its own keys, pooling is a centred window with zero
// padding.
//
// Work item = one chunk of one layer and KV head; persistent CTAs (one per SM) walk the items.  Warp 0
// loads an item's keys once and streams the query heads' rows in halves of 128 through a two-slot ring
// (TMA, 128-byte swizzle).  One thread of warp 1 issues, per half, S = Q_half K^T (tcgen05.mma,
// 128 x 256 fp32) into one of two accumulators in tensor memory, so that the products of the next half
// run beside the softmax of the current one.  Warps 2-17 share the 128 query rows (four warps per
// 32 rows, 64 keys each): row maximum, e = 2^(scale log2e (s - max)) written as fp16 into shared memory
// in the layout of an MN-major operand, and the reciprocal of the row sum (two fp16 terms) into rows 0
// and 1 of a small K-major operand w.  A second MMA, E^T w (keys x 2: the half's normalised column
// sums), lands in 32 columns of the half's own S accumulator once the softmax warps are done with S; two
// warps of each four add the sums of 128 keys each to a register per thread and write them at the end of
// the item.  The exponential phase runs at about 12 of the 16 exponentials per clock an SM can do, with the
// issue slots and the half-rate integer pipe close to their limits as well (moving a share of the
// exponentials to a polynomial on the FMA pipe made it slower): hence packed fp32x2 arithmetic,
// three-input maxima, tensor-memory loads one step ahead, four warps per scheduler, and the first
// exponentials of a half computed before the wait for the E buffer.
#include <cuda_fp16.h>

#include "common.cuh"
#include "sm100.cuh"

namespace compactor {
namespace {

using namespace sm100;

constexpr int kChunk = 256;
constexpr int kHalf = 128;
constexpr int kSplitDefault = 4;
constexpr int kMaxSplit = 4;               // softmax warps per query row quadrant (each takes 256 / split keys): 2 or 4
constexpr int kKBox = kChunk * 128;        // 64 channels x 256 tokens x 2 B
constexpr int kQBox = kHalf * 128;         // 64 channels x 128 rows
constexpr int kPBlock = kHalf * 128;       // 128 rows x 64 keys, fp16
constexpr int kWBox = 64 * 128;            // 64 rows x 64 k, fp16
constexpr uint32_t kTmemCols = 512;        // two S accumulators of 256 columns; a half's column sums reuse 32 columns of its own

struct __align__(1024) AttnSmem {
    unsigned char k[2 * kKBox];
    unsigned char q[2][2 * kQBox];
    unsigned char p[4 * kPBlock];
    unsigned char w[2 * kWBox];
    uint64_t k_full, k_empty, q_full[2], q_empty[2];
    uint64_t s_full[2];        // S of a half is in accumulator (half & 1)
    uint64_t p_ready;          // E and the weights of a half are in shared memory, its S is consumed
    uint64_t c_full[2];        // the half's column sums are in its accumulator; E and the weights may be overwritten
    uint64_t drained[2];       // the column sums have been taken out: the accumulator may be overwritten
    float xmax[kMaxSplit][kHalf];   // row maxima / row sums of the key ranges, exchanged between the warps of a quadrant
    float xsum[kMaxSplit][kHalf];
    uint32_t tmem_base;
    int abort;
    int abort_mma;             // set by the MMA warp alone, before it wakes the softmax warps: they all see the same value
};

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Two fp32 values per instruction (the softmax warps are bound by instruction issue).
__device__ __forceinline__ uint64_t pack2(float a, float b) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
template <int kSplit>
__device__ __forceinline__ void softmax_quad_sync(int q) {     // the warps that share 32 query rows
    asm volatile("bar.sync %0, %1;" :: "r"(q + 1), "n"(32 * kSplit) : "memory");
}

// Where a work item (one chunk of one layer and KV head) lies.
struct AttnItem { int layer, head, lh, b, tok_begin, n_tok; };
__device__ __forceinline__ AttnItem attn_item(const Plan& p, int item) {
    AttnItem a;
    a.lh = item / p.total_chunks;
    const int chunk_id = item % p.total_chunks;
    a.layer = a.lh / p.heads; a.head = a.lh % p.heads;
    const int b = find_segment(p.cu_chunks, p.batch, chunk_id);
    a.b = b;
    a.tok_begin = p.cu_seqlens[b] + (chunk_id - p.cu_chunks[b]) * kChunk;
    a.n_tok = min(kChunk, p.cu_seqlens[b + 1] - a.tok_begin);
    return a;
}

// Persistent: CTA c takes items c, c + grid, ...; barriers, tensor memory and the zeroed weight operand are set
// up once.  Halves are numbered through all of a CTA's items (g), which fixes every barrier's phase.
template <int kSplit>
__global__ void __launch_bounds__(64 + 128 * kSplit, 1)
attention_kernel(Plan p, const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap,
                 int q_per_kv, float scale_log2e, int n_items, float* __restrict__ out, int* __restrict__ status) {
    extern __shared__ unsigned char smem_raw[];
    AttnSmem& s = *reinterpret_cast<AttnSmem*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    constexpr int kSoftmaxWarps = 4 * kSplit;
    constexpr int kThreads = 64 + 32 * kSoftmaxWarps;
    constexpr int kCols = kChunk / kSplit;             // keys per softmax warp
    constexpr int kStep = kCols / 4;                   // columns per tensor-memory load: 32 or 16
    const int n_iter = 2 * q_per_kv;                   // halves of 128 query rows per item (even)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int my_items = ((int)blockIdx.x < n_items) ? (n_items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

    if (threadIdx.x == 0) {
        prefetch_tensormap(&qmap);
        prefetch_tensormap(&kmap);
        mbar_init(&s.k_full, 1);
        mbar_init(&s.k_empty, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(&s.q_full[i], 1); mbar_init(&s.q_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&s.s_full[i], 1); mbar_init(&s.c_full[i], 1); mbar_init(&s.drained[i], 8); }
        mbar_init(&s.p_ready, 32 * kSoftmaxWarps);
        s.abort = 0;
        s.abort_mma = 0;
        fence_barrier_init();
    }
    for (int i = threadIdx.x; i < 2 * kWBox / 16; i += kThreads)       // rows 2.. of the weight operand stay zero
        reinterpret_cast<uint4*>(s.w)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    if (warp == 1) { tmem_alloc(&s.tmem_base, kTmemCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = s.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            for (int r = 0; r < my_items && ok; ++r) {
                const AttnItem a = attn_item(p, blockIdx.x + r * gridDim.x);
                if (r > 0 && !mbar_wait(&s.k_empty, (r - 1) & 1)) { s.abort = 1; break; }   // the previous item's S products are done
                mbar_arrive_expect_tx(&s.k_full, 2 * kKBox);
                tma_load_4d(s.k, &kmap, &s.k_full, 0, a.tok_begin, a.head, a.layer);
                tma_load_4d(s.k + kKBox, &kmap, &s.k_full, 64, a.tok_begin, a.head, a.layer);
                for (int it = 0; it < n_iter; ++it) {
                    const int g = r * n_iter + it, st = g & 1, use = g >> 1;
                    if (use > 0 && !mbar_wait(&s.q_empty[st], (use - 1) & 1)) { s.abort = 1; ok = false; break; }
                    if (*(volatile int*)&s.abort) { ok = false; break; }
                    mbar_arrive_expect_tx(&s.q_full[st], 2 * kQBox);
                    const int qhead = a.head * q_per_kv + (it >> 1);
                    const int row = a.tok_begin + (it & 1) * kHalf;
                    tma_load_4d(s.q[st], &qmap, &s.q_full[st], 0, row, qhead, a.layer);
                    tma_load_4d(s.q[st] + kQBox, &qmap, &s.q_full[st], 64, row, qhead, a.layer);
                }
            }
        }
    } else if (warp == 1) {
        constexpr uint32_t idesc_s = umma_idesc_16bit(1, 128, kChunk, 0, 0);     // bf16: Q (K-major) x K^T (K-major)
        constexpr uint32_t idesc_c = umma_idesc_16bit(0, 128, 16, 1, 0);         // fp16: E^T (MN-major: keys x rows) x w (K-major)
        const uint32_t k_base = smem_u32(s.k), p_base = smem_u32(s.p), w_base = smem_u32(s.w);
        // Column sums of half g: D[key][0..1] = sum_rows E[row][key] * (hi, lo of 1 / row sum), keys 0-127 in
        // columns 0-15 and keys 128-255 in columns 16-31 of the half's own accumulator, whose S is consumed.
        auto column_sums = [&](int g) {
            const uint32_t d = tmem + (uint32_t)(g & 1) * 256;
#pragma unroll
            for (int kh = 0; kh < 2; ++kh)
#pragma unroll
                for (int ks = 0; ks < kHalf / 16; ++ks) {
                    const uint64_t a_desc = umma_desc_sw128(p_base + kh * 2 * kPBlock + ks * 2048, kPBlock, 1024);
                    const uint64_t b_desc = umma_desc_sw128(w_base + (ks >> 2) * kWBox + (ks & 3) * 32, 16, 1024);
                    umma_bf16(d + kh * 16, a_desc, b_desc, idesc_c, ks > 0);
                }
        };
        const int n_halves = my_items * n_iter;
        bool ok = true;
        for (int g = 0, r = 0, it = 0; g < n_halves && ok; ++g, it = (it + 1 == n_iter) ? 0 : it + 1, r += (it == 0)) {
            const int st = g & 1, use = g >> 1;
            if (it == 0) ok = mbar_wait(&s.k_full, r & 1);
            if (ok) ok = mbar_wait(&s.q_full[st], use & 1);
            if (ok && g >= 2) ok = mbar_wait(&s.drained[st], (use - 1) & 1);   // the accumulator's previous column sums are out
            ok = ok && !*(volatile int*)&s.abort;
            if (!ok) break;
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t q_base = smem_u32(s.q[st]);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t a_desc = umma_desc_sw128(q_base + (ks >> 2) * kQBox + (ks & 3) * 32, 16, 1024);
                    const uint64_t b_desc = umma_desc_sw128(k_base + (ks >> 2) * kKBox + (ks & 3) * 32, 16, 1024);
                    umma_bf16(tmem + (uint32_t)st * 256, a_desc, b_desc, idesc_s, ks > 0);
                }
                umma_commit(&s.q_empty[st]);
                umma_commit(&s.s_full[st]);
                if (it == n_iter - 1) umma_commit(&s.k_empty);                // the item's keys are no longer needed
            }
            __syncwarp();
            if (g > 0) {                                    // the previous half's softmax ran beside the products above
                ok = mbar_wait(&s.p_ready, (g - 1) & 1);
                if (!ok) break;
                tc_fence_after_sync();
                if (lane == 0) { column_sums(g - 1); umma_commit(&s.c_full[(g - 1) & 1]); }
                __syncwarp();
            }
        }
        if (ok && n_halves > 0) ok = mbar_wait(&s.p_ready, (n_halves - 1) & 1);
        if (ok) {
            if (n_halves > 0) {
                tc_fence_after_sync();
                if (lane == 0) { column_sums(n_halves - 1); umma_commit(&s.c_full[(n_halves - 1) & 1]); }
                __syncwarp();
            }
        } else {
            s.abort = 1;
            s.abort_mma = 1;
            __threadfence_block();
            __syncwarp();
            if (lane == 0)                                  // wake the other warps
                for (int i = 0; i < 2; ++i) { mbar_arrive(&s.s_full[i]); mbar_arrive(&s.c_full[i]); }
        }
    } else {
        const int q = warp & 3;                              // TMEM lane quadrant
        const int ch = (warp - 2) >> 2;                      // which kCols of the 256 keys
        const int row = q * 32 + lane;                       // query row within the half = TMEM lane
        const uint32_t quad_addr = tmem + ((uint32_t)(q * 32) << 16);
        float col = 0.f;                                     // column sum of key ch * 128 + `row` (TMEM lane = key here)
        // the sums of keys 0-127 and 128-255 lie in columns 0-15 and 16-31: the quadrant's first two warps take one each
        auto take_column_sums = [&](int g) {
            if (ch < 2) {
                uint32_t c[2];
                tmem_ld_32x32b_x2(quad_addr + (uint32_t)(g & 1) * 256 + ch * 16, c);
                tmem_ld_wait();
                col += __uint_as_float(c[0]) + __uint_as_float(c[1]);    // hi and lo weights
            }
        };
        auto write_result = [&](const AttnItem& a) {         // an item's column sums are complete
            float* dst = out + (size_t)a.lh * p.total_tokens + a.tok_begin;
            if (ch < 2 && ch * kHalf + row < a.n_tok) dst[ch * kHalf + row] = col;
            col = 0.f;
        };
        const int n_halves = my_items * n_iter;
        AttnItem cur = attn_item(p, blockIdx.x), prev = cur;
        // A wait that gives up raises the abort flag; from then on no softmax thread waits any more, and all of them
        // keep the same control flow (so nobody is left alone at a named barrier); the results are then garbage
        // and the unit is flagged.
        auto wait_ft = [&](uint64_t* bar, uint32_t parity) {
            if (*(volatile int*)&s.abort || *(volatile int*)&s.abort_mma) return;
            if (!mbar_wait(bar, parity)) s.abort = 1;
        };
        for (int g = 0, r = 0, it = 0; g < n_halves; ++g, it = (it + 1 == n_iter) ? 0 : it + 1, r += (it == 0)) {
            if (it == 0 && r > 0) { prev = cur; cur = attn_item(p, blockIdx.x + r * gridDim.x); }
            const int n_tok = cur.n_tok;
            const bool full = n_tok == kChunk;               // only the last chunk of a sequence needs masks
            wait_ft(&s.s_full[g & 1], (g >> 1) & 1);
            tc_fence_after_sync();
            const uint32_t lane_addr = quad_addr + (uint32_t)(g & 1) * 256 + ch * kCols;
            const bool row_valid = (it & 1) * kHalf + row < n_tok;
            // the load of the next 32 columns is in flight while this thread works on the current ones
            uint32_t ra[kStep], rb[kStep];
            float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            auto max_of = [&](const uint32_t (&x)[kStep], int c0) {
                if (full) {
#pragma unroll
                    for (int i = 0; i < kStep; i += 2)
                        m4[(i >> 1) & 3] = max3(m4[(i >> 1) & 3], __uint_as_float(x[i]), __uint_as_float(x[i + 1]));
                } else {
#pragma unroll
                    for (int i = 0; i < kStep; ++i)
                        if (ch * kCols + c0 + i < n_tok) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(x[i]));
                }
            };
            tmem_ld_cols(lane_addr, ra);
            tmem_ld_wait_for(ra);
            tmem_ld_cols(lane_addr + kStep, rb);
            max_of(ra, 0);
            tmem_ld_wait_for(rb);
            tmem_ld_cols(lane_addr + 2 * kStep, ra);
            max_of(rb, kStep);
            tmem_ld_wait_for(ra);
            tmem_ld_cols(lane_addr + 3 * kStep, rb);
            max_of(ra, 2 * kStep);
            tmem_ld_wait_for(rb);
            max_of(rb, 3 * kStep);
            s.xmax[ch][row] = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
            softmax_quad_sync<kSplit>(q);
            float mx = fmaxf(s.xmax[0][row], s.xmax[1][row]);            // finite: key 0 of the chunk always exists
            if (kSplit == 4) mx = fmaxf(mx, fmaxf(s.xmax[2][row], s.xmax[3][row]));
            const float bias = -mx * scale_log2e;
            uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};     // four pairs of partial row sums
            const uint64_t scale2 = pack2(scale_log2e, scale_log2e), bias2 = pack2(bias, bias);
            uint32_t packed[kStep / 2];
            auto exp_of = [&](const uint32_t (&r)[kStep], int c0) {
#pragma unroll
                for (int i = 0; i < kStep; i += 2) {
                    float y0, y1;
                    unpack2(fma2(pack2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), scale2, bias2), y0, y1);
                    float e0 = ex2_approx(y0), e1 = ex2_approx(y1);
                    if (!full) {
                        if (!row_valid || ch * kCols + c0 + i >= n_tok) e0 = 0.f;
                        if (!row_valid || ch * kCols + c0 + i + 1 >= n_tok) e1 = 0.f;
                    }
                    sum2[(i >> 1) & 3] = add2(sum2[(i >> 1) & 3], pack2(e0, e1));
                    const __half2 h = __floats2half2_rn(e0, e1);
                    packed[i >> 1] = *reinterpret_cast<const uint32_t*>(&h);
                }
            };
            auto store = [&](int c0) {
                const int col = ch * kCols + c0;
                unsigned char* blk = s.p + (col >> 6) * kPBlock + row * 128;
#pragma unroll
                for (int j = 0; j < kStep / 8; ++j) {
                    const int piece = ((col & 63) >> 3) + j;
                    *reinterpret_cast<uint4*>(blk + ((piece ^ (row & 7)) << 4)) =
                        make_uint4(packed[4 * j], packed[4 * j + 1], packed[4 * j + 2], packed[4 * j + 3]);
                }
            };
            tmem_ld_cols(lane_addr, ra);
            tmem_ld_wait_for(ra);
            tmem_ld_cols(lane_addr + kStep, rb);
            exp_of(ra, 0);                                   // the first exponentials need no room in shared memory yet
            if (g > 0) {
                // E and the weights of the previous half have been multiplied: they may be overwritten,
                // and its column sums are waiting in its accumulator
                wait_ft(&s.c_full[(g - 1) & 1], ((g - 1) >> 1) & 1);
                tc_fence_after_sync();
                take_column_sums(g - 1);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0 && ch < 2) mbar_arrive(&s.drained[(g - 1) & 1]);
                if (it == 0) write_result(prev);             // that was the last half of the previous item
            }
            store(0);
            tmem_ld_wait_for(rb);
            tmem_ld_cols(lane_addr + 2 * kStep, ra);
            exp_of(rb, kStep);
            store(kStep);
            tmem_ld_wait_for(ra);
            tmem_ld_cols(lane_addr + 3 * kStep, rb);
            exp_of(ra, 2 * kStep);
            store(2 * kStep);
            tmem_ld_wait_for(rb);
            exp_of(rb, 3 * kStep);
            store(3 * kStep);
            {
                float lo, hi;
                unpack2(add2(add2(sum2[0], sum2[1]), add2(sum2[2], sum2[3])), lo, hi);
                s.xsum[ch][row] = lo + hi;
            }
            softmax_quad_sync<kSplit>(q);
            if (ch == 0) {
                // 1 / (row sum) as two fp16 terms in rows 0 and 1 of the weight operand (row 1 is swizzled by its index)
                float sum = s.xsum[0][row] + s.xsum[1][row];
                if (kSplit == 4) sum += s.xsum[2][row] + s.xsum[3][row];
                const float wgt = (row_valid && sum > 0.f) ? 1.0f / sum : 0.f;
                const __half w_hi = __float2half_rn(wgt);
                const __half w_lo = __float2half_rn(wgt - __half2float(w_hi));
                unsigned char* wbox = s.w + (row >> 6) * kWBox;
                const int piece = (row & 63) >> 3, within = (row & 7) * 2;
                *reinterpret_cast<__half*>(wbox + (piece << 4) + within) = w_hi;
                *reinterpret_cast<__half*>(wbox + 128 + ((piece ^ 1) << 4) + within) = w_lo;
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&s.p_ready);
        }
        if (n_halves > 0) {                       // the last half's column sums, then the last item's result
            const int last = n_halves - 1;
            wait_ft(&s.c_full[last & 1], (last >> 1) & 1);
            tc_fence_after_sync();
            take_column_sums(last);
            write_result(cur);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
    if (threadIdx.x == 0 && (s.abort || s.abort_mma) && status != nullptr && my_items > 0) {
        // a bounded wait ran out: flag every unit this CTA worked on
        for (int r = 0; r < my_items; ++r) {
            const AttnItem it = attn_item(p, blockIdx.x + r * gridDim.x);
            atomicOr(&status[it.lh * p.batch + it.b], COMPACTOR_STATUS_TIMEOUT);
        }
    }
}

// Centred mean over `pool` tokens inside each sequence, zero beyond its ends.
__global__ void pool_kernel(Plan p, const float* __restrict__ raw, float* __restrict__ out, int pool) {
    const int lh = blockIdx.y;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.total_tokens) return;
    const int b = find_segment(p.cu_seqlens, p.batch, i);
    const int lo = p.cu_seqlens[b], hi = p.cu_seqlens[b + 1];
    const float* src = raw + (size_t)lh * p.total_tokens;
    const int half = pool / 2;
    float acc = 0.f;
    for (int j = max(lo, i - half); j <= min(hi - 1, i + half); ++j) acc += src[j];
    out[(size_t)lh * p.total_tokens + i] = acc / (float)pool;
}

}  // namespace

cudaError_t launch_attention(const Plan& p, const Mat& q, const Mat& k, int q_per_kv, float scale, int pool,
                             float* raw, float* out, int* status, cudaStream_t stream) {
    if (p.total_chunks == 0) return cudaSuccess;
    CUtensorMap qmap, kmap;
    if (!make_kv_tensor_map(&qmap, q.ptr, p.layers, p.heads * q_per_kv, p.total_tokens, q.stride_layer, q.stride_head,
                            q.stride_token, kHalf) ||
        !make_kv_tensor_map(&kmap, k.ptr, p.layers, p.heads, p.total_tokens, k.stride_layer, k.stride_head,
                            k.stride_token, kChunk))
        return cudaErrorInvalidValue;
    const int smem = (int)sizeof(AttnSmem) + 1024;
    float* dst = pool > 1 ? raw : out;
    const long long n_items = (long long)p.total_chunks * p.layers * p.heads;
    if (n_items > 0x7fffffffLL) return cudaErrorInvalidValue;
    int dev = 0, n_sm = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    const int grid = (int)(n_items < n_sm ? n_items : n_sm);          // one CTA per SM (shared memory)
    cudaError_t e = cudaFuncSetAttribute(attention_kernel<kSplitDefault>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    attention_kernel<kSplitDefault><<<grid, 64 + 128 * kSplitDefault, smem, stream>>>(
        p, qmap, kmap, q_per_kv, scale * 1.4426950408889634f, (int)n_items, dst, status);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    e = cudaGetLastError();
    if (e != cudaSuccess || pool <= 1) return e;
    pool_kernel<<<dim3((p.total_tokens + 255) / 256, p.layers * p.heads), 256, 0, stream>>>(p, raw, out, pool);
    return cudaGetLastError();
}

}  // namespace compactor

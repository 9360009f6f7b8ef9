// Scoring pass (Algorithm 1, lines 5-6, fused): o_i = || k_i W ||^2 with W = Phi L^-T from the
// factor kernel, so that U~ = K^ V~ Sigma~^-1 is never stored.  W arrives as two bf16 terms
// (hi + lo); both are multiplied with the bf16 keys on the tensor cores and added in fp32.
//
// One CTA per block of tokens of one unit, one CTA per SM.  Warp 0 streams 128-token tiles of K
// (and W once) through a six-stage ring with TMA; one thread of warp 1 issues tcgen05.mma (A = key
// tile, K-major; B = the rows of W_hi on top of the rows of W_lo, K-major: one MMA per k-step, so
// the key tile is fetched from shared memory once; D = 128 tokens x 2 MP fp32 in tensor memory,
// four accumulators in rotation); warps 2-5 read D back, add the two halves, square, sum along the
// row and park the scores of eight tiles in shared memory, from where they leave in 4 KB bursts.
// Sketches wider than 64 columns keep the two terms as separate MMAs into one accumulator.
#include "common.cuh"
#include "sm100.cuh"

namespace compactor {
namespace {

using namespace sm100;

constexpr int kTile = 128;
// Ring depth: six 32 KB stages, four when the W operand of a 128-column sketch takes 64 KB.
template <int MP> struct Stages { static constexpr int value = MP <= 64 ? 6 : 4; };
constexpr int kBoxBytes = kTile * 128;
constexpr int kTileBytes = 2 * kBoxBytes;
constexpr int kThreads = 192;
// Tiles whose scores are stored together (4 KB bursts instead of 512 B); at MP = 64 the W operand
// leaves no shared memory for that.
template <int MP> struct OutTiles { static constexpr int value = MP <= 48 ? 8 : 1; };
constexpr int kBufs = 4;                  // accumulators in rotation
// Up to 64 sketch columns the two bf16 terms of W are one operand of 2 MP rows (hi on top of lo): one MMA per
// k-step reads the key tile once and leaves k W_hi in columns [0, MP) and k W_lo in [MP, 2 MP) of the accumulator.
template <int MP> struct Fused { static constexpr bool value = MP <= 64; };
template <int MP> struct BufCols {                        // tensor-memory columns per accumulator (a power of two)
    static constexpr uint32_t value = MP <= 16 ? 32 : (MP <= 32 ? 64 : 128);
};

template <int MP>
struct __align__(1024) ScoreSmem {
    static constexpr int kStages = Stages<MP>::value;
    unsigned char tiles[kStages][kTileBytes];
    unsigned char w[2][2][MP * 128];      // fused: [channel half][term][MP rows x 64 channels]; else [term][channel half][...]
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t w_full;
    uint64_t d_full[kBufs];
    uint64_t d_empty[kBufs];
    float obuf[2][OutTiles<MP>::value * kTile];     // scores of a group of tiles, written to global memory in one burst
    uint32_t tmem_base;
    int abort;
    int abort_mma;                        // set by the MMA warp alone before it wakes the epilogue: seen alike by all its threads
};

template <int MP>
__global__ void __launch_bounds__(kThreads, 1)
score_kernel(Plan p, const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap wmap,
             float* __restrict__ scores, int* __restrict__ status, int chained, int tiny_done) {
    extern __shared__ unsigned char smem_raw[];
    using Smem = ScoreSmem<MP>;
    constexpr int kStages = Smem::kStages;
    constexpr uint32_t kCols = BufCols<MP>::value;
    constexpr uint32_t kTmemCols = kCols * kBufs;
    Smem& s = *reinterpret_cast<Smem*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    pdl_trigger();
    const int chunk_id = blockIdx.x;
    const int lh = blockIdx.y;
    const int layer = lh / p.heads, head = lh % p.heads;
    const int b = find_segment(p.cu_schunks, p.batch, chunk_id);
    const int tok_begin = p.cu_seqlens[b] + (chunk_id - p.cu_schunks[b]) * p.schunk;
    const int tok_end = min(tok_begin + p.schunk, p.cu_seqlens[b + 1]);
    const int n_tok = tok_end - tok_begin;
    const int n_tiles = (n_tok + kTile - 1) / kTile;
    const int unit = lh * p.batch + b;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // a unit about as short as the sketch is wide has been scored in fp64 by the factor kernel (W in two bf16 terms
    // is too coarse for its nearly singular G).  In a chained launch this grid must not be complete before the factor
    // kernel is: what follows waits for this grid alone.
    if (tiny_done && p.cu_seqlens[b + 1] - p.cu_seqlens[b] <= p.m + kTinyExtra) {
        pdl_wait();
        return;
    }

    if (threadIdx.x == 0) {
        prefetch_tensormap(&kmap);
        prefetch_tensormap(&wmap);
        for (int i = 0; i < kStages; ++i) { mbar_init(&s.full[i], 1); mbar_init(&s.empty[i], 1); }
        mbar_init(&s.w_full, 1);
        for (int i = 0; i < kBufs; ++i) { mbar_init(&s.d_full[i], 1); mbar_init(&s.d_empty[i], 4); }
        s.abort = 0;
        s.abort_mma = 0;
        fence_barrier_init();
    }
    if (warp == 1) { tmem_alloc(&s.tmem_base, kTmemCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = s.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            // In a chained launch the first key tiles, which come from the caller, are fetched at once and W, which is the
            // factor stage's, waits for it; otherwise W goes first (the first product needs it) and the tiles follow.
            int t = 0;
            for (; chained && t < n_tiles && t < kStages; ++t) {
                mbar_arrive_expect_tx(&s.full[t], kTileBytes);
                const int tok = tok_begin + t * kTile;
                tma_load_4d(s.tiles[t], &kmap, &s.full[t], 0, tok, head, layer);
                tma_load_4d(s.tiles[t] + kBoxBytes, &kmap, &s.full[t], 64, tok, head, layer);
            }
            pdl_wait();
            mbar_arrive_expect_tx(&s.w_full, 4 * MP * 128);
#pragma unroll
            for (int term = 0; term < 2; ++term)
#pragma unroll
                for (int half = 0; half < 2; ++half)
                    tma_load_2d(Fused<MP>::value ? s.w[half][term] : s.w[term][half], &wmap, &s.w_full, half * 64,
                                (unit * 2 + term) * MP);
            for (; t < n_tiles; ++t) {
                const int stage = t % kStages, round = t / kStages;
                if (round > 0 && !mbar_wait(&s.empty[stage], (round - 1) & 1)) { s.abort = 1; break; }
                if (*(volatile int*)&s.abort) break;
                mbar_arrive_expect_tx(&s.full[stage], kTileBytes);
                const int tok = tok_begin + t * kTile;
                tma_load_4d(s.tiles[stage], &kmap, &s.full[stage], 0, tok, head, layer);
                tma_load_4d(s.tiles[stage] + kBoxBytes, &kmap, &s.full[stage], 64, tok, head, layer);
            }
        }
    } else if (warp == 1) {
        constexpr uint32_t idesc = umma_idesc_bf16(128, Fused<MP>::value ? 2 * MP : MP, 0, 0);
        bool ok = mbar_wait(&s.w_full, 0);
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int stage = t % kStages, round = t / kStages;
            const int buf = t % kBufs, use = t / kBufs;
            ok = mbar_wait(&s.full[stage], round & 1);
            if (ok && use > 0) ok = mbar_wait(&s.d_empty[buf], (use - 1) & 1);
            ok = ok && !*(volatile int*)&s.abort;
            if (!ok) break;
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t a_base = smem_u32(s.tiles[stage]);
                const uint32_t d_addr = tmem + buf * kCols;
                if constexpr (Fused<MP>::value) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const int half = ks >> 2, off = (ks & 3) * 32;
                        const uint64_t a_desc = umma_desc_sw128(a_base + half * kBoxBytes + off, 16, 1024);
                        const uint64_t b_desc = umma_desc_sw128(smem_u32(s.w[half][0]) + off, 16, 1024);
                        umma_bf16(d_addr, a_desc, b_desc, idesc, ks > 0);
                    }
                } else {
#pragma unroll
                    for (int term = 0; term < 2; ++term)
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const int half = ks >> 2, off = (ks & 3) * 32;
                            const uint64_t a_desc = umma_desc_sw128(a_base + half * kBoxBytes + off, 16, 1024);
                            const uint64_t b_desc = umma_desc_sw128(smem_u32(s.w[term][half]) + off, 16, 1024);
                            umma_bf16(d_addr, a_desc, b_desc, idesc, (term > 0) || (ks > 0));
                        }
                }
                umma_commit(&s.empty[stage]);
                umma_commit(&s.d_full[buf]);
            }
            __syncwarp();
        }
        if (!ok) {
            s.abort = 1;
            s.abort_mma = 1;
            __threadfence_block();
            __syncwarp();
            if (lane == 0)
                for (int i = 0; i < kBufs; ++i) mbar_arrive(&s.d_full[i]);   // wake the epilogue
        }
    } else {
        const int q = warp & 3;
        float* out = scores + (size_t)lh * p.total_tokens + tok_begin;
        constexpr int kOutTiles = OutTiles<MP>::value;
        const int et = threadIdx.x - 64;                     // 0..127 among the epilogue threads
        for (int t = 0; t < n_tiles; ++t) {
            const int buf = t % kBufs, use = t / kBufs;
            // A wait that gives up raises the abort flag; after that no epilogue thread waits any more, and all of
            // them keep walking the tiles (so that nobody is left alone at the named barrier below): the scores
            // of the unit are then garbage and the unit is flagged.
            if (!*(volatile int*)&s.abort && !*(volatile int*)&s.abort_mma && !mbar_wait(&s.d_full[buf], use & 1)) s.abort = 1;
            tc_fence_after_sync();
            // all loads of a group are issued before the one wait: their latencies overlap
            const uint32_t d_row = tmem + ((uint32_t)(q * 32) << 16) + buf * kCols;
            float acc4[4] = {0.f, 0.f, 0.f, 0.f};
            if constexpr (Fused<MP>::value) {
                uint32_t hi[MP / 16][16], lo[MP / 16][16];
#pragma unroll
                for (int c = 0; c < MP / 16; ++c) {
                    tmem_ld_32x32b_x16(d_row + c * 16, hi[c]);
                    tmem_ld_32x32b_x16(d_row + MP + c * 16, lo[c]);
                }
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < MP / 16; ++c)
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float v = __uint_as_float(hi[c][i]) + __uint_as_float(lo[c][i]);
                        acc4[i & 3] = fmaf(v, v, acc4[i & 3]);
                    }
            } else {
#pragma unroll
                for (int g0 = 0; g0 < MP; g0 += 64) {
                    uint32_t r[4][16];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld_32x32b_x16(d_row + g0 + c * 16, r[c]);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const float v = __uint_as_float(r[c][i]);
                            acc4[i & 3] = fmaf(v, v, acc4[i & 3]);
                        }
                }
            }
            const float acc = (acc4[0] + acc4[1]) + (acc4[2] + acc4[3]);
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.d_empty[buf]);
            const int group = t / kOutTiles, in_group = t % kOutTiles;
            s.obuf[group & 1][in_group * kTile + q * 32 + lane] = acc;
            if (in_group == kOutTiles - 1 || t == n_tiles - 1) {
                asm volatile("bar.sync 2, 128;" ::: "memory");         // the group's scores are in shared memory
                const int g0 = group * kOutTiles * kTile;
                const int count = min(n_tok - g0, (in_group + 1) * kTile);
                for (int i = et; i < count; i += 128) out[g0 + i] = s.obuf[group & 1][i];
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
    if (threadIdx.x == 0 && s.abort && status != nullptr) atomicOr(&status[unit], COMPACTOR_STATUS_TIMEOUT);
}

template <int MP>
cudaError_t launch_score_mp(const Plan& p, const CUtensorMap& kmap, const CUtensorMap& wmap, float* scores,
                            int* status, bool tiny_done, cudaStream_t stream) {
    const int smem = (int)sizeof(ScoreSmem<MP>) + 1024;
    cudaError_t e = cudaFuncSetAttribute(score_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(p.total_schunks, p.layers * p.heads);
    e = launch_chained(kPdlScore, score_kernel<MP>, grid, dim3(kThreads), smem, stream, p, kmap, wmap, scores, status,
                       pdl_enabled(kPdlScore) ? 1 : 0, tiny_done ? 1 : 0);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score(const Plan& p, const Mat& k, const __nv_bfloat16* w, float* scores, int* status, bool tiny_done,
                         cudaStream_t stream) {
    if (p.total_schunks == 0) return cudaSuccess;
    CUtensorMap kmap, wmap;
    const long long units = (long long)p.layers * p.heads * p.batch;
    if (!make_kv_tensor_map(&kmap, k.ptr, p.layers, p.heads, p.total_tokens, k.stride_layer, k.stride_head,
                            k.stride_token, kTile) ||
        !make_rows_tensor_map(&wmap, w, units * 2 * p.mp, p.mp))
        return cudaErrorInvalidValue;
    switch (p.mp) {
        case 16: return launch_score_mp<16>(p, kmap, wmap, scores, status, tiny_done, stream);
        case 32: return launch_score_mp<32>(p, kmap, wmap, scores, status, tiny_done, stream);
        case 48: return launch_score_mp<48>(p, kmap, wmap, scores, status, tiny_done, stream);
        case 64: return launch_score_mp<64>(p, kmap, wmap, scores, status, tiny_done, stream);
        case 128: return launch_score_mp<128>(p, kmap, wmap, scores, status, tiny_done, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace compactor

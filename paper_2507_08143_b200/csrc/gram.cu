// Gram pass: C_p = K_p^T K_p (128 x 128) for every block p of at most `chunk` tokens of every
// unit.  Together with the fp64 projection G = Phi^T (sum_p C_p) Phi in the factor kernel this is
// Algorithm 1, lines 2-3, (K Phi)^T (K Phi), evaluated from exact bf16 products.
//
// One CTA per block, one CTA per SM.  A producer warp streams 128-token tiles of K through a
// six-stage ring of shared memory with TMA (two 64-channel boxes per tile, 128-byte swizzle); one
// thread issues tcgen05.mma with the same tile as both operands (the token axis is the
// contraction axis, so both are MN-major) into one of two 128 x 128 fp32 accumulators in tensor
// memory.  Every 512 tokens the accumulator is handed to eight epilogue warps, which add it
// into fp64 registers (64 columns of one row per thread) while the other accumulator fills; the
// fp64 sums go to global memory once, at the end of the block.  So no fp32 sum is longer than
// 512 tokens, whatever the block length: the tensor-core accumulator loses accuracy in proportion
// to the length of the run.  C_p is symmetric: of its sixteen 32 x 32 blocks only the ten on and
// above the diagonal are summed and written (the projection reads no others).
#include "common.cuh"
#include "sm100.cuh"

namespace compactor {
namespace {

using namespace sm100;

constexpr int kTile = 128;                 // tokens per tile
constexpr int kStages = 6;
constexpr int kBoxBytes = kTile * 128;     // 64 channels x 128 tokens x 2 B
constexpr int kTileBytes = 2 * kBoxBytes;
constexpr int kFlushTiles = kGramFlushTokens / kTile;
constexpr int kEpilogueWarps = 8;
constexpr int kThreads = 64 + 32 * kEpilogueWarps;   // warp 0: TMA, warp 1: MMA, warps 2-9: epilogue
constexpr uint32_t kTmemCols = 256;        // two accumulators

struct __align__(1024) GramSmem {
    unsigned char tiles[kStages][kTileBytes];
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    int abort;
};

__global__ void __launch_bounds__(kThreads, 1)
gram_kernel(Plan p, const __grid_constant__ CUtensorMap kmap, double* __restrict__ partials,
            int* __restrict__ status) {
    pdl_trigger();
    extern __shared__ unsigned char smem_raw[];
    GramSmem& s = *reinterpret_cast<GramSmem*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    const int chunk_id = blockIdx.x;
    const int lh = blockIdx.y;
    const int layer = lh / p.heads, head = lh % p.heads;
    const int b = find_segment(p.cu_chunks, p.batch, chunk_id);
    const int tok_begin = p.cu_seqlens[b] + (chunk_id - p.cu_chunks[b]) * p.chunk;
    const int tok_end = min(tok_begin + p.chunk, p.cu_seqlens[b + 1]);
    const int n_tok = tok_end - tok_begin;
    const int n_tiles = (n_tok + kTile - 1) / kTile;
    const int n_groups = (n_tiles + kFlushTiles - 1) / kFlushTiles;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        prefetch_tensormap(&kmap);
        for (int i = 0; i < kStages; ++i) { mbar_init(&s.full[i], 1); mbar_init(&s.empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&s.acc_full[i], 1); mbar_init(&s.acc_empty[i], kEpilogueWarps); }
        s.abort = 0;
        fence_barrier_init();
    }
    if (warp == 1) { tmem_alloc(&s.tmem_base, kTmemCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = s.tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            for (int t = 0; t < n_tiles; ++t) {
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
        constexpr uint32_t idesc = umma_idesc_bf16(128, 128, 1, 1);
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int stage = t % kStages, round = t / kStages;
            const int g = t / kFlushTiles, in_group = t % kFlushTiles, buf = g & 1;
            if (in_group == 0 && g >= 2) ok = mbar_wait(&s.acc_empty[buf], ((g >> 1) - 1) & 1);
            ok = ok && mbar_wait(&s.full[stage], round & 1) && !*(volatile int*)&s.abort;
            if (!ok) break;
            tc_fence_after_sync();
            const int valid = min(kTile, n_tok - t * kTile);
            if (valid < kTile) {
                // rows past the end of the sequence belong to someone else (or to nobody): clear them
                const int rows = kTile - valid;
                for (int i = lane; i < rows * 16; i += 32) {
                    int box = i / (rows * 8), j = i % (rows * 8);
                    int row = valid + (j >> 3), piece = j & 7;
                    *reinterpret_cast<uint4*>(s.tiles[stage] + box * kBoxBytes + row * 128 + piece * 16) =
                        make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async_smem();
                __syncwarp();
            }
            if (lane == 0) {
                const uint32_t base = smem_u32(s.tiles[stage]);
                const uint32_t d_addr = tmem + buf * 128;
#pragma unroll
                for (int ks = 0; ks < kTile / 16; ++ks) {
                    const uint64_t desc = umma_desc_sw128(base + ks * 2048, kBoxBytes, 1024);
                    umma_bf16(d_addr, desc, desc, idesc, (in_group > 0) || (ks > 0));
                }
                umma_commit(&s.empty[stage]);
                if (in_group == kFlushTiles - 1 || t == n_tiles - 1) umma_commit(&s.acc_full[buf]);
            }
            __syncwarp();
        }
        if (!ok) {
            s.abort = 1;
            if (lane == 0) { mbar_arrive(&s.acc_full[0]); mbar_arrive(&s.acc_full[1]); }   // wake the epilogue
        }
    } else {
        const int q = warp & 3;                       // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;             // which 64 columns
        const int row = q * 32 + lane;
        double acc[64];
#pragma unroll
        for (int i = 0; i < 64; ++i) acc[i] = 0.0;
        bool ok = true;
        for (int g = 0; g < n_groups && ok; ++g) {
            const int buf = g & 1;
            ok = mbar_wait(&s.acc_full[buf], (g >> 1) & 1) && !*(volatile int*)&s.abort;
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                if (half * 2 + c0 / 32 < q) continue;         // a block below the diagonal: its mirror image is kept
                uint32_t r[32];
                tmem_ld_32x32b_x32(tmem + ((uint32_t)(q * 32) << 16) + buf * 128 + half * 64 + c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) acc[c0 + i] += (double)__uint_as_float(r[i]);
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.acc_empty[buf]);
        }
        if (!ok) s.abort = 1;
        if (ok) {
            double* out = partials + ((size_t)lh * p.total_chunks + chunk_id) * kGramElems + (size_t)row * kD + half * 64;
#pragma unroll
            for (int i = 0; i < 64; i += 2)
                if (half * 2 + i / 32 >= q) *reinterpret_cast<double2*>(out + i) = make_double2(acc[i], acc[i + 1]);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
    if (threadIdx.x == 0 && s.abort && status != nullptr)
        atomicOr(&status[lh * p.batch + b], COMPACTOR_STATUS_TIMEOUT);
}

}  // namespace

cudaError_t launch_gram(const Plan& p, const Mat& k, double* partials, int* status, cudaStream_t stream) {
    if (p.total_chunks == 0) return cudaSuccess;
    CUtensorMap kmap;
    if (!make_kv_tensor_map(&kmap, k.ptr, p.layers, p.heads, p.total_tokens, k.stride_layer, k.stride_head,
                            k.stride_token, kTile))
        return cudaErrorInvalidValue;
    const int smem = (int)sizeof(GramSmem) + 1024;
    cudaError_t e = cudaFuncSetAttribute(gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(p.total_chunks, p.layers * p.heads);
    gram_kernel<<<grid, kThreads, smem, stream>>>(p, kmap, partials, status);
    return cudaGetLastError();
}

}  // namespace compactor

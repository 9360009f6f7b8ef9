// Scoring pass (Algorithm 1, lines 5-6, fused): o_i = || k_i W ||^2 with W = Phi L^-T from the
// factor kernel, so that U~ = K^ V~ Sigma~^-1 is never stored.  W arrives as two bf16 terms
// (hi + lo); both are multiplied with the bf16 keys on the tensor cores and summed in fp32.
#include "common.cuh"

namespace compactor {
namespace {

constexpr int kTileTokens = 128;
constexpr int kStages = 2;
constexpr int kThreads = 256;
constexpr int kTileBytes = kTileTokens * kD * 2;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint32_t tile_offset(int row, int col) {
    return (uint32_t)(row * (kD * 2) + ((((col >> 3) ^ (row & 7))) << 4));
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool valid) {
    int bytes = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(bytes));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// MP = padded sketch dimension (multiple of 16).  One CTA scores one Gram chunk of one unit.
template <int MP>
__global__ void __launch_bounds__(kThreads, 1)
score_kernel(Plan p, Mat k, const __nv_bfloat16* __restrict__ w, float* __restrict__ scores) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int kWBytes = 2 * MP * kD * 2;
    const int chunk_id = blockIdx.x;
    const int lh = blockIdx.y;
    const int layer = lh / p.heads, head = lh % p.heads;
    const int b = find_segment(p.cu_chunks, p.batch, chunk_id);
    const int tok_begin = p.cu_seqlens[b] + (chunk_id - p.cu_chunks[b]) * p.chunk;
    const int tok_end = min(tok_begin + p.chunk, p.cu_seqlens[b + 1]);
    const int n_tok = tok_end - tok_begin;
    const int n_tiles = (n_tok + kTileTokens - 1) / kTileTokens;
    const int unit = lh * p.batch + b;

    const __nv_bfloat16* base = k.ptr + layer * k.stride_layer + head * k.stride_head +
                                (long long)tok_begin * k.stride_token;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t w_base = smem_u32(smem);
    const uint32_t k_base = w_base + kWBytes;

    // W of this unit: rows = (term, sketch column), 128 channels each, same piece permutation as
    // the key tiles.
    {
        const __nv_bfloat16* wsrc = w + (size_t)unit * w_elems_per_unit(MP);
        for (int c = tid; c < 2 * MP * 16; c += kThreads) {
            int row = c >> 4, piece = c & 15;
            cp_async_16(w_base + tile_offset(row, piece * 8), wsrc + row * kD + piece * 8, true);
        }
    }
    auto load_tile = [&](int tile, int stage) {
        const uint32_t dst = k_base + stage * kTileBytes;
#pragma unroll
        for (int i = 0; i < (kTileTokens * 16) / kThreads; ++i) {
            int c = tid + i * kThreads;
            int row = c >> 4, piece = c & 15;
            int tok = tile * kTileTokens + row;
            bool valid = tok < n_tok;
            const __nv_bfloat16* src = base + (long long)(valid ? tok : 0) * k.stride_token + piece * 8;
            cp_async_16(dst + tile_offset(row, piece * 8), src, valid);
        }
    };
    load_tile(0, 0);
    asm volatile("cp.async.commit_group;\n");

    float* out = scores + (size_t)lh * p.total_tokens + tok_begin;
    const int j = lane >> 3, r = lane & 7;
    for (int t = 0; t < n_tiles; ++t) {
        if (t + 1 < n_tiles) load_tile(t + 1, (t + 1) & 1);
        asm volatile("cp.async.commit_group;\n");
        asm volatile("cp.async.wait_group 1;\n");
        __syncthreads();
        const uint32_t tile_base = k_base + (t & 1) * kTileBytes;
        float acc[MP / 8][4];
#pragma unroll
        for (int nt = 0; nt < MP / 8; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
            uint32_t a[4];
            ldmatrix_x4(a, tile_base + tile_offset(warp * 16 + r + ((j & 1) ? 8 : 0), ks * 16 + ((j & 2) ? 8 : 0)));
#pragma unroll
            for (int term = 0; term < 2; ++term)
#pragma unroll
                for (int np = 0; np < MP / 16; ++np) {
                    uint32_t bf[4];
                    ldmatrix_x4(bf, w_base + tile_offset(term * MP + np * 16 + r + ((j & 2) ? 8 : 0),
                                                         ks * 16 + ((j & 1) ? 8 : 0)));
                    mma_bf16(acc[2 * np], a, bf[0], bf[1]);
                    mma_bf16(acc[2 * np + 1], a, bf[2], bf[3]);
                }
        }
        float lo = 0.f, hi = 0.f;     // rows lane/4 and lane/4 + 8 of the warp's 16 tokens
#pragma unroll
        for (int nt = 0; nt < MP / 8; ++nt) {
            lo = fmaf(acc[nt][0], acc[nt][0], lo); lo = fmaf(acc[nt][1], acc[nt][1], lo);
            hi = fmaf(acc[nt][2], acc[nt][2], hi); hi = fmaf(acc[nt][3], acc[nt][3], hi);
        }
        lo += __shfl_xor_sync(0xffffffffu, lo, 1); lo += __shfl_xor_sync(0xffffffffu, lo, 2);
        hi += __shfl_xor_sync(0xffffffffu, hi, 1); hi += __shfl_xor_sync(0xffffffffu, hi, 2);
        if ((lane & 3) == 0) {
            int tok = t * kTileTokens + warp * 16 + (lane >> 2);
            if (tok < n_tok) out[tok] = lo;
            if (tok + 8 < n_tok) out[tok + 8] = hi;
        }
        __syncthreads();   // the stage read here is refilled at the top of the next iteration
    }
    asm volatile("cp.async.wait_group 0;\n");
}

template <int MP>
cudaError_t launch_score_mp(const Plan& p, const Mat& k, const __nv_bfloat16* w, float* scores, cudaStream_t stream) {
    const int smem = 2 * MP * kD * 2 + kStages * kTileBytes;
    cudaError_t e = cudaFuncSetAttribute(score_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(p.total_chunks, p.layers * p.heads);
    score_kernel<MP><<<grid, kThreads, smem, stream>>>(p, k, w, scores);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score(const Plan& p, const Mat& k, const __nv_bfloat16* w, float* scores, cudaStream_t stream) {
    if (p.total_chunks == 0) return cudaSuccess;
    switch (p.mp) {
        case 16: return launch_score_mp<16>(p, k, w, scores, stream);
        case 32: return launch_score_mp<32>(p, k, w, scores, stream);
        case 48: return launch_score_mp<48>(p, k, w, scores, stream);
        case 64: return launch_score_mp<64>(p, k, w, scores, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace compactor

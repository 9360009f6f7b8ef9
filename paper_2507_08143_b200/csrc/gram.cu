// Gram pass: C_p = K_p^T K_p (128 x 128, fp32) for every block p of at most `chunk` tokens of
// every unit.  Together with the fp64 projection G = Phi^T (sum_p C_p) Phi in the factor kernel
// this is Algorithm 1, lines 2-3, (K Phi)^T (K Phi), evaluated from exact bf16 products.
#include "common.cuh"

namespace compactor {
namespace {

constexpr int kTileTokens = 64;
constexpr int kStages = 3;
constexpr int kThreads = 256;
constexpr int kTileBytes = kTileTokens * kD * 2;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

// Byte offset inside a tile of the 16-byte piece holding channels [col, col+8) of token `row`.
// Pieces of a row are permuted by the row's low bits so that 8 consecutive rows of one column
// group fall into distinct banks.
__device__ __forceinline__ uint32_t tile_offset(int row, int col) {
    return (uint32_t)(row * (kD * 2) + ((((col >> 3) ^ (row & 7))) << 4));
}

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, bool valid) {
    int bytes = valid ? 16 : 0;   // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(bytes));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(kThreads, 1)
gram_kernel(Plan p, Mat k, float* __restrict__ partials) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int chunk_id = blockIdx.x;
    const int lh = blockIdx.y;
    const int layer = lh / p.heads, head = lh % p.heads;
    const int b = find_segment(p.cu_chunks, p.batch, chunk_id);
    const int tok_begin = p.cu_seqlens[b] + (chunk_id - p.cu_chunks[b]) * p.chunk;
    const int tok_end = min(tok_begin + p.chunk, p.cu_seqlens[b + 1]);
    const int n_tok = tok_end - tok_begin;
    const int n_tiles = (n_tok + kTileTokens - 1) / kTileTokens;

    const __nv_bfloat16* base = k.ptr + layer * k.stride_layer + head * k.stride_head +
                                (long long)tok_begin * k.stride_token;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int warp_m = warp >> 2, warp_n = warp & 3;
    const uint32_t smem_base = smem_u32(smem);

    auto load_tile = [&](int tile, int stage) {
        const uint32_t dst = smem_base + stage * kTileBytes;
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

    float acc[4][4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

    for (int s = 0; s < kStages - 1; ++s) {
        if (s < n_tiles) load_tile(s, s);
        asm volatile("cp.async.commit_group;\n");
    }

    const int j = lane >> 3, r = lane & 7;
    for (int t = 0; t < n_tiles; ++t) {
        asm volatile("cp.async.wait_group %0;\n" ::"n"(kStages - 2));
        __syncthreads();
        {   // prefetch tile t + kStages - 1 into the stage that was consumed at iteration t - 1
            int nt = t + kStages - 1;
            if (nt < n_tiles) load_tile(nt, nt % kStages);
            asm volatile("cp.async.commit_group;\n");
        }
        const uint32_t tile_base = smem_base + (t % kStages) * kTileBytes;
#pragma unroll
        for (int ks = 0; ks < kTileTokens / 16; ++ks) {
            const int k0 = ks * 16;
            uint32_t a[4][4], bfrag[2][4];
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                int row = k0 + r + ((j & 2) ? 8 : 0);
                int col = warp_m * 64 + mt * 16 + ((j & 1) ? 8 : 0);
                ldmatrix_x4_trans(a[mt], tile_base + tile_offset(row, col));
            }
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                int row = k0 + r + ((j & 1) ? 8 : 0);
                int col = warp_n * 32 + np * 16 + ((j & 2) ? 8 : 0);
                ldmatrix_x4_trans(bfrag[np], tile_base + tile_offset(row, col));
            }
#pragma unroll
            for (int mt = 0; mt < 4; ++mt)
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
                    mma_bf16(acc[mt][nt], a[mt], bfrag[nt >> 1][(nt & 1) * 2], bfrag[nt >> 1][(nt & 1) * 2 + 1]);
        }
    }
    asm volatile("cp.async.wait_group 0;\n");

    float* out = partials + ((size_t)lh * p.total_chunks + chunk_id) * kGramElems;
    const int g = lane >> 2, tq = lane & 3;
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            int row = warp_m * 64 + mt * 16 + g;
            int col = warp_n * 32 + nt * 8 + tq * 2;
            *reinterpret_cast<float2*>(out + row * kD + col) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
            *reinterpret_cast<float2*>(out + (row + 8) * kD + col) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
        }
}

}  // namespace

cudaError_t launch_gram(const Plan& p, const Mat& k, float* partials, cudaStream_t stream) {
    if (p.total_chunks == 0) return cudaSuccess;
    static bool configured = false;
    const int smem = kStages * kTileBytes;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid(p.total_chunks, p.layers * p.heads);
    gram_kernel<<<grid, kThreads, smem, stream>>>(p, k, partials);
    return cudaGetLastError();
}

}  // namespace compactor

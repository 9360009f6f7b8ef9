// Token-averaged negative log-likelihood (Section 3.5): NLL = -(1/L) sum_i log softmax(logits_i)[t_i],
// the context statistic that the calibrated retention ratio is a function of.
//
//   nll_rows_kernel   one CTA per row of logits: a single streaming pass keeps, per thread, a
//                     running maximum and the sum of 2^(y - max) (y = logit * log2 e), 16-byte
//                     loads, several in flight; the threads' pairs are merged through shuffles and
//                     shared memory; row result = ln 2 * (max + log2 sum) - logit[target].
//   nll_mean_kernel   one CTA per sequence: fp64 sum of its rows' results in a fixed order
//                     (deterministic), divided by the number of scored rows.
// Bound by HBM: every logit is read once (2 or 4 bytes per logit).
#include "common.cuh"

namespace compactor {
namespace {

constexpr int kNllThreads = 256;
constexpr int kNllInFlight = 4;            // 16-byte loads issued before the first is used
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint4 ld_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Elements of one 16-byte vector as floats.
template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
    static constexpr int kElems = 8;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ float scalar(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};
template <> struct Vec<float> {
    static constexpr int kElems = 4;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ float scalar(const float* p) { return *p; }
};

// Running (max, sum of 2^(y - max)) pair; `add` takes values already scaled by log2 e.
struct MaxSum {
    float mx, sum;
    __device__ __forceinline__ void merge(const MaxSum& o) {
        const float m = fmaxf(mx, o.mx);
        if (m == -INFINITY) return;                       // both empty
        sum = sum * ex2f(mx - m) + o.sum * ex2f(o.mx - m);
        mx = m;
    }
};

template <typename T>
__global__ void __launch_bounds__(kNllThreads)
nll_rows_kernel(const T* __restrict__ logits, long long row_stride, int vocab, const int* __restrict__ targets,
                long long rows, float* __restrict__ row_nll) {
    constexpr int E = Vec<T>::kElems;
    __shared__ MaxSum part[kNllThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_vec = vocab / E;
    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const int target = targets[row];
        if (target < 0 || target >= vocab) {               // not scored
            if (tid == 0) row_nll[row] = 0.f;
            continue;
        }
        const T* x = logits + row * row_stride;
        MaxSum acc{-INFINITY, 0.f};
        for (int v0 = tid; v0 < n_vec; v0 += kNllThreads * kNllInFlight) {
            uint4 raw[kNllInFlight];
#pragma unroll
            for (int u = 0; u < kNllInFlight; ++u) {
                const int v = v0 + u * kNllThreads;
                raw[u] = v < n_vec ? ld_stream(x + (size_t)v * E) : make_uint4(0, 0, 0, 0);
            }
            float y[kNllInFlight][E];
            float mx = acc.mx;
#pragma unroll
            for (int u = 0; u < kNllInFlight; ++u) {
                const bool live = v0 + u * kNllThreads < n_vec;
                float f[E];
                Vec<T>::unpack(raw[u], f);
#pragma unroll
                for (int i = 0; i < E; ++i) {
                    y[u][i] = live ? f[i] * kLog2e : -INFINITY;
                    mx = fmaxf(mx, y[u][i]);
                }
            }
            if (mx == -INFINITY) continue;                  // nothing but -inf so far
            float s = acc.sum * ex2f(acc.mx - mx);
#pragma unroll
            for (int u = 0; u < kNllInFlight; ++u)
#pragma unroll
                for (int i = 0; i < E; ++i) s += ex2f(y[u][i] - mx);
            acc.mx = mx; acc.sum = s;
        }
        if (tid < vocab - n_vec * E) {                      // the last few logits of a row
            MaxSum one{Vec<T>::scalar(x + n_vec * E + tid) * kLog2e, 1.f};
            acc.merge(one);
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            MaxSum o{__shfl_xor_sync(0xffffffffu, acc.mx, d), __shfl_xor_sync(0xffffffffu, acc.sum, d)};
            acc.merge(o);
        }
        if (lane == 0) part[warp] = acc;
        __syncthreads();
        if (tid == 0) {
            MaxSum all = part[0];
            for (int w = 1; w < kNllThreads / 32; ++w) all.merge(part[w]);
            const float log_z = kLn2 * (all.mx + log2f(all.sum));
            row_nll[row] = log_z - Vec<T>::scalar(x + target);
        }
        __syncthreads();
    }
}

constexpr int kMeanSeqs = 64;              // sequences per launch of the averaging kernel
struct MeanArgs { long long begin[kMeanSeqs + 1]; };

__global__ void __launch_bounds__(kNllThreads)
nll_mean_kernel(const float* __restrict__ row_nll, const int* __restrict__ targets, int vocab, MeanArgs a,
                double* __restrict__ out) {
    __shared__ double sum_s[kNllThreads];
    __shared__ long long cnt_s[kNllThreads];
    const int tid = threadIdx.x;
    const long long r0 = a.begin[blockIdx.x], r1 = a.begin[blockIdx.x + 1];
    double sum = 0.0; long long cnt = 0;
    for (long long r = r0 + tid; r < r1; r += kNllThreads) {
        const int t = targets[r];
        if (t >= 0 && t < vocab) { sum += (double)row_nll[r]; ++cnt; }
    }
    sum_s[tid] = sum; cnt_s[tid] = cnt;
    __syncthreads();
    for (int d = kNllThreads / 2; d > 0; d >>= 1) {
        if (tid < d) { sum_s[tid] += sum_s[tid + d]; cnt_s[tid] += cnt_s[tid + d]; }
        __syncthreads();
    }
    if (tid == 0) out[blockIdx.x] = cnt_s[0] > 0 ? sum_s[0] / (double)cnt_s[0] : 0.0;
}

}  // namespace

cudaError_t launch_nll(const void* logits, int is_fp32, long long rows, int vocab, long long row_stride,
                       const int* targets, int batch, const int* cu_rows_host, float* row_nll, double* nll_out,
                       cudaStream_t stream) {
    if (rows > 0) {
        const int grid = (int)(rows < (1LL << 30) ? rows : (1LL << 30));
        if (is_fp32)
            nll_rows_kernel<float><<<grid, kNllThreads, 0, stream>>>(static_cast<const float*>(logits), row_stride,
                                                                     vocab, targets, rows, row_nll);
        else
            nll_rows_kernel<__nv_bfloat16><<<grid, kNllThreads, 0, stream>>>(
                static_cast<const __nv_bfloat16*>(logits), row_stride, vocab, targets, rows, row_nll);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    for (int b0 = 0; b0 < batch; b0 += kMeanSeqs) {
        const int nb = batch - b0 < kMeanSeqs ? batch - b0 : kMeanSeqs;
        MeanArgs a;
        for (int i = 0; i <= nb; ++i) a.begin[i] = cu_rows_host[b0 + i];
        nll_mean_kernel<<<nb, kNllThreads, 0, stream>>>(row_nll, targets, vocab, a, nll_out + b0);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace compactor

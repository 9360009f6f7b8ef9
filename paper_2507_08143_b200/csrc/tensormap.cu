// Host-side construction of the TMA descriptors.  The driver entry point is looked up through
// the runtime so that the library does not link against libcuda directly.
#include <cudaTypedefs.h>

#include "sm100.cuh"

namespace compactor {
namespace {

PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    }();
    return fn;
}

}  // namespace

bool make_kv_tensor_map(CUtensorMap* map, const void* base, int layers, int heads, long long tokens,
                        long long stride_layer, long long stride_head, long long stride_token, int box_tokens) {
    auto fn = encode_fn();
    if (fn == nullptr || tokens < 1) return false;
    // A dimension of extent 1 still needs a legal (16-byte multiple, non-zero) stride.
    const long long row_bytes = 128 * 2;
    cuuint64_t dims[4] = {128, (cuuint64_t)tokens, (cuuint64_t)heads, (cuuint64_t)layers};
    cuuint64_t strides[3] = {(cuuint64_t)(stride_token * 2),
                             (cuuint64_t)((heads > 1 ? stride_head : 128) * 2),
                             (cuuint64_t)((layers > 1 ? stride_layer : 128) * 2)};
    if (strides[1] == 0) strides[1] = row_bytes;
    if (strides[2] == 0) strides[2] = row_bytes;
    cuuint32_t box[4] = {64, (cuuint32_t)box_tokens, 1, 1};
    cuuint32_t elem[4] = {1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, elem,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_rows_tensor_map(CUtensorMap* map, const void* base, long long rows, int box_rows) {
    auto fn = encode_fn();
    if (fn == nullptr || rows < 1) return false;
    cuuint64_t dims[2] = {128, (cuuint64_t)rows};
    cuuint64_t strides[1] = {128 * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t elem[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace compactor

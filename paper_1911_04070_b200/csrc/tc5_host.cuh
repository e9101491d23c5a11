// Host side of the TMA loads of the tensor-memory kernels: tensor maps over the node-major
// [B, N, H, 64] bf16 tensors and the [n_rel, 64] relation table.  A box is 16 consecutive rows of 64
// elements of one (batch entry, head), written to shared memory in the 128-byte swizzle the tensor
// core reads.  The maps cover this GPU's own memory only and every CTA issues its own loads.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

namespace bpt {
namespace tc5 {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (the library does not link libcuda).
inline EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) != cudaSuccess ||
            qr != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Map over a [B, N, H, 64] bf16 tensor; coordinates (0, head, node, batch entry).  Rows past the last node
// of the tensor read as zeros.
inline bool node_rows_map(CUtensorMap* m, const void* base, int B, int N, int H) {
    const cuuint64_t dims[4] = {64, (cuuint64_t)H, (cuuint64_t)N, (cuuint64_t)B};
    const cuuint64_t strides[3] = {128, (cuuint64_t)H * 128, (cuuint64_t)N * H * 128};
    const cuuint32_t box[4] = {64, 1, 16, 1}, estr[4] = {1, 1, 1, 1};
    return encode_tiled()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// Map over the [n_rel, 64] relation table; coordinates (0, relation).
inline bool rel_rows_map(CUtensorMap* m, const void* base, int n_rel) {
    const cuuint64_t dims[2] = {64, (cuuint64_t)n_rel};
    const cuuint64_t strides[1] = {128};
    const cuuint32_t box[2] = {64, 16}, estr[2] = {1, 1};
    return encode_tiled()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc5
}  // namespace bpt

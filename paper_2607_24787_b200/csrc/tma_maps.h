// Host-side construction of the TMA tensor maps used by the grouped FFN kernel.
// cuTensorMapEncodeTiled is looked up through the runtime, so the library has no link-time
// dependency on libcuda and still loads on a machine without a driver.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace spm {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// cuStreamWriteValue32: a 32-bit store to device memory in stream order (used to publish "this
// slot's copy has landed" to kernels that wait on the device side).
typedef CUresult (*StreamWriteValue32Fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);

inline StreamWriteValue32Fn stream_write32_fn() {
    static StreamWriteValue32Fn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuStreamWriteValue32", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<StreamWriteValue32Fn>(p);
    }
    return fn;
}

// Packed bf16 expert blobs [n_slots][I][3][D] viewed as a 4-D tensor (D, 3, I, n_slots); a box is
// 64 consecutive elements of D x 128 consecutive rows of one plane of one slot, 128-byte swizzle.
inline bool make_weight_map(CUtensorMap* map, const void* base, int D, int I, uint64_t n_slots) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {cuuint64_t(D), 3, cuuint64_t(I), n_slots};
    const cuuint64_t strides[3] = {cuuint64_t(D) * 2, cuuint64_t(D) * 6, cuuint64_t(D) * 6 * cuuint64_t(I)};
    const cuuint32_t box[4] = {64, 1, 128, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 token rows [rows][D]; a box is 64 elements x `box_rows` rows, 128-byte swizzle.
inline bool make_token_map(CUtensorMap* map, const void* base, int D, uint64_t rows, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cuuint64_t(D), rows};
    const cuuint64_t strides[1] = {cuuint64_t(D) * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Packed 4-bit expert blobs [n_slots][I][3][RB bytes] (RB = D/2 nibble bytes + D/16 scale bytes per
// row) viewed as a 4-D byte tensor (RB, 3, I, n_slots). Two box shapes over the same memory:
// 64 nibble bytes (128 weights) x 128 rows with the 64-byte swizzle, and 16 scale bytes x 128 rows.
inline bool make_q4_maps(CUtensorMap* nib64, CUtensorMap* sc16, const void* base, int D, int I, uint64_t n_slots) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t rb = cuuint64_t(D) / 2 + cuuint64_t(D) / 16;
    const cuuint64_t dims[4] = {rb, 3, cuuint64_t(I), n_slots};
    const cuuint64_t strides[3] = {rb, rb * 3, rb * 3 * cuuint64_t(I)};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const cuuint32_t box_n[4] = {64, 1, 128, 1}, box_s[4] = {16, 1, 128, 1};
    return fn(nib64, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box_n, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS &&
           fn(sc16, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box_s, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace spm

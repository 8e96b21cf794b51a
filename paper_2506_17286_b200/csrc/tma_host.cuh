// Host-side construction of TMA tensor maps (bf16, 128-byte swizzle) through the driver entry
// point, so that the library needs no link-time dependency on libcuda.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gta {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Dense bf16 tensor of `rank` dimensions (innermost first), box `box`, 128-byte swizzle, zero
// fill outside the tensor.  The innermost box extent must be 64 elements (one swizzle row).
// `alloc`, when given, holds the allocated extent of every dimension (>= dims): the strides follow the
// allocation while only `dims` is addressable, so that rows that exist in memory but are not part of the
// problem (the unused tail of a cache) read as zeros like everything else outside the tensor.
inline bool make_bf16_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint32_t* box,
                          const uint64_t* alloc = nullptr) {
    EncodeTiledFn fn = tensor_map_encoder();
    if (!fn) return false;
    cuuint64_t gdim[5], gstride[5];
    cuuint32_t bx[5], estr[5];
    uint64_t stride = 2;
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bx[i] = box[i];
        estr[i] = 1;
        stride *= alloc ? alloc[i] : dims[i];
        if (i < rank - 1) gstride[i] = stride;   // byte stride of dimension i+1
    }
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstride, bx, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Dense tensor of bytes (8-bit codes), same conventions: the innermost box extent is 128 bytes (one swizzle row).
inline bool make_u8_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint32_t* box) {
    EncodeTiledFn fn = tensor_map_encoder();
    if (!fn) return false;
    cuuint64_t gdim[5], gstride[5];
    cuuint32_t bx[5], estr[5];
    uint64_t stride = 1;
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bx[i] = box[i];
        estr[i] = 1;
        stride *= dims[i];
        if (i < rank - 1) gstride[i] = stride;
    }
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstride, bx, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace gta

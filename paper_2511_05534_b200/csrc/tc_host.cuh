// Host side of the tensor-core kernels: building TMA tensor maps through the driver entry point
// (looked up at run time, so the library does not link against libcuda).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace flowmm {
namespace tc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 tensor of `rank` dims (innermost first, contiguous innermost), box as given (box[0] = 64
// elements = one 128-byte swizzle span), 128-byte swizzle, zero fill outside the tensor.
// strides_bytes[i] is the stride of dim i+1.  Returns false if the driver rejects the description.
inline bool make_bf16_map(CUtensorMap *map, const void *base, int rank, const uint64_t *dims,
                          const uint64_t *strides_bytes, const uint32_t *box_dims) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[5], gstride[4];
    cuuint32_t box[5], estr[5];
    for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; box[i] = box_dims[i]; estr[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) gstride[i] = strides_bytes[i];
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), gdim, gstride, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// SM count of the current device (a benign race: every thread would store the same value).
inline int sm_count() {
    constexpr int kSlots = 64;
    static int n[kSlots] = {};
    int dev = 0, count = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < kSlots && n[dev] != 0) return n[dev];
    cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev);
    if (dev >= 0 && dev < kSlots) n[dev] = count;
    return count;
}

}  // namespace tc
}  // namespace flowmm

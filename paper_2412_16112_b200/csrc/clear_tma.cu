// Tensor maps (TMA descriptors) of the tensor-core kernels: one encoder for both.
#include <cuda.h>
#include <cuda_runtime.h>

#include "clear_internal.hpp"

namespace clear {
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// the driver's encoder, looked up through the runtime (the library does not link against libcuda)
EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

}  // namespace

bool encode_bf16_map(void *tensor_map, const void *base, int rank, const uint64_t *dims, const uint64_t *strides,
                     const uint32_t *box)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    CUresult rc = fn(static_cast<CUtensorMap *>(tensor_map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
                     const_cast<void *>(base), reinterpret_cast<const cuuint64_t *>(dims),
                     reinterpret_cast<const cuuint64_t *>(strides), reinterpret_cast<const cuuint32_t *>(box), ones,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

}  // namespace clear

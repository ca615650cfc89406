#include "rq_tmap.h"

namespace rq {

namespace {

typedef CUresult (*TensorMapEncodeTiled)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                         const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                         CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

TensorMapEncodeTiled tensor_map_encoder()
{
    static TensorMapEncodeTiled fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = (TensorMapEncodeTiled)p;
    }
    return fn;
}

}  // namespace

cudaError_t cache_tensor_map(CUtensorMap *out, const void *kv, int D, int S, int64_t pages_total, int positions)
{
    if (positions % S != 0 || D % 64 != 0) return cudaErrorInvalidValue;
    if (pages_total < 1 || pages_total >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;   // box coordinates are 32-bit
    const TensorMapEncodeTiled encode = tensor_map_encoder();
    if (!encode) return cudaErrorNotSupported;
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)S, 2, (cuuint64_t)pages_total};
    const cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)S * D * 2, (cuuint64_t)2 * S * D * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)S, 1, (cuuint32_t)(positions / S)}, steps[4] = {1, 1, 1, 1};
    if (encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(kv), dims, strides, box, steps,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    return cudaSuccess;
}

}  // namespace rq

// Tensor map (TMA descriptor) of a paged cache of decayed keys and values.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rq {

// The bf16 cache [pages of all heads][key / value][slot][channel] as a rank-4 tensor (channel, slot, key / value,
// page) with a box of 64 channels x the slots of a page x one of key / value x the pages of `positions`
// consecutive positions (a multiple of the page size), 128-byte swizzle: one tiled bulk-tensor copy brings a
// 64-channel half of `positions` rows into shared memory as rows of 128 bytes in the layout the tensor core
// reads.  The driver's encoder is looked up once through the runtime (the library does not link the driver).
cudaError_t cache_tensor_map(CUtensorMap *out, const void *kv, int D, int S, int64_t pages_total, int positions);

}  // namespace rq

// Tensor maps of the paged KV pools, shared by the kernels that fetch pages with tiled TMA copies.
#pragma once

#include <cuda.h>  // CUtensorMap and its enums only; the encoder is looked up at run time

#include "arb_common.cuh"

namespace arb {

// False when the driver has no cuTensorMapEncodeTiled: the callers then use their CUDA-core paths.
bool tma_available();

// Encodes `map` as the 2-D view of a page pool: rows = (page, kv head, slot), 128 elements each.
// bf16 pools: rows of 256 bytes, a box is 16 rows x 64 elements; E4M3 pools: rows of 128 bytes, a box is
// 16 whole rows.  128-byte swizzle either way.
bool encode_pool_map(CUtensorMap *map, const void *pool, int num_pages, int num_kv_heads, bool e4m3);

// The same map out of the context's cache, copied to `map` (encoded on first use: a model's pools come back
// every token, and encoding two maps costs about as much host time as launching a kernel).  Host-side, not
// thread-safe, like ctx.
bool pool_map(Ctx *ctx, CUtensorMap *map, const void *pool, int num_pages, int num_kv_heads, bool e4m3);

void pool_map_cache_free(Ctx *ctx);

}  // namespace arb

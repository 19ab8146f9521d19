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

// The views of a pool the kernels use.
enum class PoolView : int {
    kBf16HalfRows = 0,    // 2-D, box 16 rows x 64 elements (one 128-byte-swizzled half tile)
    kE4m3 = 1,            // 2-D over E4M3 codes, box 16 whole rows of 128 bytes
    kBf16WholeRows = 2,   // 3-D (64 elements, rows, 2 halves), box 16 rows x both halves: a page in one copy
    kI4 = 3,              // 2-D over 4-bit codes, box 16 whole rows of 64 bytes, not swizzled
};

// 3-D view kBf16WholeRows; false if the driver refuses the encoding (the caller then uses kBf16HalfRows).
bool encode_pool_map3(CUtensorMap *map, const void *pool, int num_pages, int num_kv_heads);

// A view's map out of the context's cache, copied to `map` (encoded on first use: a model's pools come back
// every token, and encoding two maps costs about as much host time as launching a kernel).  Host-side, not
// thread-safe, like ctx.
bool pool_map(Ctx *ctx, CUtensorMap *map, const void *pool, int num_pages, int num_kv_heads, PoolView view);

void pool_map_cache_free(Ctx *ctx);

}  // namespace arb

// Tensor maps of the paged KV pools: encoder lookup, encoding, and a small per-context cache.
#include <new>

#include "arb_tma.cuh"

namespace arb {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        cudaGetLastError();
    }
    return fn;
}

constexpr int kD = 128;
constexpr int kMapSlots = 512;   // a power of two; a pool hashes to kMapProbe neighbouring slots
constexpr int kMapProbe = 4;

struct MapEntry {
    alignas(64) CUtensorMap map;
    const void *pool = nullptr;
    int num_pages = 0, num_kv_heads = 0, view = 0;
};

}  // namespace

bool tma_available() { return encode_tiled_fn() != nullptr; }

bool encode_pool_map(CUtensorMap *map, const void *pool, int num_pages, int num_kv_heads, bool e4m3) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)num_pages * num_kv_heads * kPage};
    const cuuint64_t strides[1] = {(cuuint64_t)kD * (e4m3 ? 1 : 2)};
    const cuuint32_t box[2] = {(cuuint32_t)(e4m3 ? kD : 64), (cuuint32_t)kPage};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, e4m3 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
              const_cast<void *>(pool), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same bf16 pool as a 3-D view (64 elements, rows, the two 64-element halves of a row; the third
// dimension's stride, 128 bytes, is smaller than the second's, 256): one box of 16 rows x both halves lands
// as [half][row][128 bytes], the layout two boxes of the 2-D view give, with one copy instead of two.
bool encode_pool_map3(CUtensorMap *map, const void *pool, int num_pages, int num_kv_heads) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {64, (cuuint64_t)num_pages * num_kv_heads * kPage, 2};
    const cuuint64_t strides[2] = {(cuuint64_t)kD * 2, 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)kPage, 2};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(pool), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A pool of 4-bit codes: rows of 64 bytes; one box is the 16 rows of a (page, kv head), landing row-major (no swizzle:
// the rows are read by plain shared-memory loads, 32 bytes per lane, before they are widened).
bool encode_pool_map_i4(CUtensorMap *map, const void *pool, int num_pages, int num_kv_heads) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)kD / 2, (cuuint64_t)num_pages * num_kv_heads * kPage};
    const cuuint64_t strides[1] = {(cuuint64_t)kD / 2};
    const cuuint32_t box[2] = {(cuuint32_t)kD / 2, (cuuint32_t)kPage};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(pool), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {
bool encode_view(CUtensorMap *map, const void *pool, int num_pages, int num_kv_heads, PoolView view) {
    if (view == PoolView::kI4) return encode_pool_map_i4(map, pool, num_pages, num_kv_heads);
    if (view == PoolView::kBf16WholeRows) return encode_pool_map3(map, pool, num_pages, num_kv_heads);
    return encode_pool_map(map, pool, num_pages, num_kv_heads, view == PoolView::kE4m3);
}
}  // namespace

bool pool_map(Ctx *ctx, CUtensorMap *map, const void *pool, int num_pages, int num_kv_heads, PoolView view) {
    MapEntry *cache = static_cast<MapEntry *>(ctx->map_cache);
    if (cache == nullptr) {
        cache = new (std::nothrow) MapEntry[kMapSlots];
        if (cache == nullptr) return encode_view(map, pool, num_pages, num_kv_heads, view);
        ctx->map_cache = cache;
    }
    // pools are large allocations: the low bits of their addresses carry nothing
    const uintptr_t a = reinterpret_cast<uintptr_t>(pool);
    const unsigned h = (unsigned)((a >> 9) ^ (a >> 18) ^ (a >> 27)) * 2654435761u;
    const unsigned first = (h >> 16) & (kMapSlots - 1);
    for (int i = 0; i < kMapProbe; ++i) {
        MapEntry &e = cache[(first + i) & (kMapSlots - 1)];
        if (e.pool == pool && e.num_pages == num_pages && e.num_kv_heads == num_kv_heads && e.view == (int)view) {
            *map = e.map;
            return true;
        }
    }
    // not there: take a free neighbour, else turn one out (in rotation, so that none is stuck forever)
    MapEntry *slot = nullptr;
    for (int i = 0; i < kMapProbe && slot == nullptr; ++i) {
        MapEntry &e = cache[(first + i) & (kMapSlots - 1)];
        if (e.pool == nullptr) slot = &e;
    }
    if (slot == nullptr) slot = &cache[(first + (ctx->map_evictions++ % kMapProbe)) & (kMapSlots - 1)];
    slot->pool = nullptr;
    if (!encode_view(&slot->map, pool, num_pages, num_kv_heads, view)) return false;
    slot->pool = pool;
    slot->num_pages = num_pages;
    slot->num_kv_heads = num_kv_heads;
    slot->view = (int)view;
    *map = slot->map;
    return true;
}

void pool_map_cache_free(Ctx *ctx) {
    delete[] static_cast<MapEntry *>(ctx->map_cache);
    ctx->map_cache = nullptr;
}

}  // namespace arb

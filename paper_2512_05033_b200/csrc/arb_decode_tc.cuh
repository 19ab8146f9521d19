// Pieces shared by the tensor-core decode kernels (arb_decode_mma.cu: the two-kernel form for back-to-back
// series and the E4M3 cache; arb_decode_step.cu: the single-launch form): the cut of the flat
// (sequence, kv head, page) list into per-CTA ranges, tiled TMA loads, ldmatrix / mma.sync wrappers.
#pragma once

#include "arb_tma.cuh"

namespace arb {

constexpr int kD = 128;               // head_dim of the tensor-core decode kernels
constexpr int kMinChunk = 4;          // fewest pages worth giving a CTA
constexpr int kSmallCallPages = 64;   // up to this many pages per SM a call runs one CTA per SM

struct Segment {
    int b, kvh, pg0, pg1, L, bk, nparts, c_first;
};

// The cut of the flat (sequence, kv head, page) list into per-CTA ranges: both kernels of a call must
// agree on it.  Small calls use the first `small_ctas` CTAs of the grid -- one per SM, or one per
// two SMs for a call that runs back to back with its neighbours (see launch_decode_mma) -- and
// large ones the whole grid.
__device__ __forceinline__ int plan_chunk(int total, int grid, int small_ctas) {
    const int one_per_sm = min(grid, small_ctas);
    const int active = total <= one_per_sm * kSmallCallPages ? one_per_sm : grid;
    const int chunk = (total + active - 1) / active;
    return chunk < kMinChunk ? kMinChunk : chunk;
}

__device__ __forceinline__ bool next_segment(int &cur, int r1, const int *pref, const int *slen, int B, int Hkv,
                                             int chunk, Segment &s) {
    if (cur >= r1) return false;
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (pref[mid] <= cur) lo = mid; else hi = mid;
    }
    const int b = lo;
    const int pages = (pref[b + 1] - pref[b]) / Hkv;
    const int r = cur - pref[b];
    const int kvh = r / pages;
    const int pg0 = r - kvh * pages;
    const int s0 = pref[b] + kvh * pages;
    const int s1 = s0 + pages;
    const int end = s1 < r1 ? s1 : r1;
    s.b = b;
    s.kvh = kvh;
    s.pg0 = pg0;
    s.pg1 = pg0 + (end - cur);
    s.L = slen[b];
    s.bk = b * Hkv + kvh;
    s.c_first = s0 / chunk;
    s.nparts = (s1 - 1) / chunk - s.c_first + 1;
    cur = end;
    return true;
}


__device__ __forceinline__ void tma_box_load(void *dst_smem, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void tma_box_load3(void *dst_smem, const CUtensorMap *map, int x, int y, int z, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}

// four 8x8 bf16 blocks; lanes 8i..8i+7 give the row addresses of block i
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D(16x8, fp32) += A(16x16, row) * B(16x8, col), operands bf16 (bf16 cache) or f16 (widened E4M3 codes)
template <bool F16>
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    if constexpr (F16)
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
            "{%0, %1, %2, %3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    else
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
            "{%0, %1, %2, %3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// transposes an 8 x 8 matrix of 16-bit elements held one row per four lanes, two elements per lane
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t v) {
    uint32_t r;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(v));
    return r;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}


}  // namespace arb

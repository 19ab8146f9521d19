// One decode token in one launch (bf16, head_dim 128, group size <= 8): the cache write of the token's new
// K/V rows, split-KV attention over the paged cache, the split combine and the length update, all in one
// kernel.  This is what a token of a draft or target step costs in Algorithm 1 of the paper ("Sample draft
// step" / "Sample target step": z_i ~ q(z_i | x, z_<i), Section 3.1): every call of that chain reads what the
// call before it wrote, so nothing overlaps and a token pays the latency of every launch on its way.  Three
// launches (append, decode, combine) become one.
//
// What is shared with the two-kernel decode (arb_decode_mma.cu): the flat (sequence, kv head, page) list cut
// into equal ranges per CTA, a producer warp feeding a ring of 4 KB page tiles through tiled TMA copies, one
// consumer warp per page with its own online softmax.  What differs:
//   - The product is transposed.  S^T = K q^T puts the 16 keys of a page on the 16 rows of an m16n8k16 tile and
//     the group's heads (padded to 8) on its 8 columns; O^T += V^T P^T does the same for the second product.
//     A page costs 8 + 8 MMAs instead of 16 + 16, the accumulators take 32 registers instead of 64, and the
//     CTA runs eight consumer warps, two per scheduler, which hide one another's latencies.  P^T reaches the
//     second product's B fragment through two movmatrix transposes; the row maximum is a reduction over the
//     lanes that share a column pair (three shuffles).
//   - The kernel waits for its predecessor at its top (griddepcontrol.wait) and lets its successor come up at
//     once (griddepcontrol.launch_dependents): launched as a programmatic dependent it is resident, barriers
//     initialised, when the kernel before it ends.  Nothing is read or written before the wait, so this is
//     safe behind any kernel.
//   - The combine is inside: a CTA that holds a part of a split (sequence, kv head) stores its partial, fences,
//     and adds one to the item's arrival counter; the CTA that arrives last merges the parts (two round trips
//     to L2) and writes the rows.  No CTA waits for another.
//   - With k_new / v_new given, the warp that owns a sequence's last page puts the token's new row into the
//     tile in shared memory (the tile arrives with whatever the slot held) and stores it to the pool; the
//     lengths move forward once every CTA has read them (a counter in the prologue tells the last reader).
//
// The template parameter KV names the cache.  Compiled a second time (KV = E4M3) the kernel serves an E4M3 cache (arb_decode_step_e4m3: the token
// of a quantised draft).  A page tile is 2 KB of codes; the consumer warp that owns it widens it to f16 (exact) into
// a tile of its own in shared memory, laid out like a bf16 tile, frees the ring stage at once, and runs the same
// fragment loads and MMAs on f16 operands (q converted bf16 -> f16, P rounded to f16).  The token's new rows are
// quantised by the warp that patches them in (x * inv_scale, nearest code, saturating: the arithmetic of
// arb_kv_append_e4m3), stored to the pool as codes and patched into the widened tile.
// A third time (KV = 4-bit; arb_decode_step_i4) it serves a cache of 4-bit codes with one fp32 scale per (token, kv head)
// row: a stage is 1 KB of codes and the rows' 16 scales; the consumer warp widens the codes to bf16 (exact), keeps the
// scales of its two keys in registers, multiplies them into the scores and into the weights, and runs the bf16 MMAs; the
// token's rows are quantised in the kernel (row max by shuffles, IEEE divisions, nearest with ties to even).
#include "arb_decode_tc.cuh"

namespace arb {

namespace {

constexpr int kCW = 8;                        // consumer warps
constexpr int kCT = kCW * 32;                 // consumer threads
constexpr int kProdWarp = kCW;                // the producer warp
constexpr int kAuxWarp = kCW + 1;             // bookkeeping: length update, rows of refused sequences
constexpr int kNT = kCT + 64;
constexpr int kTileBytes = kPage * kD * 2;    // 4 KB: one (page, kv head) tile of K or of V
constexpr int kHalfTile = kTileBytes / 2;
constexpr int kCodeTileBytes = kPage * kD;    // 2 KB: the same tile of an E4M3 cache
constexpr int kI4CodeBytes = kPage * kD / 2;  // 1 KB: the same tile of a 4-bit cache (16 rows x 64 bytes, not swizzled) ...
constexpr int kI4ScaleBytes = kPage * 4;      // ... followed by the 16 fp32 scales of its rows
constexpr int kI4StageBytes = 1152;           // both, rounded up to 128
enum { kKvBf16 = 0, kKvE4m3 = 1, kKvI4 = 2 }; // the cache a kernel instance reads
constexpr int kBatch = 32;                    // producer lanes issuing side by side
constexpr int kParked = 2;                    // segment results parked in shared memory before they are written
constexpr int kOStride = kD + 4;              // floats between two heads of a warp record (spreads the banks)
// What a boundary costs is time (the warps meet, a second arrival, perhaps a second merge), a few microseconds
// whatever the call's size: as pages it is the CTA's even share, but no more than this many.
constexpr int kBoundaryCap = 32;
// Hints for the next call: every CTA leaves the pool rows of the first kHintPages page tiles of its range in a record
// of the context.  The next call of the same shape asks for those tiles into L2 before it waits for its predecessor
// (the bookkeeping warp does, off every other warp's path): in a chain of dependent calls the bytes of call n + 1
// cross from HBM while call n is in its latency-bound tail.  A prefetch is a hint: rows are range-checked, a stale or
// foreign record costs some bandwidth and nothing else, and every real read comes after the wait.
constexpr int kHintPages = 64;
constexpr int kHintStride = kHintPages + 4;   // [tag, count, -, -, rows ...]

struct StepArgs {
    const char *q;
    const char *k_new, *v_new;   // [rows, Hkv, D]; null: no cache write, seq_lens already count the token
    char *k_pool, *v_pool;
    const int32_t *block_table;
    int32_t *seq_lens;
    const int32_t *q_lens;
    char *out;
    float *part_o;     // [slots][G][D]
    float *part_ml;    // [slots][GP][2]
    int *counters;     // [batch * Hkv] arrival counters, zero between calls
    int *lens_counter; // CTAs that have read the lengths, zero between calls
    int *hint;         // [grid][kHintStride] the page tiles each CTA streamed last time (see kHintPages)
    int hint_tag;      // shape of this call; a record with another tag is ignored
    uint32_t *status;
    int batch, Hq, Hkv, num_pages, max_pages;
    int whole_rows;    // the tensor maps are 3-D: one copy per page tile instead of one per half
    int slots;         // partial slots in the workspace region (bounds-check build)
    int rows;          // rows of q and out
    int min_chunk;     // fewest pages worth giving a CTA
    int boundary_pct;  // cost of a (sequence, kv head) boundary inside a CTA's range: percent of min(even share, kBoundaryCap) pages
    float scale_log2;  // softmax scale (times the key scale of an E4M3 cache) * log2(e)
    float v_scale;     // value scale of an E4M3 cache, 1 otherwise
    float k_inv_scale, v_inv_scale;   // E4M3 cache with a cache write: code = e4m3(x * inv_scale)
    float *k_scales, *v_scales;       // 4-bit cache: the scale pools [num_pages, Hkv, 16]
};

template <int STAGES>
struct Tail {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t merge_bar;   // the bulk copies of a merge
    int abort;
    int last[kParked];
};

template <int G>
struct Cfg {
    static constexpr int GP = (G + 3) / 4 * 4;
    static constexpr int WREC = 2 * 8 + G * kOStride;     // warp record: [m[8] | l[8] | o[G][kOStride]]
    static constexpr int REC = 2 * GP + G * kD;           // parked record: [m[GP] | l[GP] | o[G][D]]
    static constexpr int OSM_BYTES = kCW * WREC * 4;
    static constexpr int PARK_BYTES = kParked * REC * 4;
};

// E4M3: the ring holds tiles of codes; every consumer warp has a widened K tile and a widened V tile of its own
template <int G, int STAGES, int KV>
size_t smem_bytes(int batch) {
    using C = Cfg<G>;
    const size_t wide = (size_t)kCW * 2 * kTileBytes;
    const size_t tiles = KV == kKvE4m3 ? (size_t)STAGES * kCodeTileBytes + wide
                         : KV == kKvI4 ? (size_t)STAGES * kI4StageBytes + wide : (size_t)STAGES * kTileBytes;
    return 1024 + tiles + C::OSM_BYTES + C::PARK_BYTES + sizeof(Tail<STAGES>) + sizeof(int) * (4 * (size_t)batch + 3 + 8);
}

struct Parked {
    int bk, nparts, c_first;
    size_t out_base;
};

struct Pending {   // a split (sequence, kv head) this CTA was the last to reach
    int slot0, nparts;
    size_t out_base;
};

__device__ __forceinline__ uint32_t tile_off(int r, int c) {   // 16-byte chunk c of row r of a swizzled bf16 tile
    return (uint32_t)((c >> 3) * kHalfTile + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float2 unpack_f16(uint32_t v) {
    float lo, hi;
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, h;\n\t}" : "=f"(lo), "=f"(hi) : "r"(v));
    return make_float2(lo, hi);
}
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t v) {
    return pack_f16(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
}
// two E4M3 codes (a 16-bit pair) -> f16x2, exact; the low byte lands in the low half
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint16_t v) {
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(v));
    return r;
}
// two values -> two E4M3 codes (nearest, ties to even, saturating); lo lands in the low byte
__device__ __forceinline__ uint32_t e4m3x2_from_f32(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
// A warp widens a tile of codes (16 rows x 128 B, 128-byte swizzle) into an f16 tile laid out like a bf16 tile:
// lane (r, h) = (lane / 2, lane % 2) takes the 64 codes of half h of row r, four 16-byte pieces in, eight out.
__device__ __forceinline__ void widen_tile(const char *codes, char *dst, int lane) {
    const int r = lane >> 1, h = lane & 1;
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) {
        const int c = 4 * h + c4;
        const uint4 cd = *reinterpret_cast<const uint4 *>(codes + r * 128 + ((c ^ (r & 7)) << 4));
        uint4 lo, hi;
        lo.x = e4m3x2_to_f16x2((uint16_t)cd.x); lo.y = e4m3x2_to_f16x2((uint16_t)(cd.x >> 16));
        lo.z = e4m3x2_to_f16x2((uint16_t)cd.y); lo.w = e4m3x2_to_f16x2((uint16_t)(cd.y >> 16));
        hi.x = e4m3x2_to_f16x2((uint16_t)cd.z); hi.y = e4m3x2_to_f16x2((uint16_t)(cd.z >> 16));
        hi.z = e4m3x2_to_f16x2((uint16_t)cd.w); hi.w = e4m3x2_to_f16x2((uint16_t)(cd.w >> 16));
        *reinterpret_cast<uint4 *>(dst + tile_off(r, 2 * c)) = lo;
        *reinterpret_cast<uint4 *>(dst + tile_off(r, 2 * c + 1)) = hi;
    }
}

// 4-bit cache: a 32-bit word holds 8 dimensions as nibbles (code + 8), nibble i and nibble i + 4 being the neighbouring
// dimensions 2i and 2i + 1.  (word >> 4i) & 0x000F000F | 0x43004300 is the bf16 pair (128 + nibble i, 128 + nibble i + 4)
// -- a bf16 with exponent 2^7 counts in ones -- and subtracting 136 leaves the two codes, exactly.
__device__ __forceinline__ uint4 i4_word_to_bf16x8(uint32_t w) {
    uint32_t r[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t biased = ((w >> (4 * i)) & 0x000F000Fu) | 0x43004300u;
        asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(r[i]) : "r"(biased), "r"(0x3F803F80u), "r"(0xC308C308u));
    }
    return make_uint4(r[0], r[1], r[2], r[3]);
}
// A warp widens a tile of 4-bit codes (16 rows x 64 bytes, plain row-major) into a bf16 tile laid out like a tile of
// a bf16 cache: lane (r, h) = (lane / 2, lane % 2) takes the 32 bytes (64 dimensions) of half h of row r.
__device__ __forceinline__ void widen_tile_i4(const char *codes, char *dst, int lane) {
    const int r = lane >> 1, h = lane & 1;
    const uint4 c0 = *reinterpret_cast<const uint4 *>(codes + r * 64 + h * 32);
    const uint4 c1 = *reinterpret_cast<const uint4 *>(codes + r * 64 + h * 32 + 16);
    const uint32_t w[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) *reinterpret_cast<uint4 *>(dst + tile_off(r, 8 * h + i)) = i4_word_to_bf16x8(w[i]);
}

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// A sequence takes part when it decodes (q_len 1) and its length after the token fits the block table.
// L0: the length the call finds in seq_lens; with a cache write the token lands at position L0.
template <bool APPEND>
__device__ __forceinline__ bool step_ok(int n, int L0, int max_pages) {
    if (n != 1) return false;
    const long long L = (long long)L0 + (APPEND ? 1 : 0);
    return L0 >= (APPEND ? 0 : 1) && L <= (long long)max_pages * kPage;
}

// a / b for 0 <= a, 0 < b: through the float reciprocal with a correction step while a is exactly representable
// (the plan sits on every CTA's path to its first copy, and an integer division is some forty dependent instructions)
__device__ __forceinline__ int fast_div(int a, int b) {
    if (a >= (1 << 24)) return a / b;
    int q = __float2int_rz(__fdividef((float)a, (float)b));
    const int r = a - q * b;
    if (r < 0) --q; else if (r >= b) ++q;
    return q;
}

// a / b where the quotient is a kv head index (small): a few subtractions beat any division
__device__ __forceinline__ int small_div(int a, int b, int &rem) {
    int q = 0;
    while (a >= b) { a -= b; ++q; }
    rem = a;
    return q;
}

// The cut of the flat (sequence, kv head, page) list into per-CTA ranges.  A CTA whose range crosses from one
// (sequence, kv head) into the next pays for it (the warps meet, their records are merged, the next q is
// loaded), and it then tends to be the last to arrive at both items and merges both.  So a boundary counts as
// `pen` pages of work: the list is cut evenly in a padded coordinate in which every item is preceded by `pen`
// virtual pages.  Item j (in list order) with real range [s, s + n) occupies [s + j pen, s + (j + 1) pen + n) there,
// its real pages the last n of them.  Everything after the cut works in real coordinates.
struct Plan {
    const int *pref;   // [B + 1] real flat start of sequence b (pages times kv heads)
    const int *act;    // [B + 1] sequences before b that take part
    const int *slen;   // [B] length of sequence b (with the new token)
    int B, Hkv, pen, chunk, total_padded;

    __device__ __forceinline__ int pages_of(int b) const { return pref[b + 1] != pref[b] ? (slen[b] + kPage - 1) / kPage : 0; }
    __device__ __forceinline__ int padded_start(int b) const { return pref[b] + pen * Hkv * act[b]; }
    // real flat position of padded position r inside sequence b (a virtual page maps to the first real page behind it)
    __device__ __forceinline__ int real_in(int b, long long r) const {
        const int pages = pages_of(b);
        int o2;
        const int kvh = small_div((int)r - padded_start(b), pages + pen, o2);
        return pref[b] + kvh * pages + max(0, o2 - pen);
    }
    // the CTA that holds real page `pg` of item (b, kvh)
    __device__ __forceinline__ int cta_of(int b, int kvh, int pages, int pg) const {
        return fast_div(padded_start(b) + kvh * (pages + pen) + pen + pg, chunk);
    }
    // the sequence that holds real flat position r, walking up from a sequence known to start at or before r
    __device__ __forceinline__ int seq_of(int r, int b) const {
        while (b + 1 < B && pref[b + 1] <= r) ++b;
        return b;
    }
};

// Next segment of the real flat range [cur, r1); `b` is the sequence of the segment before (or of r0) and moves along.
__device__ __forceinline__ bool next_segment(int &cur, int r1, int &b, const Plan &pl, Segment &s) {
    if (cur >= r1) return false;
    b = pl.seq_of(cur, b);
    const int pages = pl.pages_of(b);
    int pg0;
    const int kvh = small_div(cur - pl.pref[b], pages, pg0);
    const int s1 = pl.pref[b] + (kvh + 1) * pages;
    const int end = s1 < r1 ? s1 : r1;
    s.b = b;
    s.kvh = kvh;
    s.pg0 = pg0;
    s.pg1 = pg0 + (end - cur);
    s.L = pl.slen[b];
    s.bk = b * pl.Hkv + kvh;
    s.c_first = -1;   // filled in by parts_of when the segment's result is parked
    s.nparts = 0;
    cur = end;
    return true;
}

__device__ __forceinline__ void parts_of(const Plan &pl, Segment &s) {
    const int pages = pl.pages_of(s.b);
    s.c_first = pl.cta_of(s.b, s.kvh, pages, 0);
    s.nparts = pl.cta_of(s.b, s.kvh, pages, pages - 1) - s.c_first + 1;
}

template <int G, int STAGES, bool APPEND, int KV>
__global__ void __launch_bounds__(kNT, 1)
decode_step_kernel(const StepArgs a, const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map) {
    using C = Cfg<G>;
    using Tail = arb::Tail<STAGES>;
    constexpr int GP = C::GP, WREC = C::WREC, REC = C::REC;
    constexpr bool E4M3 = KV == kKvE4m3, I4 = KV == kKvI4, WIDE = KV != kKvBf16;
    constexpr int kStageBytes = E4M3 ? kCodeTileBytes : I4 ? kI4StageBytes : kTileBytes;   // a ring stage
    constexpr int kTxBytes = I4 ? kI4CodeBytes + kI4ScaleBytes : kStageBytes;               // what the copies of a stage bring
    constexpr int kRowBytes = E4M3 ? kD : I4 ? kD / 2 : kD * 2;         // bytes of a cache row
    constexpr int kWideBytes = WIDE ? kCW * 2 * kTileBytes : 0;         // codes: a widened K and V tile per consumer warp
    constexpr int kRingBytes = STAGES * kStageBytes + kWideBytes;       // the merges use all of it
    static_assert(G >= 1 && G <= 8, "the group's heads are the 8 columns of the tile");
    static_assert(STAGES % (2 * kCW) == 0 && kBatch <= STAGES, "a ring stage always belongs to the same warp of a segment");

    extern __shared__ char smem_raw[];
    char *base = reinterpret_cast<char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    char *ring = base;
    float *osm = reinterpret_cast<float *>(base + kRingBytes);
    float *park = reinterpret_cast<float *>(base + kRingBytes + C::OSM_BYTES);
    Tail *tail = reinterpret_cast<Tail *>(base + kRingBytes + C::OSM_BYTES + C::PARK_BYTES);
    int *pref = reinterpret_cast<int *>(tail + 1);
    int *row0 = pref + a.batch + 1;
    int *act = row0 + a.batch + 1;
    int *slen = act + a.batch + 1;
    int *plan_s = slen + a.batch;    // [8]: this CTA's cut, worked out by warp 0

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.batch, Hkv = a.Hkv;

    let_successor_start();
    if (tid == kCT) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&k_map)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&v_map)) : "memory");
    }
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&tail->full[s], 1);
            mbar_init(&tail->empty[s], 1);
        }
        mbar_init(&tail->merge_bar, 1);
        tail->abort = 0;
        mbar_fence_init();
        pref[0] = 0;
        row0[0] = 0;
        act[0] = 0;
    }
    int *hint = a.hint + (size_t)blockIdx.x * kHintStride;
    if (warp == kAuxWarp) {
        // the tiles this CTA streamed last time are asked into L2 while the predecessor is still at work
        const int tag = __ldcg(hint), cnt = __ldcg(hint + 1);
        if (tag == a.hint_tag) {
            const int n = min(cnt, kHintPages);
            for (int i = lane; i < n; i += 32) {
                const int row = __ldcg(hint + 4 + i);
                if ((unsigned)row < (unsigned)(a.num_pages * Hkv * kPage)) {
                    const size_t off = (size_t)row * kRowBytes;
                    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a.k_pool + off), "r"(kPage * kRowBytes) : "memory");
                    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a.v_pool + off), "r"(kPage * kRowBytes) : "memory");
                }
            }
        }
    }
    // Everything below may read what the kernel before this one wrote (lengths, q, new rows, the cache).
    wait_for_predecessor();

    // ---- prologue: lengths -> page counts and q row offsets (the bookkeeping warp joins when the plan is there) ----
    constexpr int kPT = kNT - 32;   // threads of the prologue: all but the bookkeeping warp
    if (warp == kAuxWarp) {
        asm volatile("bar.sync 3, %0;" ::"r"(kNT) : "memory");
    } else {
    for (int b = tid; b < B; b += kPT) {
        const int n = a.q_lens[b], L0 = a.seq_lens[b];
        const bool ok = step_ok<APPEND>(n, L0, a.max_pages);
        const int L = L0 + (APPEND ? 1 : 0);
        pref[b + 1] = ok ? (L + kPage - 1) / kPage * Hkv : 0;
        row0[b + 1] = n > 0 ? n : 0;
        act[b + 1] = ok ? 1 : 0;
        slen[b] = L;
    }
    named_barrier(2, kPT);
    if (warp == 0) {
        int carry_p = 0, carry_r = 0, carry_a = 0;
        for (int b0 = 0; b0 < B; b0 += 32) {
            const int b = b0 + lane;
            int vp = b < B ? pref[b + 1] : 0;
            int vr = b < B ? row0[b + 1] : 0;
            int va = b < B ? act[b + 1] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int tp = __shfl_up_sync(0xffffffffu, vp, off);
                const int tr = __shfl_up_sync(0xffffffffu, vr, off);
                const int ta = __shfl_up_sync(0xffffffffu, va, off);
                if (lane >= off) { vp += tp; vr += tr; va += ta; }
            }
            if (b < B) { pref[b + 1] = vp + carry_p; row0[b + 1] = vr + carry_r; act[b + 1] = va + carry_a; }
            carry_p += __shfl_sync(0xffffffffu, vp, 31);
            carry_r += __shfl_sync(0xffffffffu, vr, 31);
            carry_a += __shfl_sync(0xffffffffu, va, 31);
        }
        // The cut, while the warp is at it: an even share of the padded list per CTA; both ends of this CTA's range
        // are looked up with one ballot per 32 sequences (the padded starts ascend, so the sequence that holds a
        // position is the last one that starts at or before it) instead of a search in every warp.
        __syncwarp();
        Plan pl;
        pl.pref = pref; pl.act = act; pl.slen = slen; pl.B = B; pl.Hkv = Hkv;
        const int total = pref[B], items = act[B] * Hkv, grid = (int)gridDim.x;
        const int even = max(a.min_chunk, fast_div(total + grid - 1, grid));
        pl.pen = items > 1 ? (min(even, kBoundaryCap) * a.boundary_pct + 99) / 100 : 0;
        pl.total_padded = total + pl.pen * items;
        pl.chunk = max(a.min_chunk, fast_div(pl.total_padded + grid - 1, grid));
        int ends[2], seq0 = 0;
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            const long long t = (long long)(blockIdx.x + w) * pl.chunk;
            int best = 0;
            for (int b0 = 0; b0 < B; b0 += 32) {
                const int b = b0 + lane;
                const unsigned mask = __ballot_sync(0xffffffffu, b < B && pl.padded_start(b) <= t);
                if (mask) best = b0 + 31 - __clz(mask);
            }
            ends[w] = t >= pl.total_padded ? total : pl.real_in(best, t);
            if (w == 0) seq0 = best;
        }
        if (lane == 0) {
            plan_s[0] = ends[0];
            plan_s[1] = ends[1];
            plan_s[2] = pl.pen;
            plan_s[3] = pl.chunk;
            plan_s[4] = seq0;
        }
    }
    named_barrier(2, kPT);
    asm volatile("bar.arrive 3, %0;" ::"r"(kNT) : "memory");   // the plan is there: the bookkeeping warp may go on
    }

    if (warp == kAuxWarp) {
        // ================================ bookkeeping warp ==========================================
        // Lengths: every CTA has its copy in shared memory by now.  The CTA whose count completes the grid
        // knows that nobody will read seq_lens again and moves them forward: for the sequences that take part
        // and whose new row has a page inside the pool to go to (the same test the writer of the row makes).
        if constexpr (APPEND) {
            int last = 0;
            if (lane == 0) last = atomicAdd(a.lens_counter, 1) == (int)gridDim.x - 1;
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                for (int b = lane; b < B; b += 32) {
                    const int L0 = slen[b] - 1;
                    if (step_ok<true>(a.q_lens[b], L0, a.max_pages)) {
                        const int pid = a.block_table[(size_t)b * a.max_pages + L0 / kPage];
                        if ((unsigned)pid < (unsigned)a.num_pages) a.seq_lens[b] = L0 + 1;
                    }
                }
                if (lane == 0) *a.lens_counter = 0;
            }
        }
        // Sequences that were asked to decode but cannot: status bit, rows of zeros.
        if (blockIdx.x == 0) {
            for (int b = 0; b < B; ++b) {
                const int n = row0[b + 1] - row0[b];
                if (n != 1 || pref[b + 1] != pref[b]) continue;
                if (lane == 0) atomicOr(a.status, (uint32_t)ARB_DEV_BAD_SEQ_LEN);
                uint4 *o = reinterpret_cast<uint4 *>(a.out + (size_t)row0[b] * a.Hq * kD * 2);
                for (int i = lane; i < a.Hq * kD * 2 / 16; i += 32) o[i] = make_uint4(0, 0, 0, 0);
            }
        }
        return;
    }

    Plan pl;
    pl.pref = pref;
    pl.act = act;
    pl.slen = slen;
    pl.B = B;
    pl.Hkv = Hkv;
    const int r0 = plan_s[0], r1 = plan_s[1], seq0 = plan_s[4];
    pl.pen = plan_s[2];
    pl.chunk = plan_s[3];
    pl.total_padded = 0;   // only the cut needs it
    if (r0 >= r1) {
        if (tid == 0) hint[1] = 0;   // nothing streamed: nothing to ask for next time
        return;
    }
    volatile int *abort = &tail->abort;

    if (warp == kProdWarp) {
        // ================================ producer warp ==========================================
        // The CTA's flat range of (sequence, kv head, page) triples goes through in groups of 32: lane i finds
        // triple i of the group (a short walk up the prefix table from the range's first sequence) and fetches its block-table entry; the entries
        // of the next group are asked for before the tiles of this one are issued, so that the look-up is off the
        // path after the first group, across sequence boundaries too.  Tiles enter the ring page by page, K then
        // V; lanes 0 .. kBatch-1 each own one stage at a time.
        const int nflat = r1 - r0;
        auto tile_row = [&](int r) -> int {   // first row, in the 2-D view of the pool, of the tile of flat triple r
            const int lo = pl.seq_of(r, seq0);
            const int pages = pl.pages_of(lo);
            int pg;
            const int kvh = small_div(r - pref[lo], pages, pg);
            int pid = ARB_IN_RANGE(a.status, pg, a.max_pages) && ARB_IN_RANGE(a.status, kvh, Hkv)
                          ? a.block_table[(size_t)lo * a.max_pages + pg] : 0;
            if ((unsigned)pid >= (unsigned)a.num_pages) {
                atomicOr(a.status, (uint32_t)ARB_DEV_BAD_PAGE);
                pid = 0;
            }
            return (pid * Hkv + kvh) * kPage;
        };
        uint32_t c = 0;
        int row_next = lane < nflat ? tile_row(r0 + lane) : 0;
        if (lane == 0) {
            hint[0] = a.hint_tag;
            hint[1] = nflat;
        }
        for (int g0 = 0; g0 < nflat; g0 += 32) {
            const int row_cur = row_next;
            if (g0 + lane < min(nflat, kHintPages)) hint[4 + g0 + lane] = row_cur;
            const int ntiles = 2 * min(32, nflat - g0);
#pragma unroll 1
            for (int i0 = 0; i0 < ntiles; i0 += kBatch) {
                // the next group's look-up goes out behind this group's first copies, not in front of them
                if (i0 == kBatch && g0 + 32 + lane < nflat) row_next = tile_row(r0 + g0 + 32 + lane);
                const int i = i0 + lane;
                const int row = __shfl_sync(0xffffffffu, row_cur, (i >> 1) & 31);
                const uint32_t cc = c + i, st = cc % STAGES, par = (cc / STAGES) & 1u;
                const CUtensorMap *map = (i & 1) ? &v_map : &k_map;
                // The lanes wait for 32 different stages.  A blocking wait would put the whole warp to sleep until its
                // time limit whenever one stage is not free yet, and copies for stages that are would go out late, in
                // clumps (seen: 0.7 us apart).  So the warp polls, converged: every round each lane tests its own
                // stage without blocking and issues its copy the moment the stage is free.
                bool pending = i < ntiles && ARB_IN_RANGE(a.status, row, (long long)a.num_pages * Hkv * kPage);
                const long long t0 = clock64();
                while (__any_sync(0xffffffffu, pending)) {
                    if (pending && mbar_test_wait(&tail->empty[st], par ^ 1u)) {
                        mbar_arrive_expect_tx(&tail->full[st], kTxBytes);
                        if constexpr (I4) {   // 16 rows x 64 bytes of codes, then the rows' 16 scales
                            tma_box_load(ring + st * kStageBytes, map, 0, row, &tail->full[st]);
                            bulk_load(ring + st * kStageBytes + kI4CodeBytes, ((i & 1) ? a.v_scales : a.k_scales) + row,
                                      kI4ScaleBytes, &tail->full[st]);
                        } else if constexpr (E4M3) {
                            tma_box_load(ring + st * kStageBytes, map, 0, row, &tail->full[st]);   // 16 rows x 128 codes
                        } else if (a.whole_rows) {
                            tma_box_load3(ring + st * kTileBytes, map, 0, row, 0, &tail->full[st]);
                        } else {
                            tma_box_load(ring + st * kTileBytes, map, 0, row, &tail->full[st]);
                            tma_box_load(ring + st * kTileBytes + kHalfTile, map, 64, row, &tail->full[st]);
                        }
                        pending = false;
                    }
                    if (pending && (*abort || clock64() - t0 > kWaitCycles)) {   // give up, like every other wait
                        if (!*abort) {
                            *abort = 1;
                            atomicOr(a.status, (uint32_t)ARB_DEV_WAIT_TIMEOUT);
                        }
                        pending = false;
                    }
                }
            }
            if (ntiles <= kBatch && g0 + 32 + lane < nflat) row_next = tile_row(r0 + g0 + 32 + lane);
            c += ntiles;
        }
        // After a timeout the consumers may have left copies unconsumed: wait (bounded) for the last ring's
        // worth, so that no copy is in flight into this CTA's shared memory when it exits.
        if (lane == 0 && *abort) {
            const uint32_t n = c < (uint32_t)STAGES ? c : (uint32_t)STAGES;
            for (uint32_t i = 0; i < n; ++i) {
                const uint32_t cc = c - 1 - i;
                const long long t0 = clock64();
                while (!mbar_try_wait(&tail->full[cc % STAGES], (cc / STAGES) & 1u) && clock64() - t0 < (1ll << 24)) {
                }
            }
        }
        return;
    }

    // ==================================== consumer warps ==========================================
    const int gq = lane >> 2, tq = lane & 3;   // fragment coordinates
    const bool head_ok = gq < G;               // as a B-fragment column: this lane's head is a real one
    const int h0 = 2 * tq, h1 = 2 * tq + 1;    // as accumulator columns: the two heads this lane holds
    uint32_t seg_base = 0;                     // ring counter of the segment's first tile
    int cur = r0;
    Segment s;
    int n_parked = 0, pend_n = 0;
    Parked pk[kParked];
    Pending pend[2];

    // Writes what is parked: whole (sequence, kv head)s to `out`, parts of split ones to the workspace, followed
    // by the arrival at the item's counter.  The last to arrive notes the merge for the epilogue.
    auto flush = [&]() {
        bool any_multi = false;
        for (int j = 0; j < n_parked; ++j) {
            const float *rec = park + j * REC;
            if (pk[j].nparts == 1) {
                if (!ARB_IN_RANGE(a.status, pk[j].out_base + G * kD - 1, (size_t)a.rows * a.Hq * kD)) continue;
                for (int idx = tid; idx < G * kD; idx += kCT)
                    reinterpret_cast<__nv_bfloat16 *>(a.out)[pk[j].out_base + idx] =
                        __float2bfloat16_rn(rec[2 * GP + idx] / rec[GP + idx / kD]);
            } else {
                any_multi = true;
                const size_t slot = (size_t)pk[j].bk + blockIdx.x;
                if (!ARB_IN_RANGE(a.status, slot, a.slots)) continue;
                for (int idx = tid; idx < G * kD / 4; idx += kCT)
                    reinterpret_cast<float4 *>(a.part_o + slot * G * kD)[idx] =
                        reinterpret_cast<const float4 *>(rec + 2 * GP)[idx];
                if (tid < G) {
                    a.part_ml[(slot * GP + tid) * 2 + 0] = rec[tid];
                    a.part_ml[(slot * GP + tid) * 2 + 1] = rec[GP + tid];
                }
            }
        }
        if (any_multi) {
            __threadfence();
            asm volatile("fence.proxy.async;" ::: "memory");   // the partials are read back through bulk copies
            named_barrier(1, kCT);
            if (tid == 0) {
                int old[kParked];
                for (int j = 0; j < n_parked; ++j)
                    old[j] = pk[j].nparts > 1 ? atomicAdd(&a.counters[pk[j].bk], 1) : -1;
                for (int j = 0; j < n_parked; ++j) {
                    const int last = pk[j].nparts > 1 && old[j] == pk[j].nparts - 1;
                    if (last) a.counters[pk[j].bk] = 0;   // everyone has arrived: ready for the next call
                    tail->last[j] = last;
                }
                __threadfence();
            }
            named_barrier(1, kCT);
            for (int j = 0; j < n_parked; ++j) {
                if (pk[j].nparts > 1 && tail->last[j] && pend_n < 2) {
                    pend[pend_n].slot0 = pk[j].bk + pk[j].c_first;
                    pend[pend_n].nparts = pk[j].nparts;
                    pend[pend_n].out_base = pk[j].out_base;
                    ++pend_n;
                }
            }
        }
        named_barrier(1, kCT);   // parking slots and flags are free again
        n_parked = 0;
    };

    // B fragments of q^T (128 dims x 8 heads): k-slice ks holds dims 16 ks + 2 tq, + 1 and + 8 of head gq.  The
    // fragments of the next segment are asked for while this one streams.
    uint32_t qb[8][2], qn[8][2];
    auto load_q = [&](const Segment &g, uint32_t (&dst)[8][2]) {
        const char *qh = a.q + ((size_t)row0[g.b] * a.Hq + g.kvh * G + (head_ok ? gq : 0)) * kD * 2;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            dst[ks][0] = head_ok ? __ldg(reinterpret_cast<const uint32_t *>(qh + ks * 32 + tq * 4)) : 0u;
            dst[ks][1] = head_ok ? __ldg(reinterpret_cast<const uint32_t *>(qh + ks * 32 + 16 + tq * 4)) : 0u;
            if constexpr (E4M3) {   // the operands of one MMA share a type: q goes to f16 like the widened codes
                dst[ks][0] = bf16x2_to_f16x2(dst[ks][0]);
                dst[ks][1] = bf16x2_to_f16x2(dst[ks][1]);
            }
        }
    };
    // E4M3: this warp's widened K and V tiles
    char *wide_k = ring + STAGES * kStageBytes + warp * 2 * kTileBytes, *wide_v = wide_k + kTileBytes;
    Segment s_next;
    int seq_at = seq0;
    bool have = next_segment(cur, r1, seq_at, pl, s);
    if (have) load_q(s, qb);
    while (have) {
        const bool have_next = next_segment(cur, r1, seq_at, pl, s_next);
        if (have_next) load_q(s_next, qn);
        const int qrow = row0[s.b];
        // The token's new row: it belongs in slot (L - 1) mod 16 of the sequence's last page.  The warp that owns
        // that page fetches the row (lanes 0..15: K, lanes 16..31: V, 16 bytes each), stores it to the pool and
        // patches it into the tiles when they arrive.
        const int seg_pages = s.pg1 - s.pg0;
        const int last_pg = (s.L - 1) / kPage, new_slot = (s.L - 1) % kPage;
        bool patch = false;
        uint4 new_row = make_uint4(0, 0, 0, 0);
        float new_scale = 0.f;   // 4-bit cache: the scale of the new K row (lanes 0..15) / V row (lanes 16..31)
        if constexpr (APPEND) {
            patch = last_pg >= s.pg0 && last_pg < s.pg1 && ((last_pg - s.pg0) % kCW) == warp;
            if (patch) {
                const char *src = (lane < 16 ? a.k_new : a.v_new) + ((size_t)qrow * Hkv + s.kvh) * kD * 2 + (lane & 15) * 16;
                new_row = __ldg(reinterpret_cast<const uint4 *>(src));
                const int pid = a.block_table[(size_t)s.b * a.max_pages + last_pg];
                const bool store = (unsigned)pid < (unsigned)a.num_pages && ARB_IN_RANGE(a.status, qrow, a.rows);
                // (a page outside the pool: the producer has raised ARB_DEV_BAD_PAGE; nothing is written)
                if constexpr (I4) {
                    // The row's scale is max|x| / 7 over its 128 values (16 lanes), the codes rint(x * (7 / max|x|))
                    // clamped to -7 .. 7, both divisions IEEE; this lane's eight values are one word of nibbles
                    // (code + 8; nibbles 0..7 = dimensions 0, 2, 4, 6, 1, 3, 5, 7 of the eight).
                    const uint32_t w[4] = {new_row.x, new_row.y, new_row.z, new_row.w};
                    float x[8];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        x[2 * j] = __uint_as_float(w[j] << 16);
                        x[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
                    }
                    float m = 0.f;
#pragma unroll
                    for (int j = 0; j < 8; ++j) m = fmaxf(m, fabsf(x[j]));
#pragma unroll
                    for (int off = 8; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
                    new_scale = m > 0.f ? __fdiv_rn(m, 7.f) : 0.f;
                    const float inv = m > 0.f ? __fdiv_rn(7.f, m) : 0.f;
                    uint32_t word = 0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int c = max(-7, min(7, __float2int_rn(__fmul_rn(x[j], inv))));
                        word |= (uint32_t)(c + 8) << (4 * ((j >> 1) + 4 * (j & 1)));
                    }
                    if (store) {
                        const size_t slot_row = ((size_t)pid * Hkv + s.kvh) * kPage + new_slot;
                        *reinterpret_cast<uint32_t *>((lane < 16 ? a.k_pool : a.v_pool) + slot_row * (kD / 2) + (lane & 15) * 4) = word;
                        if ((lane & 15) == 0) (lane < 16 ? a.k_scales : a.v_scales)[slot_row] = new_scale;
                    }
                    new_row = i4_word_to_bf16x8(word);
                } else if constexpr (E4M3) {
                    // quantise this lane's eight values as arb_kv_append_e4m3 does (x * inv_scale in fp32, nearest code,
                    // ties to even, saturating), store the codes, and keep their widened form for the tile
                    const float inv = lane < 16 ? a.k_inv_scale : a.v_inv_scale;
                    const uint32_t w[4] = {new_row.x, new_row.y, new_row.z, new_row.w};
                    uint32_t code[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        code[j] = e4m3x2_from_f32(__uint_as_float(w[j] << 16) * inv, __uint_as_float(w[j] & 0xffff0000u) * inv);
                    if (store) {
                        char *dst = (lane < 16 ? a.k_pool : a.v_pool) +
                                    (((size_t)pid * Hkv + s.kvh) * kPage + new_slot) * kD + (lane & 15) * 8;
                        *reinterpret_cast<uint2 *>(dst) = make_uint2(code[0] | (code[1] << 16), code[2] | (code[3] << 16));
                    }
                    new_row = make_uint4(e4m3x2_to_f16x2((uint16_t)code[0]), e4m3x2_to_f16x2((uint16_t)code[1]),
                                         e4m3x2_to_f16x2((uint16_t)code[2]), e4m3x2_to_f16x2((uint16_t)code[3]));
                } else if (store) {
                    char *dst = (lane < 16 ? a.k_pool : a.v_pool) +
                                (((size_t)pid * Hkv + s.kvh) * kPage + new_slot) * (kD * 2) + (lane & 15) * 16;
                    *reinterpret_cast<uint4 *>(dst) = new_row;
                }
            }
        }

        // this lane's columns (heads h0, h1): running max (the same in the 8 lanes of a column pair), its share of
        // the sum, and 8 m-tiles of O^T: o[mt][0..1] = dim 16 mt + gq of heads h0, h1; o[mt][2..3] = dim + 8
        float m_run0 = -INFINITY, m_run1 = -INFINITY, l_run0 = 0.f, l_run1 = 0.f;
        float o[8][4];
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }

        for (int gi = warp; gi < seg_pages; gi += kCW) {
            const int pg = s.pg0 + gi;
            const int ntok = min(s.L - pg * kPage, kPage);
            const bool patch_here = APPEND && patch && pg == last_pg;
            const uint32_t ck = seg_base + 2u * (uint32_t)gi;

            // ---- S^T = K q^T: 16 keys x 8 heads, two accumulators so that the chain is four deep ----------
            float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
            float ksc0 = 1.f, ksc1 = 1.f, vsc0 = 1.f, vsc1 = 1.f;   // 4-bit cache: the scales of keys gq and gq + 8
            {
                const uint32_t st = ck % STAGES, par = (ck / STAGES) & 1u;
                mbar_wait(&tail->full[st], par, abort, a.status);
                char *tile_p = ring + st * kStageBytes;
                if constexpr (WIDE) {   // widen into this warp's tile; the ring stage is free at once
                    if constexpr (I4) {
                        widen_tile_i4(tile_p, wide_k, lane);
                        const float *sc = reinterpret_cast<const float *>(tile_p + kI4CodeBytes);
                        ksc0 = sc[gq];
                        ksc1 = sc[gq + 8];
                    } else {
                        widen_tile(tile_p, wide_k, lane);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tail->empty[st]);
                    tile_p = wide_k;
                }
                if (patch_here) {
                    if (lane < 16) *reinterpret_cast<uint4 *>(tile_p + tile_off(new_slot, lane)) = new_row;
                    if constexpr (I4) {
                        const float ns = __shfl_sync(0xffffffffu, new_scale, 0);
                        if (gq == new_slot) ksc0 = ns;
                        if (gq + 8 == new_slot) ksc1 = ns;
                    }
                    __syncwarp();
                }
                const uint32_t tile = smem_u32(tile_p);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    uint32_t af[4];   // rows: keys; matrices: (keys 0-7 | 8-15) x (dims 16 ks + 0-7 | 8-15)
                    ldmatrix_x4(tile + tile_off((lane & 7) + ((lane >> 3) & 1) * 8, 2 * ks + (lane >> 4)), af);
                    if (ks & 1) mma_16816<E4M3>(sb, af, qb[ks][0], qb[ks][1]);
                    else mma_16816<E4M3>(sa, af, qb[ks][0], qb[ks][1]);
                }
                __syncwarp();
                if constexpr (!WIDE) {
                    if (patch_here) fence_proxy_async_smem();   // the stage's next writer is the TMA unit
                    if (lane == 0) mbar_arrive(&tail->empty[st]);
                }
            }
            if constexpr (I4) {   // a key is scale * code: the scores of keys gq and gq + 8 take their rows' scales
                sa[0] *= ksc0; sa[1] *= ksc0; sb[0] *= ksc0; sb[1] *= ksc0;
                sa[2] *= ksc1; sa[3] *= ksc1; sb[2] *= ksc1; sb[3] *= ksc1;
            }

            // ---- online softmax: this lane has keys gq and gq + 8 of heads h0 and h1 -------------------
            const bool k0 = gq < ntok, k1 = gq + 8 < ntok;
            const float s00 = k0 ? (sa[0] + sb[0]) * a.scale_log2 : -INFINITY;
            const float s01 = k0 ? (sa[1] + sb[1]) * a.scale_log2 : -INFINITY;
            const float s10 = k1 ? (sa[2] + sb[2]) * a.scale_log2 : -INFINITY;
            const float s11 = k1 ? (sa[3] + sb[3]) * a.scale_log2 : -INFINITY;
            float mx0 = fmaxf(s00, s10), mx1 = fmaxf(s01, s11);
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
            }
            const float mn0 = fmaxf(m_run0, mx0), mn1 = fmaxf(m_run1, mx1);   // finite: key 0 of the page is visible
            const float f0 = fast_exp2(m_run0 - mn0), f1 = fast_exp2(m_run1 - mn1);   // 0 on the first page
            m_run0 = mn0;
            m_run1 = mn1;
            // P^T, rounded to bf16 (f16 over an E4M3 cache); the sums use the rounded weights, like the tensor core
            const float p00 = fast_exp2(s00 - mn0), p01 = fast_exp2(s01 - mn1);
            const float p10 = fast_exp2(s10 - mn0), p11 = fast_exp2(s11 - mn1);
            uint32_t w0 = E4M3 ? pack_f16(p00, p01) : pack_bf16(p00, p01);   // key gq:     heads h0, h1
            uint32_t w1 = E4M3 ? pack_f16(p10, p11) : pack_bf16(p10, p11);   // key gq + 8
            if constexpr (I4) {   // (the weights that reach the tensor core carry the value scales: packed below)
                l_run0 = fmaf(l_run0, f0, p00 + p10);
                l_run1 = fmaf(l_run1, f1, p01 + p11);
            } else if constexpr (E4M3) {
                const float2 r0 = unpack_f16(w0), r1 = unpack_f16(w1);
                l_run0 = fmaf(l_run0, f0, r0.x + r1.x);
                l_run1 = fmaf(l_run1, f1, r0.y + r1.y);
            } else {
                l_run0 = fmaf(l_run0, f0, __uint_as_float(w0 << 16) + __uint_as_float(w1 << 16));
                l_run1 = fmaf(l_run1, f1, __uint_as_float(w0 & 0xffff0000u) + __uint_as_float(w1 & 0xffff0000u));
            }
            // B fragment of P^T (16 keys x 8 heads): keys 2 tq, + 1 (and + 8) of head gq
            uint32_t pb0 = 0, pb1 = 0;
            if constexpr (!I4) {
                pb0 = movmatrix_trans(w0);
                pb1 = movmatrix_trans(w1);
            }
            if (__any_sync(0xffffffffu, f0 != 1.0f || f1 != 1.0f)) {
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) { o[mt][0] *= f0; o[mt][1] *= f1; o[mt][2] *= f0; o[mt][3] *= f1; }
            }

            // ---- O^T += V^T P^T: 8 m-tiles of 16 dims ---------------------------------------------------
            {
                const uint32_t cv = ck + 1u, st = cv % STAGES, par = (cv / STAGES) & 1u;
                mbar_wait(&tail->full[st], par, abort, a.status);
                char *tile_p = ring + st * kStageBytes;
                if constexpr (WIDE) {
                    if constexpr (I4) {
                        widen_tile_i4(tile_p, wide_v, lane);
                        const float *sc = reinterpret_cast<const float *>(tile_p + kI4CodeBytes);
                        vsc0 = k0 ? sc[gq] : 0.f;        // (the scale of a slot past the sequence end may be anything)
                        vsc1 = k1 ? sc[gq + 8] : 0.f;
                    } else {
                        widen_tile(tile_p, wide_v, lane);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tail->empty[st]);
                    tile_p = wide_v;
                }
                if (patch_here) {
                    if (lane >= 16) *reinterpret_cast<uint4 *>(tile_p + tile_off(new_slot, lane - 16)) = new_row;
                    if constexpr (I4) {
                        const float ns = __shfl_sync(0xffffffffu, new_scale, 16);
                        if (gq == new_slot) vsc0 = ns;
                        if (gq + 8 == new_slot) vsc1 = ns;
                    }
                    __syncwarp();
                }
                if constexpr (I4) {   // a value is scale * code: the weight of a key takes its row's scale
                    w0 = pack_bf16(p00 * vsc0, p01 * vsc0);
                    w1 = pack_bf16(p10 * vsc1, p11 * vsc1);
                    pb0 = movmatrix_trans(w0);
                    pb1 = movmatrix_trans(w1);
                }
                if (ntok < kPage) {
                    // slots past the sequence end may hold anything; they must not reach the tensor core, not even
                    // times zero: blank them in shared memory
                    for (int i = lane; i < (kPage - ntok) * 16; i += 32)
                        *reinterpret_cast<uint4 *>(tile_p + tile_off(ntok + (i >> 4), i & 15)) = make_uint4(0, 0, 0, 0);
                    __syncwarp();
                }
                const uint32_t tile = smem_u32(tile_p);
#pragma unroll
                for (int mt = 0; mt < 8; ++mt) {
                    uint32_t af[4];   // transposed on the way: rows dims (16 mt + 0-7 | 8-15), columns keys (0-7 | 8-15)
                    ldmatrix_x4_trans(tile + tile_off((lane & 7) + (lane >> 4) * 8, 2 * mt + ((lane >> 3) & 1)), af);
                    mma_16816<E4M3>(o[mt], af, pb0, pb1);
                }
                __syncwarp();
                if constexpr (!WIDE) {
                    if (patch_here || ntok < kPage) fence_proxy_async_smem();
                    if (lane == 0) mbar_arrive(&tail->empty[st]);
                }
            }
        }
        seg_base += 2u * (uint32_t)seg_pages;

        // ---- segment end: every warp leaves (max, sum, accumulators); all consumer threads merge them ----
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            l_run0 += __shfl_xor_sync(0xffffffffu, l_run0, off);
            l_run1 += __shfl_xor_sync(0xffffffffu, l_run1, off);
        }
        float *rec = osm + warp * WREC;
        if (gq == 0) {
            rec[h0] = m_run0; rec[h1] = m_run1;
            rec[8 + h0] = l_run0; rec[8 + h1] = l_run1;
        }
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
            const int d = 16 * mt + gq;
            if (h0 < G) { rec[16 + h0 * kOStride + d] = o[mt][0]; rec[16 + h0 * kOStride + d + 8] = o[mt][2]; }
            if (h1 < G) { rec[16 + h1 * kOStride + d] = o[mt][1]; rec[16 + h1 * kOStride + d + 8] = o[mt][3]; }
        }
        if (n_parked == kParked) flush();   // uniform across the consumer threads
        named_barrier(1, kCT);
        float *dst = park + n_parked * REC;
        for (int idx = tid; idx < G * kD; idx += kCT) {
            const int h = idx / kD, d = idx - h * kD;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kCW; ++w) M = fmaxf(M, osm[w * WREC + h]);
            float l = 0.f, acc = 0.f;
#pragma unroll
            for (int w = 0; w < kCW; ++w) {
                const float ff = fast_exp2(osm[w * WREC + h] - M);   // 0 for a warp that had no page
                l = fmaf(ff, osm[w * WREC + 8 + h], l);
                acc = fmaf(ff, osm[w * WREC + 16 + h * kOStride + d], acc);
            }
            dst[2 * GP + idx] = E4M3 ? acc * a.v_scale : acc;   // values of an E4M3 cache are v_scale * code
            if (d == 0) { dst[h] = M; dst[GP + h] = l; }
        }
        parts_of(pl, s);
        pk[n_parked].bk = s.bk;
        pk[n_parked].nparts = s.nparts;
        pk[n_parked].c_first = s.c_first;
        pk[n_parked].out_base = ((size_t)qrow * a.Hq + s.kvh * G) * kD;
        ++n_parked;
        named_barrier(1, kCT);   // warp records are free for the next segment
        s = s_next;
        have = have_next;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) { qb[ks][0] = qn[ks][0]; qb[ks][1] = qn[ks][1]; }
    }
    if (n_parked > 0) flush();

    // ---- merges of the split (sequence, kv head)s this CTA was the last to reach ------------------------
    //     m = max_p m_p,  w_p = 2^(m_p - m),  out = sum_p w_p o_p / sum_p w_p l_p,
    // one 4-dimension piece of the group's G x 128 outputs per thread.  The parts of an item lie in consecutive
    // workspace slots, and the ring is idle by now (every tile has been consumed, the producer issues nothing
    // more): one bulk copy brings the (max, sum) records, one the partial outputs -- a single round trip however
    // many parts there are -- and the sum runs out of shared memory.  More parts than the ring holds go in pieces.
    constexpr int VECS = G * kD / 4;
    constexpr int kPartBytes = G * kD * 4;
    static_assert(VECS <= kCT, "one piece per consumer thread");
    if (pend_n == 0) return;
    // up to two merges, each in its own half of the ring, their first copies in flight together
    const int cap = kRingBytes / pend_n;
    const bool mine = tid < VECS;
    const int e = mine ? tid : 0, eh = e / (kD / 4);
    uint32_t merge_phase = 0;
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    float4 x[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
    int done[2] = {0, 0};
    auto ml_area = [&](int j) -> uint32_t { return ((uint32_t)pend[j].nparts * GP * 8u + 127u) & ~127u; };
    auto per_piece = [&](int j) -> int { return (cap - (int)ml_area(j)) / kPartBytes; };   // >= 6: at most 148 parts of 64-byte records
    auto issue = [&](int j, int p0, uint32_t &bytes_out) {   // thread 0
        const int np = min(per_piece(j), pend[j].nparts - p0);
        const uint32_t bytes = (uint32_t)np * kPartBytes, ml_bytes = (uint32_t)pend[j].nparts * GP * 8u;
        char *dst = ring + j * cap;
        if (p0 == 0) bulk_load(dst, a.part_ml + (size_t)pend[j].slot0 * GP * 2, ml_bytes, &tail->merge_bar);
        bulk_load(dst + ml_area(j), a.part_o + ((size_t)pend[j].slot0 + p0) * G * kD, bytes, &tail->merge_bar);
        bytes_out += bytes + (p0 == 0 ? ml_bytes : 0u);
    };
    auto add_piece = [&](int j, int p0) {
        const float2 *ml_s = reinterpret_cast<const float2 *>(ring + j * cap);
        const float4 *po_s = reinterpret_cast<const float4 *>(ring + j * cap + ml_area(j));
        const int np = min(per_piece(j), pend[j].nparts - p0);
        if (p0 == 0)
            for (int p = 0; p < pend[j].nparts; ++p) m[j] = fmaxf(m[j], ml_s[p * GP + eh].x);
#pragma unroll 4
        for (int p = 0; p < np; ++p) {
            const float2 ml = ml_s[(p0 + p) * GP + eh];
            const float w = fast_exp2(ml.x - m[j]);
            const float4 v = po_s[p * VECS + e];
            l[j] = fmaf(w, ml.y, l[j]);
            x[j].x = fmaf(w, v.x, x[j].x);
            x[j].y = fmaf(w, v.y, x[j].y);
            x[j].z = fmaf(w, v.z, x[j].z);
            x[j].w = fmaf(w, v.w, x[j].w);
        }
        done[j] = p0 + np;
    };
    while (true) {
        bool more = false;
#pragma unroll
        for (int j = 0; j < 2; ++j) more = more || (j < pend_n && done[j] < pend[j].nparts);
        if (!more) break;
        if (tid == 0) {
            asm volatile("fence.proxy.async;" ::: "memory");
            uint32_t bytes = 0;
            // the expected bytes are known before the copies are issued: same arithmetic as issue()
#pragma unroll
            for (int j = 0; j < 2; ++j)
                if (j < pend_n && done[j] < pend[j].nparts) {
                    const int np = min(per_piece(j), pend[j].nparts - done[j]);
                    bytes += (uint32_t)np * kPartBytes + (done[j] == 0 ? (uint32_t)pend[j].nparts * GP * 8u : 0u);
                }
            mbar_arrive_expect_tx(&tail->merge_bar, bytes);
            uint32_t issued = 0;
#pragma unroll
            for (int j = 0; j < 2; ++j)
                if (j < pend_n && done[j] < pend[j].nparts) issue(j, done[j], issued);
        }
        __syncwarp();
        mbar_wait(&tail->merge_bar, merge_phase & 1u, abort, a.status);
        ++merge_phase;
#pragma unroll
        for (int j = 0; j < 2; ++j)
            if (j < pend_n && done[j] < pend[j].nparts) add_piece(j, done[j]);
        named_barrier(1, kCT);   // everyone is done with the ring before the next pieces overwrite it
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        if (j < pend_n && mine && ARB_IN_RANGE(a.status, pend[j].out_base + G * kD - 1, (size_t)a.rows * a.Hq * kD)) {
            const float inv = 1.0f / l[j];
            uint2 o2;
            o2.x = pack_bf16(x[j].x * inv, x[j].y * inv);
            o2.y = pack_bf16(x[j].z * inv, x[j].w * inv);
            *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(a.out) + pend[j].out_base + (size_t)e * 4) = o2;
        }
    }
}

// Ring depth: 32 stages, 128 KB of tiles in flight per SM with one CTA per SM.  A 16-stage ring with room for two
// CTAs per SM (so that the next kernel of a chain is resident before this one ends) was measured and is slower on
// every workload: a lone call is bound by bytes in flight, and the successor's CTAs come up SM by SM as this
// kernel's CTAs leave anyway.
// Ring stages.  What is in flight per SM is stages x bytes of a stage, and it has to cover latency x bandwidth: 32 tiles
// of a bf16 cache are 128 KB; the tiles of the code caches are 2 KB and 1.1 KB, so their rings are deeper (with 32
// stages a large call over 4-bit codes could keep 16 KB per SM in flight: 1.4 TB/s).  The widened tiles of the code
// forms take 64 KB beside the ring.
template <int KV>
constexpr int stages_of() { return KV == kKvBf16 ? 32 : KV == kKvE4m3 ? 48 : 80; }

template <int G, bool APPEND, int KV>
arb_status launch_variant(Ctx *ctx, const StepArgs &a, const CUtensorMap &km, const CUtensorMap &vm, cudaStream_t stream) {
    static bool attr_set[64] = {};
    if (!attr_set[ctx->device & 63]) {
        if (cudaFuncSetAttribute(decode_step_kernel<G, stages_of<KV>(), APPEND, KV>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem_bytes<G, stages_of<KV>(), KV>(kMaxBatch)) != cudaSuccess)
            return ARB_ERR_CUDA;
        attr_set[ctx->device & 63] = true;
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctx->num_sms);
    cfg.blockDim = dim3(kNT);
    cfg.dynamicSmemBytes = smem_bytes<G, stages_of<KV>(), KV>(a.batch);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, decode_step_kernel<G, stages_of<KV>(), APPEND, KV>, a, km, vm) != cudaSuccess) return ARB_ERR_CUDA;
    ctx->launches++;
    return ARB_OK;
}

// The E4M3 and the 4-bit forms exist with the cache write only (decode alone over an E4M3 cache is arb_attn_decode_e4m3).
template <int G>
arb_status launch_g(Ctx *ctx, const StepArgs &a, int kv, const CUtensorMap &km, const CUtensorMap &vm, cudaStream_t stream) {
    if (kv == kKvE4m3) return launch_variant<G, true, kKvE4m3>(ctx, a, km, vm, stream);
    if (kv == kKvI4) return launch_variant<G, true, kKvI4>(ctx, a, km, vm, stream);
    return a.k_new != nullptr ? launch_variant<G, true, kKvBf16>(ctx, a, km, vm, stream)
                              : launch_variant<G, false, kKvBf16>(ctx, a, km, vm, stream);
}

}  // namespace

size_t decode_step_hint_bytes(int num_sms) { return sizeof(int) * (size_t)num_sms * kHintStride; }

bool decode_step_supported(const arb_attn_params &p) {
    const int g = p.num_q_heads / p.num_kv_heads;
    return p.dtype == ARB_BF16 && p.head_dim == kD && g >= 1 && g <= 8 && tma_available();
}

// k_new == nullptr: attention only (seq_lens is not written).  scales != nullptr: an E4M3 cache with scales =
// {k_scale, v_scale, k_inv_scale, v_inv_scale}; k_row_scales != nullptr: a 4-bit cache with its two scale pools
// (k_new is required for both); neither: a bf16 cache.
arb_status launch_decode_step(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_new, const void *v_new,
                              void *k_pages, void *v_pages, const float *scales, const int32_t *block_table,
                              int32_t *seq_lens, const int32_t *q_lens, void *out, cudaStream_t stream,
                              float *k_row_scales, float *v_row_scales) {
    alignas(64) CUtensorMap km, vm;
    const bool e4m3 = scales != nullptr, i4 = k_row_scales != nullptr;
    if ((e4m3 || i4) && k_new == nullptr) return ARB_ERR_INVALID_ARG;
    if (e4m3 && i4) return ARB_ERR_INVALID_ARG;
    bool whole_rows = false;
    if (i4) {
        if (!pool_map(ctx, &km, k_pages, p.num_pages, p.num_kv_heads, PoolView::kI4) ||
            !pool_map(ctx, &vm, v_pages, p.num_pages, p.num_kv_heads, PoolView::kI4))
            return ARB_ERR_CUDA;
    } else if (e4m3) {
        if (!pool_map(ctx, &km, k_pages, p.num_pages, p.num_kv_heads, PoolView::kE4m3) ||
            !pool_map(ctx, &vm, v_pages, p.num_pages, p.num_kv_heads, PoolView::kE4m3))
            return ARB_ERR_CUDA;
    } else {
        whole_rows = pool_map(ctx, &km, k_pages, p.num_pages, p.num_kv_heads, PoolView::kBf16WholeRows) &&
                     pool_map(ctx, &vm, v_pages, p.num_pages, p.num_kv_heads, PoolView::kBf16WholeRows);
        if (!whole_rows && (!pool_map(ctx, &km, k_pages, p.num_pages, p.num_kv_heads, PoolView::kBf16HalfRows) ||
                            !pool_map(ctx, &vm, v_pages, p.num_pages, p.num_kv_heads, PoolView::kBf16HalfRows)))
            return ARB_ERR_CUDA;
    }
    const int g = p.num_q_heads / p.num_kv_heads;
    const int gp = (g + 3) / 4 * 4;
    const size_t slots = (size_t)p.batch * p.num_kv_heads + (size_t)ctx->num_sms;
    const size_t part_o_floats = (slots * g * p.head_dim + 63) & ~size_t(63);
    const size_t bytes = (part_o_floats + slots * gp * 2) * sizeof(float);
    if (bytes > ctx->workspace_bytes) return ARB_ERR_WORKSPACE;
    note_unnumbered_decode(ctx, bytes);   // region 0 of the workspace: this kernel waits for its predecessor first
    StepArgs a;
    a.q = static_cast<const char *>(q);
    a.k_new = static_cast<const char *>(k_new);
    a.v_new = static_cast<const char *>(v_new);
    a.k_pool = static_cast<char *>(k_pages);
    a.v_pool = static_cast<char *>(v_pages);
    a.block_table = block_table;
    a.seq_lens = seq_lens;
    a.q_lens = q_lens;
    a.out = static_cast<char *>(out);
    a.part_o = reinterpret_cast<float *>(ctx->workspace);
    a.part_ml = a.part_o + part_o_floats;
    a.counters = ctx->rot;                                                       // [kRotCounters]
    a.lens_counter = ctx->rot + (size_t)kRotSets * kRotCounters + kRotSets + 4;
    a.hint = ctx->step_hint;
    a.hint_tag = (int)(((uint32_t)p.batch * 2654435761u) ^ ((uint32_t)p.num_kv_heads * 40503u) ^
                       ((uint32_t)p.num_pages * 2246822519u) ^ ((uint32_t)p.max_pages_per_seq * 3266489917u)) | 1;
    a.status = ctx->status;
    a.batch = p.batch;
    a.Hq = p.num_q_heads;
    a.Hkv = p.num_kv_heads;
    a.num_pages = p.num_pages;
    a.max_pages = p.max_pages_per_seq;
    a.whole_rows = whole_rows ? 1 : 0;
    a.slots = (int)slots;
    a.rows = p.total_q;
    a.boundary_pct = ctx->step_boundary_pct;
    a.min_chunk = ctx->step_min_chunk;
    const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.head_dim);
    a.scale_log2 = scale * (e4m3 ? scales[0] : 1.0f) * 1.4426950408889634f;
    a.v_scale = e4m3 ? scales[1] : 1.0f;
    a.k_inv_scale = e4m3 ? scales[2] : 1.0f;
    a.v_inv_scale = e4m3 ? scales[3] : 1.0f;
    a.k_scales = k_row_scales;
    a.v_scales = v_row_scales;
    const int kv = i4 ? kKvI4 : e4m3 ? kKvE4m3 : kKvBf16;
    switch (g) {
        case 1: return launch_g<1>(ctx, a, kv, km, vm, stream);
        case 2: return launch_g<2>(ctx, a, kv, km, vm, stream);
        case 3: return launch_g<3>(ctx, a, kv, km, vm, stream);
        case 4: return launch_g<4>(ctx, a, kv, km, vm, stream);
        case 5: return launch_g<5>(ctx, a, kv, km, vm, stream);
        case 6: return launch_g<6>(ctx, a, kv, km, vm, stream);
        case 7: return launch_g<7>(ctx, a, kv, km, vm, stream);
        case 8: return launch_g<8>(ctx, a, kv, km, vm, stream);
        default: return ARB_ERR_UNSUPPORTED;
    }
}

}  // namespace arb

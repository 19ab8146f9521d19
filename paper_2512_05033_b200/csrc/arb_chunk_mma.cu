// Step-chunk attention on the 5th-generation tensor cores (tcgen05 + TMEM), bf16, head_dim 128.
//
// A chunk of n query tokens against one KV head is a contraction over shared operands: the
// M = n * group query rows (token-major, the group's heads of one token are consecutive rows) all read
// the same keys (dense enough to keep the tensor core busy from M of about 64; below that the tile is
// mostly padding, but it still reads every key once).  One work item is a pair of row tiles (A, B: 128 query rows each, B may be
// missing) of one (sequence, kv head); it walks the visible keys in tiles of 128 (eight pages), and
// both row tiles use every K/V tile that is loaded.  Per row tile and KV tile:
//
//     S = Q K^T      tcgen05.mma, A = Q tile, B = K tile, both K-major in shared memory (128-byte
//                    swizzle), fp32 accumulator in the 128 TMEM columns for S
//     P = exp2(scale * S - m)   by a softmax group of 128 threads, one TMEM lane (= query row)
//                    each: tcgen05.ld, causal / length mask, row max, exponentials; P, rounded to
//                    bf16, goes to the group's own TMEM columns (tcgen05.st, two keys per column)
//     O += P V       tcgen05.mma with P as the TMEM A operand and the V tile read MN-major straight
//                    from its page layout; fp32 accumulator in the group's 128 TMEM columns for O
//
// TMEM: S 0-127 (one region for both groups), P_A 128-191, P_B 192-255, O_A 256-383, O_B 384-511.  The
// work of an item is a sequence of units (one group on one KV tile; the groups alternate).  S of a unit is
// wanted only until its group holds it in registers, so one S region serves both groups, and with P in
// columns of its own the next unit's Q K^T runs under this unit's exponentials: a softmax group goes from
// one unit to its next without waiting for a product.  Q K^T and P V are issued by two threads of two
// warps, so that neither kind waits while the other thread looks at its barriers.  An item with a single row
// tile gives its KV tiles to the two groups in turn (both against Q tile A); they merge their two O in the
// epilogue.  The running max is lazy: O is rescaled
// (tcgen05.ld / st) only when a row's max grows by more than 2^8, otherwise the stale max keeps the
// exponentials bounded by 2^8 and nothing is touched.  K and V tiles are fetched page by page with
// tiled TMA copies (one 16 x 64 box per page and half of head_dim, landing in the canonical swizzled
// layout) into a two-stage ring.  Roles: warps 0-3 softmax group A, warps 4-7 group B (softmax and epilogue),
// warp 8 TMA producer of K, warp 10 of V, warp 9 issue of Q K^T and TMEM allocation, warp 11 issue of P V.  Work items are
// handed out dynamically, longest sequences first: the K producer takes the next item from an atomic
// counter and announces it to the other roles through a small queue in shared memory.  Every mbarrier wait
// is bounded; TMEM is released on every path.
//
// The same kernel, compiled a second time (template parameter E4M3), reads an E4M3 KV cache (one byte per element;
// keys are k_scale * code, values v_scale * code): the chunk a quantised draft's cache absorbs when the target's
// step replaces its own (Algorithm 1, escalation branch).  The codes widen to f16 exactly, so the products run as
// f16 MMAs with fp32 accumulation; q is converted bf16 -> f16 as its tile is written, P is rounded to f16.  A page
// of codes (16 rows x 128 bytes) arrives through one tiled TMA copy in a small staging ring of four pages per
// operand; the producer warp of the operand widens it (cvt.rn.f16x2.e4m3x2) into the operand stage, in the
// 128-byte-swizzled layout the bf16 tiles land in, and asks for the page four ahead.  The key scale folds into the
// softmax scale, the value scale into the epilogue.
#include "arb_tma.cuh"

namespace arb {

namespace {

constexpr int kD = 128;           // head_dim
constexpr int kBM = 128;          // query rows per row tile; a work item is a pair of row tiles
constexpr int kBN = 128;          // keys per KV tile
constexpr int kTilePages = kBN / kPage;
constexpr int kStages = 2;
constexpr int kSoftmaxThreads = 128;        // per row tile
constexpr int kThreads = 3 * kSoftmaxThreads;   // two softmax groups and a group of service warps; registers are
                                                // handed out per 128 threads, so the third group's spare warps cost none
constexpr int kTmaWarp = 8, kMmaWarp = 9, kVWarp = 10, kPvWarp = 11;
// The E4M3 form runs a fourth group of warps: warps 12, 13 widen pairs of pages of K beside warp 8, warps 14, 15 pairs of
// V beside warp 10 (one warp per operand widens a tile in about twice the time the tensor core and the softmax groups
// need for it).  The pairs of an operand are numbered through the tiles; pair n belongs to warp n % 3 of the operand and
// to staging slot n % 3, so every warp has a slot of its own, asks for its own next pair, and takes part in every
// tile (four consecutive numbers cover the three residues).  512 threads start with 128 registers each; the softmax
// groups then take 168 and the two service groups keep 88 (setmaxnreg; 2 * 168 + 2 * 88 = 4 * 128).
constexpr int kKHelpWarp = 12, kVHelpWarp = 14;   // and the warp after each
constexpr int kWideners = 3;                      // warps per operand in the E4M3 form
static_assert(kWideners == 3 && kWideners <= 4, "a slot per widening warp; every warp has a pair in every full tile");
__host__ __device__ constexpr int threads_of(bool e4m3) { return e4m3 ? 4 * kSoftmaxThreads : kThreads; }
constexpr int kHalfBytes = 128 * 128;      // [128 rows x 64 bf16]: one 128-byte-swizzled half tile
constexpr int kTileBytes = 2 * kHalfBytes;  // [128 x 128] bf16
constexpr int kBoxBytes = kPage * 128;      // one TMA box: 16 rows x 64 bf16
constexpr int kStagePages = 6;              // E4M3: pages of codes in flight per operand ...
constexpr int kStagePairs = kStagePages / 2;   // ... asked for, waited for and widened two at a time
constexpr int kTilePairs = kTilePages / 2;
constexpr int kCodePageBytes = kPage * kD;  // 2 KB: one (page, kv head) tile of codes
constexpr uint32_t kTmemCols = 512;         // S (shared): columns 0..127, P of group A: 128..191, of B: 192..255,
constexpr uint32_t kPCol = 128;             // O of group A: 256..383, of B: 384..511
constexpr uint32_t kOCol = 256;
constexpr float kRescaleThreshold = 8.0f;   // log2 units
constexpr int kItemSlots = 8;               // work items announced ahead of their use
constexpr int kPrefetchTiles = 4;            // K/V tiles asked into L2 ahead of the ring
constexpr int kSortMaxBatch = 256;          // up to this batch size sequences are served longest first
// Split-KV for long sequences: a sequence that sees more than kSplitMinTiles KV tiles has its key range
// cut into parts of about kSplitPartTiles tiles; every (row tile pair, part) is a work item of its own
// and leaves un-normalised partial results, which chunk_combine_kernel merges.  Without this one 64k-token
// sequence in a batch keeps a single CTA busy long after all others have run dry.
constexpr int kSplitMinTiles = 160;
constexpr int kSplitPartTiles = 96;
constexpr int kSplitMaxParts = 32;          // a warp's lanes cover the parts in the combine
// A call with few work items (a small batch of short steps) leaves most SMs idle while each item walks its keys at
// the pace of one row tile's chain.  Such a call is cut the same way, down to parts of kFillPartTiles tiles, for
// sequences of at least kFillMinTiles tiles.
constexpr int kFillMinTiles = 8;
constexpr int kFillPartTiles = 4;
constexpr size_t kSlotFloats = (size_t)kBM * kD + 2 * kBM;   // one row tile's partial: O as [32 groups of 4 dims][128 rows][4],
                                                             // so that the rows' 16-byte pieces lie side by side; then (max, sum) [128][2]

struct MmaArgs {
    const char *q;
    const char *k_pool, *v_pool;  // for L2 prefetches; the tiles themselves come through the tensor maps
    const int32_t *block_table;
    const int32_t *seq_lens;
    const int32_t *q_lens;
    char *out;
    uint32_t *status;
    int batch, Hq, Hkv, num_pages, max_pages;
    int min_rows;  // sequences with q_len * group >= min_rows are handled here
    int *work_counter;  // [0] next work item, [1] set if a chunk sequence is left for the CUDA-core kernel;
                        // both zeroed on the stream before the launch
    float *split_ws;    // partial results of split sequences, kSlotFloats per (item, row tile)
    int split_cap;      // slots that fit there
    int fill_ctas;      // CTAs a call should keep busy: a call with fewer than half as many work items has its
                        // sequences cut over their keys as well (0: never)
    int rows;           // rows of q and out (bounds-check build)
    float scale_log2;   // softmax scale (times the key scale of an E4M3 cache) * log2(e)
    float v_scale;      // value scale of an E4M3 cache, 1 otherwise
};

struct Bars {
    uint64_t q_full;             // both softmax groups wrote their Q tiles
    uint64_t k_full[kStages];    // TMA bytes of a K tile landed
    uint64_t v_full[kStages];
    uint64_t k_empty[kStages];   // the first products that read the K stage have completed
    uint64_t v_empty[kStages];   // the second products that read the V stage have completed
    uint64_t s_full[2];          // S = Q K^T of row tile A / B is in TMEM
    uint64_t p_full[2];          // P of row tile A / B is in TMEM (over S)
    uint64_t o_full[2];          // O += P V of row tile A / B has completed
    uint64_t s_free[2];          // group A / B holds the S it was given in registers: the S region is free
    uint64_t ml_full;            // an item with one row tile: both softmax groups have left their (max, sum)
    uint64_t item_full[kItemSlots];   // the producer warp has fetched the next work item
    uint64_t item_empty[kItemSlots];  // the MMA thread, the V producer and the softmax threads have read it
    uint64_t code_full[2][kStagePages];   // E4M3: a page of codes of K / of V has landed in its staging slot
    int item_id[kItemSlots];
    uint32_t tmem_base;
    int abort;
};

constexpr size_t kSmemFixed = 1024 /*alignment*/ + 2 * kTileBytes /*Q of A, B*/ + 2 * kStages * kTileBytes /*K, V*/ +
                              sizeof(Bars);

constexpr size_t kCodeStageBytes = 2 * kStagePages * kCodePageBytes;   // E4M3: staging of both operands
constexpr int kMaxBatchE4m3 = 320;   // the staging takes 24 KB of what the plan tables of a larger batch would need

inline size_t mma_smem_bytes(int batch, bool e4m3 = false) {
    return kSmemFixed + (e4m3 ? kCodeStageBytes : 0) + sizeof(int) * (7 * (size_t)batch + 2);
}

// ---- tcgen05 / TMA wrappers -------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}

// arrives on `bar` once every tcgen05 operation issued so far by this thread has completed
__device__ __forceinline__ void mma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]; M = 128, K = 16 per instruction
__device__ __forceinline__ void mma_f16_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem]: A is bf16 packed two to a 32-bit column, row m in TMEM lane m
__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading / stride byte offsets
// (all in 16-byte units), descriptor version 1 (sm_100), layout type 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor of kind::f16: fp32 accumulator, A and B both bf16 or both f16, M = 128, N = 128.
__host__ __device__ constexpr uint32_t instr_desc(bool b_mn_major, bool f16 = false) {
    return (1u << 4)                       // accumulator format: f32
           | ((f16 ? 0u : 1u) << 7) | ((f16 ? 0u : 1u) << 10)   // A, B format: f16 = 0, bf16 = 1
           | (0u << 15)                    // A is K-major
           | ((b_mn_major ? 1u : 0u) << 16)
           | ((uint32_t)(kBN >> 3) << 17)  // N
           | ((uint32_t)(kBM >> 4) << 24); // M
}

__device__ __forceinline__ void tma_box_load(void *dst_smem, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

#define ARB_R32(v, o)                                                                                       \
    "=r"(v[o + 0]), "=r"(v[o + 1]), "=r"(v[o + 2]), "=r"(v[o + 3]), "=r"(v[o + 4]), "=r"(v[o + 5]), "=r"(v[o + 6]), \
        "=r"(v[o + 7])
// 32 consecutive fp32 columns of this thread's TMEM lane into v[O .. O + 31]
template <int O, int N>
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[N]) {
    static_assert(O + 32 <= N, "range");
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : ARB_R32(v, O + 0), ARB_R32(v, O + 8), ARB_R32(v, O + 16), ARB_R32(v, O + 24)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) { tmem_ld32<0, 32>(taddr, v); }
#undef ARB_R32
#define ARB_W8(v, o) "r"(v[o + 0]), "r"(v[o + 1]), "r"(v[o + 2]), "r"(v[o + 3]), "r"(v[o + 4]), "r"(v[o + 5]), "r"(v[o + 6]), "r"(v[o + 7])
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), ARB_W8(v, 0), ARB_W8(v, 8), ARB_W8(v, 16), ARB_W8(v, 24)
        : "memory");
}
#undef ARB_W8
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// two bf16 (one 32-bit word) -> two f16
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t v) {
    return pack_f16(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
}
// two E4M3 codes (a 16-bit pair) -> f16x2, exact; the low byte lands in the low half
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint16_t v) {
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(v));
    return r;
}

// packed pairs of fp32 (one instruction for two lanes of arithmetic)
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// A work item: up to two consecutive row tiles (A, B) of one (sequence, kv head), over the KV tiles
// [t0, t0 + ntiles) of the keys they see.  They share every K/V tile that is loaded; B may be missing
// (rows[1] == 0).  `split`: the sequence's keys are cut into parts and this item leaves partials in
// slots `slot` (tile A) and `slot + 1` (tile B).
struct Item {
    int b, kvh, n, L, rows_total, r_begin, rows[2], kv_len, t0, ntiles, qrow0, slot;
    bool split;
};

// The tables every CTA (and the combine kernel) derives from the lengths, in shared memory.
struct Plan {
    int *pref;     // [B + 1] work items before the sequence in serving position r
    int *row0;     // [B + 1] q rows before sequence b
    int *sorted;   // [B] sequences in serving order (longest first)
    int *pairs;    // [B] row tile pairs of sequence b (0: not served by this kernel)
    int *key;      // [B] visible keys of sequence b (sort key)
    int *parts;    // [B] parts the keys of the sequence in serving position r are cut into
    int *sslot;    // [B] first partial slot of the sequence in serving position r
};

__device__ __forceinline__ Plan plan_arrays(int *base, int B) {
    Plan pl;
    pl.pref = base;
    pl.row0 = pl.pref + B + 1;
    pl.sorted = pl.row0 + B + 1;
    pl.pairs = pl.sorted + B;
    pl.key = pl.pairs + B;
    pl.parts = pl.key + B;
    pl.sslot = pl.parts + B;
    return pl;
}

// Fills the plan; every thread of the block takes part.  small_flag (nullable): set to 1 by block 0 if a
// chunk sequence is left for the CUDA-core kernel.
template <int G>
__device__ void make_plan(const MmaArgs &a, Plan pl, int tid, int nthreads, int *small_flag) {
    const int B = a.batch, Hkv = a.Hkv, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) { pl.pref[0] = 0; pl.row0[0] = 0; }
    for (int b = tid; b < B; b += nthreads) {
        const int n = a.q_lens[b], L = a.seq_lens[b];
        int pairs = 0;
        if (n >= 2 && n * G >= a.min_rows && L >= n && L <= a.max_pages * kPage) pairs = (n * G + 2 * kBM - 1) / (2 * kBM);
        if (small_flag != nullptr && blockIdx.x == 0 && n >= 2 && pairs == 0) atomicOr(small_flag, 1);  // small, or invalid lengths
        pl.pairs[b] = pairs;
        pl.key[b] = pairs > 0 ? L : -1;
        pl.row0[b + 1] = n > 0 ? n : 0;
    }
    __syncthreads();
    // serving order: longest first (items of a long sequence take longest), ties by index; large
    // batches keep their own order
    for (int b = tid; b < B; b += nthreads) {
        int rank = b;
        if (B <= kSortMaxBatch) {
            rank = 0;
            const int kb = pl.key[b];
            for (int o = 0; o < B; ++o) rank += (pl.key[o] > kb) || (pl.key[o] == kb && o < b);
        }
        pl.sorted[rank] = b;
    }
    __syncthreads();
    if (warp == 0) {
        // in serving order: parts (granted while the partial slots last), partial slots and work items;
        // and, in batch order, the q rows
        // does the call fill the machine as it is?  (work items and their KV tiles without any split)
        int items0 = 0, tiles0 = 0;
        for (int r0 = 0; r0 < B; r0 += 32) {
            const int r = r0 + lane;
            if (r < B && pl.pairs[r] > 0) {
                items0 += Hkv * pl.pairs[r];
                tiles0 += Hkv * pl.pairs[r] * ((pl.key[r] + kBN - 1) / kBN);
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            items0 += __shfl_xor_sync(0xffffffffu, items0, off);
            tiles0 += __shfl_xor_sync(0xffffffffu, tiles0, off);
        }
        const bool fill = a.fill_ctas > 0 && items0 > 0 && 2 * items0 <= a.fill_ctas;
        const int fill_part = max(kFillPartTiles, (tiles0 + max(a.fill_ctas, 1) - 1) / max(a.fill_ctas, 1));
        int carry_p = 0, carry_r = 0, carry_s = 0;
        for (int r0 = 0; r0 < B; r0 += 32) {
            const int r = r0 + lane;
            int want = 1, slots = 0, pairs = 0;
            if (r < B) {
                const int sb = pl.sorted[r];
                pairs = pl.pairs[sb];
                const int nt = pairs > 0 ? (pl.key[sb] + kBN - 1) / kBN : 0;
                if (nt > kSplitMinTiles) {
                    want = min((nt + kSplitPartTiles - 1) / kSplitPartTiles, kSplitMaxParts);
                    slots = Hkv * pairs * want * 2;
                } else if (fill && nt >= kFillMinTiles) {
                    want = min((nt + fill_part - 1) / fill_part, kSplitMaxParts);
                    slots = want > 1 ? Hkv * pairs * want * 2 : 0;
                }
            }
            int vs = slots;
            int vr = r < B ? pl.row0[r + 1] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int ts = __shfl_up_sync(0xffffffffu, vs, off);
                const int tr = __shfl_up_sync(0xffffffffu, vr, off);
                if (lane >= off) { vs += ts; vr += tr; }
            }
            const bool granted = slots > 0 && vs + carry_s <= a.split_cap;
            const int P = granted ? want : 1;
            int vp = Hkv * pairs * P;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int tp = __shfl_up_sync(0xffffffffu, vp, off);
                if (lane >= off) vp += tp;
            }
            if (r < B) {
                pl.parts[r] = P;
                pl.sslot[r] = vs + carry_s - slots;
                pl.pref[r + 1] = vp + carry_p;
                pl.row0[r + 1] = vr + carry_r;
            }
            carry_p += __shfl_sync(0xffffffffu, vp, 31);
            carry_r += __shfl_sync(0xffffffffu, vr, 31);
            carry_s += __shfl_sync(0xffffffffu, vs, 31);
        }
    }
    __syncthreads();
}

// keys the row tile pair that starts at row r_begin sees, and the tiles of one part of the sequence
template <int G>
__device__ __forceinline__ int pair_kv_len(int L, int n, int rows_total, int r_begin) {
    const int r_last = min(r_begin + 2 * kBM, rows_total) - 1;
    return L - n + r_last / G + 1;
}
__device__ __forceinline__ int part_tiles(int L, int P) {
    const int nt = (L + kBN - 1) / kBN;
    return (nt + P - 1) / P;
}

template <int G>
__device__ __forceinline__ bool get_item(int item, int total, const Plan &pl, int B, int Hkv, const MmaArgs &a, Item &it) {
    if (item >= total) return false;
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (pl.pref[mid] <= item) lo = mid; else hi = mid;
    }
    const int sb = pl.sorted[lo];  // pref runs over the sequences in serving order
    it.b = sb;
    it.n = a.q_lens[sb];
    it.L = a.seq_lens[sb];
    it.rows_total = it.n * G;
    const int pairs = pl.pairs[sb], P = pl.parts[lo];
    const int r = item - pl.pref[lo];
    it.kvh = r / (pairs * P);
    const int rem = r - it.kvh * pairs * P;
    const int pt = rem / P, part = rem - pt * P;
    it.r_begin = pt * 2 * kBM;
    it.rows[0] = min(kBM, it.rows_total - it.r_begin);
    it.rows[1] = max(0, min(kBM, it.rows_total - it.r_begin - kBM));
    it.kv_len = pair_kv_len<G>(it.L, it.n, it.rows_total, it.r_begin);   // keys the pair's last row sees
    const int nt_pair = (it.kv_len + kBN - 1) / kBN;
    const int T = part_tiles(it.L, P);
    it.t0 = part * T;
    it.ntiles = max(0, min(it.t0 + T, nt_pair) - it.t0);   // 0: nothing of this part is visible to the pair
    it.split = P > 1;
    it.slot = pl.sslot[lo] + ((it.kvh * pairs + pt) * P + part) * 2;
    it.qrow0 = pl.row0[sb];
    return true;
}

template <int G, bool E4M3>
__global__ void __launch_bounds__(threads_of(E4M3), 1)
chunk_mma_kernel(const MmaArgs a, const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map) {
    extern __shared__ char smem_raw[];
    char *base = reinterpret_cast<char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    char *q_s = base;                                  // [row tile A, B][2 halves][128 rows][128 B]
    char *k_s = base + 2 * kTileBytes;                 // [stage][2 halves][128 keys][128 B]
    char *v_s = k_s + kStages * kTileBytes;
    char *code_s = v_s + kStages * kTileBytes;         // E4M3: [K, V][kStagePages][16 rows][128 B of codes]
    Bars *bars = reinterpret_cast<Bars *>(code_s + (E4M3 ? kCodeStageBytes : 0));
    const Plan pl = plan_arrays(reinterpret_cast<int *>(bars + 1), a.batch);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.batch, Hkv = a.Hkv;

    let_successor_start();
    if (tid == 0) {
        mbar_init(&bars->q_full, 2 * kSoftmaxThreads);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bars->k_full[s], E4M3 ? kWideners : 1);   // E4M3: every widening warp of the operand arrives
            mbar_init(&bars->v_full[s], E4M3 ? kWideners : 1);
            mbar_init(&bars->k_empty[s], 1);
            mbar_init(&bars->v_empty[s], 1);
        }
        mbar_init(&bars->s_full[0], 1);
        mbar_init(&bars->s_full[1], 1);
        mbar_init(&bars->p_full[0], kSoftmaxThreads);
        mbar_init(&bars->p_full[1], kSoftmaxThreads);
        mbar_init(&bars->o_full[0], 1);
        mbar_init(&bars->o_full[1], 1);
        mbar_init(&bars->s_free[0], kSoftmaxThreads);
        mbar_init(&bars->s_free[1], kSoftmaxThreads);
        mbar_init(&bars->ml_full, 2 * kSoftmaxThreads);
        for (int i = 0; i < kItemSlots; ++i) {
            mbar_init(&bars->item_full[i], 1);
            // the two MMA threads, the V warp, the softmax threads (E4M3: and the four helping warps)
            mbar_init(&bars->item_empty[i], 3 + 2 * kSoftmaxThreads + (E4M3 ? 2 * (kWideners - 1) : 0));
        }
        for (int i = 0; i < kStagePages; ++i) {
            mbar_init(&bars->code_full[0][i], 1);
            mbar_init(&bars->code_full[1][i], 1);
        }
        bars->abort = 0;
        mbar_fence_init();
    }
    wait_for_predecessor();   // everything below reads what the kernel before this one may have written
    make_plan<G>(a, pl, tid, threads_of(E4M3), a.work_counter + 1);
    const int total = pl.pref[B];
    if ((int)blockIdx.x >= total) return;  // nothing for this CTA; no TMEM taken, no barrier pending

    if (warp == kMmaWarp) tmem_alloc(&bars->tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;
    volatile int *abort = &bars->abort;

    const bool helper = E4M3 && warp >= kKHelpWarp;                          // a widening warp of the fourth group
    const int widx = helper ? 1 + (warp & 1) : 0;                            // which of the operand's wideners
    if (warp >= 2 * kSoftmaxThreads / 32) {   // the service warps
    if constexpr (E4M3) asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
    if (warp == kTmaWarp || warp == kVWarp || helper) {
        // ================================= TMA producers: K warp, V warp ==========================
        // One warp per operand: a tiled TMA copy is issued per (page, 64-dim half), sixteen to a tile, and one
        // warp issues them one after the other (about 1500 cycles per tile), so K and V of a tile are in
        // flight together only when two warps issue them.  The K warp also hands out the work: items come
        // from an atomic counter (longest sequences first) and are announced to every other role, the V warp
        // included, through a small queue in shared memory.  Both run ahead of the consumers as far as their
        // two-stage rings allow.
        const bool is_v = warp == kVWarp || warp >= kVHelpWarp;
        uint64_t *full = is_v ? bars->v_full : bars->k_full, *empty = is_v ? bars->v_empty : bars->k_empty;
        char *ring = is_v ? v_s : k_s;
        const CUtensorMap *map = is_v ? &v_map : &k_map;
        const char *pool = is_v ? a.v_pool : a.k_pool;
        uint32_t it = 0;  // KV tiles issued so far
        uint32_t pc = 0;  // E4M3: pages of codes asked for so far (staging slot and phase)
        Item w;
        for (uint32_t nq = 0;; ++nq) {
            const uint32_t slot = nq % kItemSlots, qpar = (nq / kItemSlots) & 1u;
            int item = total;
            if (lane == 0) {
                if (!is_v && !helper) {
                    if (mbar_wait(&bars->item_empty[slot], qpar ^ 1u, abort, a.status)) item = atomicAdd(a.work_counter, 1);
                    bars->item_id[slot] = item;
                    mbar_arrive(&bars->item_full[slot]);
                } else if (mbar_wait(&bars->item_full[slot], qpar, abort, a.status)) {
                    item = bars->item_id[slot];
                    mbar_arrive(&bars->item_empty[slot]);
                }
            }
            item = __shfl_sync(0xffffffffu, item, 0);
            if (!get_item<G>(item, total, pl, B, Hkv, a, w)) break;
            // Block-table entries are read one step before they are used (the tile's own pages one tile
            // ahead, the pages to ask into L2 one tile before the request), so that no global-memory round
            // trip sits between two tiles.  Lanes 0-7: the pages of a tile; -1 marks "no such page".
            auto table_entry = [&](int jt) -> int {   // jt: tile of this item, 0-based
                if (jt >= w.ntiles) return -1;
                jt += w.t0;
                const int np = min(kTilePages, (w.kv_len - jt * kBN + kPage - 1) / kPage);
                return (lane < np && ARB_IN_RANGE(a.status, jt * kTilePages + lane, a.max_pages))
                           ? a.block_table[(size_t)w.b * a.max_pages + jt * kTilePages + lane] : -1;
            };
            // K and V tiles are asked into L2 kPrefetchTiles ahead of their load into the ring, so the
            // ring (two tiles deep) only has to cover the L2 latency, not the DRAM latency
            auto prefetch_pages = [&](int pf) {
                if ((unsigned)pf < (unsigned)a.num_pages && !helper) {
                    constexpr int kPageBytes = kPage * kD * (E4M3 ? 1 : 2);
                    const char *src = pool + ((size_t)pf * Hkv + w.kvh) * kPageBytes;
                    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(kPageBytes) : "memory");
                }
            };
            for (int jt = 0; jt < kPrefetchTiles; ++jt) prefetch_pages(table_entry(jt));
            int pf_next = table_entry(kPrefetchTiles), pid_next = table_entry(0);
            for (int j = 0; j < w.ntiles; ++j, ++it) {
                const uint32_t s = it % kStages, par = (it / kStages) & 1u;
                const int jg = w.t0 + j;   // tile of the sequence
                const int npages = min(kTilePages, (w.kv_len - jg * kBN + kPage - 1) / kPage);
                int pid = pid_next;
                const int pf = pf_next;
                pid_next = table_entry(j + 1);
                pf_next = table_entry(j + 1 + kPrefetchTiles);
                prefetch_pages(pf);
                if (lane < npages && (unsigned)pid >= (unsigned)a.num_pages) {
                    atomicOr(a.status, (uint32_t)ARB_DEV_BAD_PAGE);
                    pid = 0;
                }
                // lanes 0..15: (half, page).  A K stage is free as soon as the first products of the tile
                // before last have completed, a V stage only after its second products.
                const int pg = lane & 7, half = (lane >> 3) & 1;
                const int row = (__shfl_sync(0xffffffffu, pid, pg) * Hkv + w.kvh) * kPage;
                bool ok = true;
                if constexpr (E4M3) {
                    // Codes go through the staging slots two pages at a time (a slot: 2 pages = 4 KB, one barrier):
                    // wait for a pair, take its codes into registers, ask for the pair kStagePairs ahead (of this tile
                    // or of the next), widen.  Every wait, fence and request costs the warp 100-250 cycles whatever it
                    // covers, so they are paid per pair, not per page.  Lane (r, h) = (lane / 2, lane % 2) widens
                    // the 64 codes of half h of row r of each page: four 16-byte pieces in, eight out.
                    char *stg = code_s + (is_v ? kStagePages * kCodePageBytes : 0);
                    uint64_t *cfull = bars->code_full[is_v ? 1 : 0];
                    // (an entry of the next tile that lies outside the pool is reported when that tile is the current one)
                    const int pid_ahead = __shfl_sync(0xffffffffu, pid_next, pg);
                    const int row_next = (((unsigned)pid_ahead < (unsigned)a.num_pages ? pid_ahead : 0) * Hkv + w.kvh) * kPage;
                    const int left = min(kTilePages, (w.kv_len - (jg + 1) * kBN + kPage - 1) / kPage);   // pages of the next tile
                    const int np_next = (j + 1 < w.ntiles) ? max(left, 0) : 0;
                    // pair q of this tile (q < kTilePairs) or pair q - kTilePairs of the next one, into slot `at` % kStagePairs
                    auto ask = [&](int q, uint32_t at) {
                        const bool nxt = q >= kTilePairs;
                        const int p0 = 2 * (nxt ? q - kTilePairs : q);
                        const int cnt = min(2, (nxt ? np_next : npages) - p0);   // pages of the pair that exist
                        if (cnt <= 0) return;
                        const int rr = nxt ? __shfl_sync(0xffffffffu, row_next, (p0 + (lane & 1)) & 7)
                                           : __shfl_sync(0xffffffffu, row, (p0 + (lane & 1)) & 7);
                        const uint32_t sl = at % kStagePairs;
                        if (lane == 0) mbar_arrive_expect_tx(&cfull[sl], (uint32_t)cnt * kCodePageBytes);
                        __syncwarp();
                        if (lane < cnt) tma_box_load(stg + (sl * 2 + lane) * kCodePageBytes, map, 0, rr, &cfull[sl]);
                    };
                    if (j == 0) {   // a new item: nothing of it is in flight yet; every warp asks for its first pair
                        for (int q = 0; q < kStagePairs; ++q)
                            if ((int)((pc + q) % kWideners) == widx) ask(q, pc + q);
                    }
                    if (lane == 0) ok = mbar_wait(&empty[s], par ^ 1u, abort, a.status);
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                    const int r = lane >> 1, h = lane & 1;
                    const int npairs = (npages + 1) >> 1;
                    for (int q = 0; q < npairs; ++q, ++pc) {
                        if ((int)(pc % kWideners) != widx) continue;   // the operand's warps take the pairs in turn
                        const uint32_t sl = pc % kStagePairs, ph = (pc / kStagePairs) & 1u;
                        const int cnt = min(2, npages - 2 * q);
                        mbar_wait(&cfull[sl], ph, abort, a.status);
                        // the codes come into registers first, so that the slot can be asked for again at once
                        uint4 codes[2][4];
#pragma unroll
                        for (int pp = 0; pp < 2; ++pp) {
                            const char *src = stg + (sl * 2 + pp) * kCodePageBytes + r * 128;
#pragma unroll
                            for (int c4 = 0; c4 < 4; ++c4)
                                codes[pp][c4] = (pp < cnt) ? *reinterpret_cast<const uint4 *>(src + (((4 * h + c4) ^ (r & 7)) << 4))
                                                           : make_uint4(0, 0, 0, 0);
                        }
                        fence_async_smem();   // the slot's next writer is the TMA unit
                        __syncwarp();
                        ask(q + kStagePairs, pc + kStagePairs);
                        if (ok) {
#pragma unroll
                            for (int pp = 0; pp < 2; ++pp) {
                                if (pp < cnt) {
                                    char *dst = ring + s * kTileBytes + h * kHalfBytes + ((2 * q + pp) * kPage + r) * 128;
#pragma unroll
                                    for (int c4 = 0; c4 < 4; ++c4) {
                                        const uint4 cd = codes[pp][c4];
                                        uint4 lo, hi;
                                        lo.x = e4m3x2_to_f16x2((uint16_t)cd.x); lo.y = e4m3x2_to_f16x2((uint16_t)(cd.x >> 16));
                                        lo.z = e4m3x2_to_f16x2((uint16_t)cd.y); lo.w = e4m3x2_to_f16x2((uint16_t)(cd.y >> 16));
                                        hi.x = e4m3x2_to_f16x2((uint16_t)cd.z); hi.y = e4m3x2_to_f16x2((uint16_t)(cd.z >> 16));
                                        hi.z = e4m3x2_to_f16x2((uint16_t)cd.w); hi.w = e4m3x2_to_f16x2((uint16_t)(cd.w >> 16));
                                        *reinterpret_cast<uint4 *>(dst + (((2 * c4) ^ (r & 7)) << 4)) = lo;
                                        *reinterpret_cast<uint4 *>(dst + (((2 * c4 + 1) ^ (r & 7)) << 4)) = hi;
                                    }
                                }
                            }
                        }
                    }
                    fence_async_smem();   // the stage's reader is the tensor core
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&full[s]);
                } else {
                    if (lane == 0) ok = mbar_wait(&empty[s], par ^ 1u, abort, a.status);
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                    if (ok) {
                        if (lane == 0) mbar_arrive_expect_tx(&full[s], (uint32_t)npages * 2u * kBoxBytes);
                        __syncwarp();
                        if (lane < 16 && pg < npages)
                            tma_box_load(ring + s * kTileBytes + half * kHalfBytes + pg * kBoxBytes, map, half * 64, row, &full[s]);
                    }
                }
                __syncwarp();
            }
        }
    } else if (warp == kMmaWarp) {
        // ================================ MMA issue: S = Q K^T ======================================
        // An item is a sequence of units, each the work of one softmax group on one KV tile: for a pair of row tiles
        // unit u is (row tile u % 2, KV tile u / 2); for a single row tile it is (row tile A, KV tile u), the KV tiles
        // alternating between the two groups, which merge their two O in the epilogue.  All units share ONE S region
        // in TMEM; P and O have a region per group.  So S of unit u + 1 is computed as soon as the group of unit u holds
        // S of unit u in registers, under that group's exponentials, and the softmax groups never wait for a product
        // of their own.  The two kinds of product are issued by two threads (this one: S = Q K^T; warp kPvWarp:
        // O += P V): issuing an MMA holds the thread until the tensor core has room for it, and finding a barrier
        // complete costs about a hundred cycles, so one thread issuing both kinds leaves the tensor core idle while it
        // looks at its barriers.
        if (lane == 0) {
            constexpr uint32_t idesc_qk = instr_desc(false, E4M3);
            const uint32_t q_addr = smem_u32(q_s);
            uint32_t it = 0, nitem = 0, nproc = 0;   // KV tiles so far, items, items with work
            uint32_t nfree[2] = {0u, 0u};            // S loads so far per group
            Item w;
            for (;; ++nitem) {
                const uint32_t slot = nitem % kItemSlots, qpar = (nitem / kItemSlots) & 1u;
                if (!mbar_wait(&bars->item_full[slot], qpar, abort, a.status)) break;
                const int item = bars->item_id[slot];
                mbar_arrive(&bars->item_empty[slot]);
                if (!get_item<G>(item, total, pl, B, Hkv, a, w)) break;
                if (w.ntiles == 0) continue;   // a part the pair sees nothing of: no role does anything for it
                mbar_wait(&bars->q_full, nproc & 1u, abort, a.status);
                ++nproc;
                const bool lone = w.rows[1] == 0;
                const int units = lone ? w.ntiles : 2 * w.ntiles;
                // S of unit u: 8 steps of 16 dims, 4 per 64-dim half; K-major operands, SBO = 8 rows.  A K stage is
                // waited for by the first unit that reads it and released behind the last one.
                auto issue_qk = [&](int u) {
                    const uint32_t itx = it + (lone ? u : (u >> 1)), s = itx % kStages;
                    const int g = u & 1, qt = lone ? 0 : g;
                    if (lone || g == 0) mbar_wait(&bars->k_full[s], (itx / kStages) & 1u, abort, a.status);
                    const uint32_t k_addr = smem_u32(k_s + s * kTileBytes);
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < kD / 16; ++ks) {
                        const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                        mma_f16_ss(tmem, smem_desc(q_addr + qt * kTileBytes + off, 16, 1024),
                                   smem_desc(k_addr + off, 16, 1024), idesc_qk, ks > 0 ? 1u : 0u);
                    }
                    mma_commit(&bars->s_full[g]);
                    if (lone || g == 1) mma_commit(&bars->k_empty[s]);
                };
                issue_qk(0);
                for (int u = 0; u < units; ++u) {
                    const int g = u & 1;
                    mbar_wait(&bars->s_free[g], nfree[g] & 1u, abort, a.status);   // S of unit u is in registers
                    ++nfree[g];
                    if (u + 1 < units) issue_qk(u + 1);
                }
                it += w.ntiles;
            }
        }
        __syncwarp();
    } else if (warp == kPvWarp) {
        // ================================ MMA issue: O += P V =======================================
        if (lane == 0) {
            constexpr uint32_t idesc_pv = instr_desc(true, E4M3);
            uint32_t it = 0, nitem = 0, itg[2] = {0u, 0u};  // KV tiles so far, items, units so far per group
            Item w;
            for (;; ++nitem) {
                const uint32_t slot = nitem % kItemSlots, qpar = (nitem / kItemSlots) & 1u;
                if (!mbar_wait(&bars->item_full[slot], qpar, abort, a.status)) break;
                const int item = bars->item_id[slot];
                mbar_arrive(&bars->item_empty[slot]);
                if (!get_item<G>(item, total, pl, B, Hkv, a, w)) break;
                if (w.ntiles == 0) continue;
                const bool lone = w.rows[1] == 0;
                const int units = lone ? w.ntiles : 2 * w.ntiles;
                // O of the unit's group += P V: 8 steps of 16 keys; P from the group's TMEM columns (two keys per
                // column, 8 columns per step); V MN-major: 64-dim halves LBO apart, 8-key groups SBO apart.  A V stage
                // is waited for by the first unit that reads it and released behind the last one.
                for (int u = 0; u < units; ++u) {
                    const uint32_t itx = it + (lone ? u : (u >> 1)), s = itx % kStages;
                    const int g = u & 1;
                    if (lone || g == 0) mbar_wait(&bars->v_full[s], (itx / kStages) & 1u, abort, a.status);
                    const uint32_t v_addr = smem_u32(v_s + s * kTileBytes);
                    mbar_wait(&bars->p_full[g], itg[g] & 1u, abort, a.status);
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < kBN / 16; ++ks)
                        mma_f16_ts(tmem + kOCol + g * kBN, tmem + kPCol + g * (kBN / 2) + ks * 8,
                                   smem_desc(v_addr + ks * 2 * 1024, kHalfBytes, 1024), idesc_pv,
                                   (u >= 2 || ks > 0) ? 1u : 0u);
                    mma_commit(&bars->o_full[g]);
                    ++itg[g];
                    if (lone || g == 1) mma_commit(&bars->v_empty[s]);
                }
                it += w.ntiles;
            }
        }
        __syncwarp();
    }
    } else {
        // ================================ softmax and epilogue ====================================
        if constexpr (E4M3) asm volatile("setmaxnreg.inc.sync.aligned.u32 168;");
        // two groups of 128 threads: group g works on row tile g of a pair (on every second KV tile of a single row
        // tile); thread tg of a group owns TMEM lane tg
        const int grp = warp >> 2, tg = tid & (kSoftmaxThreads - 1);
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;  // this warp's TMEM lane quadrant
        const uint32_t s_tmem = tmem + lane_base;                                  // S: one region for both groups
        const uint32_t p_tmem = tmem + lane_base + kPCol + grp * (kBN / 2);        // this group's P
        const uint32_t o_tmem = tmem + lane_base + kOCol + grp * kBN;
        char *q_tile = q_s + grp * kTileBytes;
        const int swz = tg & 7;
        uint32_t it = 0, itg = 0, nitem = 0;  // KV tiles so far: of all items, of those this group has worked on
        uint32_t nlone = 0;                   // items with one row tile so far
        Item w;
        for (;; ++nitem) {
            const uint32_t slot = nitem % kItemSlots, qpar = (nitem / kItemSlots) & 1u;
            if (!mbar_wait(&bars->item_full[slot], qpar, abort, a.status)) break;
            const int item = bars->item_id[slot];
            mbar_arrive(&bars->item_empty[slot]);
            if (!get_item<G>(item, total, pl, B, Hkv, a, w)) break;
            if (w.ntiles == 0) continue;   // a part the pair sees nothing of
            // An item with one row tile is worked on by both groups: even KV tiles by group A, odd ones by group B,
            // each with an O of its own, merged in the epilogue.
            const bool lone = w.rows[1] == 0;
            const int rows_here = lone ? w.rows[0] : w.rows[grp];
            const bool row_ok = tg < rows_here;
            const int r = min(w.r_begin + (lone ? 0 : grp * kBM) + tg, w.rows_total - 1);
            const int tok = r / G, head = r - tok * G;
            const int lim = w.L - w.n + tok + 1;  // keys this row may see
            const size_t grow = ((size_t)(w.qrow0 + tok) * a.Hq + w.kvh * G + head) * kD;
            // ---- Q tile: row `tg`, 16 chunks of 8 dims, chunk c of a half stored at c ^ (row & 7)
            if (!(lone && grp == 1)) {   // (the second group of such an item reads Q tile A as well)
                const uint4 *src = reinterpret_cast<const uint4 *>(a.q + grow * 2);
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    uint4 v = row_ok ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
                    if constexpr (E4M3) {   // the operands of one MMA share a type: q goes to f16 like the widened codes
                        v.x = bf16x2_to_f16x2(v.x); v.y = bf16x2_to_f16x2(v.y);
                        v.z = bf16x2_to_f16x2(v.z); v.w = bf16x2_to_f16x2(v.w);
                    }
                    *reinterpret_cast<uint4 *>(q_tile + (c >> 3) * kHalfBytes + tg * 128 + (((c & 7) ^ swz) << 4)) = v;
                }
                fence_async_smem();
            }
            mbar_arrive(&bars->q_full);
            float m_used = -INFINITY, l_sum = 0.f;
            const uint32_t it0 = it;
            it += w.ntiles;
            const int my_tiles = lone ? (w.ntiles + 1 - grp) / 2 : w.ntiles;   // KV tiles this group works on
            for (int j = lone ? grp : 0, jt = 0; j < w.ntiles; j += lone ? 2 : 1, ++itg, ++jt) {
                const uint32_t s = (it0 + j) % kStages, par = ((it0 + j) / kStages) & 1u;
                const int key0 = (w.t0 + j) * kBN;
                const int nvis = lim - key0;  // columns < nvis are visible to this row (may be <= 0)
                mbar_wait(&bars->s_full[grp], itg & 1u, abort, a.status);
                tc_fence_after();
                // ---- the whole row of S (128 scores) comes into registers with one round trip
                uint32_t v[kBN];
                tmem_ld32<0>(s_tmem, v);
                tmem_ld32<32>(s_tmem + 32, v);
                tmem_ld32<64>(s_tmem + 64, v);
                tmem_ld32<96>(s_tmem + 96, v);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(&bars->s_free[grp]);   // the next unit's S may be computed
                if (nvis < kBN) {  // causal edge or end of the sequence: hidden keys weigh exp2(-inf) = 0
#pragma unroll
                    for (int k = 0; k < kBN; ++k)
                        if (k >= nvis) v[k] = 0xff800000u;
                }
                // ---- row max, four independent chains of three-input maxima
                float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int k = 0; k < kBN; k += 8) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        mx4[u] = max3(mx4[u], __uint_as_float(v[k + 2 * u]), __uint_as_float(v[k + 2 * u + 1]));
                }
                const float m_tile = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * a.scale_log2;  // -inf: sees nothing
                float factor = 1.0f;
                bool rescale = false;
                if (m_tile > m_used + kRescaleThreshold || (m_used == -INFINITY && m_tile > -INFINITY)) {
                    factor = fast_exp2(m_used - m_tile);  // 0 the first time
                    rescale = m_used > -INFINITY;          // (nothing has been accumulated before the first visible key)
                    l_sum *= factor;
                    m_used = m_tile;
                }
                // this group's previous product must have completed before its P is overwritten or its O rescaled
                // (it was issued when the group delivered that P, a whole softmax pass ago)
                if (jt > 0) {
                    mbar_wait(&bars->o_full[grp], (itg - 1u) & 1u, abort, a.status);
                    tc_fence_after();
                }
                if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll 1
                    for (int c4 = 0; c4 < 4; ++c4) {
                        uint32_t o[32];
                        tmem_ld32(o_tmem + c4 * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * factor);
                        tmem_st32(o_tmem + c4 * 32, o);
                    }
                    tmem_wait_st();
                }
                // ---- P = exp2(scale * S - m) for two keys per instruction where the hardware has a packed form
                //      (fma.f32x2, add.f32x2; ex2 and the bf16 conversion have none).  The denominator sums
                //      the fp32 weights, the tensor core the same weights rounded to bf16: the two differ by
                //      independent relative errors of at most 2^-9 per key, which the sum averages out.
                //      Keys 32 c .. 32 c + 31 -> columns 16 c .. 16 c + 15 of the group's P region.
                const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
                const uint64_t sc2 = pack_f32x2(a.scale_log2, a.scale_log2), nm2 = pack_f32x2(neg_m, neg_m);
                uint64_t l2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint32_t pk[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const uint64_t t = fma_f32x2(pack_f32x2(__uint_as_float(v[c4 * 32 + 2 * k]),
                                                                __uint_as_float(v[c4 * 32 + 2 * k + 1])), sc2, nm2);
                        float t0, t1;
                        unpack_f32x2(t, t0, t1);
                        const float e0 = fast_exp2(t0), e1 = fast_exp2(t1);
                        pk[k] = E4M3 ? pack_f16(e0, e1) : pack_bf16(e0, e1);
                        l2[k & 3] = add_f32x2(l2[k & 3], pack_f32x2(e0, e1));
                    }
                    tmem_st16(p_tmem + c4 * 16, pk);
                }
                {
                    float x0, x1, y0, y1;
                    unpack_f32x2(add_f32x2(l2[0], l2[1]), x0, x1);
                    unpack_f32x2(add_f32x2(l2[2], l2[3]), y0, y1);
                    l_sum += (x0 + x1) + (y0 + y1);
                }
                tmem_wait_st();
                // ---- V rows past the last visible key of the item (stale slots, pages never loaded)
                //      must not reach the tensor core, not even times zero
                const int nvalid = w.kv_len - key0;
                if (nvalid < kBN && (grp == 0 || lone)) {   // the P of group A (of a pair) is waited for first
                    mbar_wait(&bars->v_full[s], par, abort, a.status);
                    if (tg >= nvalid) {
                        char *vrow = v_s + s * kTileBytes + tg * 128;
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            *reinterpret_cast<uint4 *>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                            *reinterpret_cast<uint4 *>(vrow + kHalfBytes + c * 16) = make_uint4(0, 0, 0, 0);
                        }
                    }
                }
                fence_async_smem();
                tc_fence_before();
                mbar_arrive(&bars->p_full[grp]);
            }
            // ---- epilogue: O / l, bf16, one 256-byte row per thread
            if (my_tiles > 0) mbar_wait(&bars->o_full[grp], (itg - 1u) & 1u, abort, a.status);
            tc_fence_after();
            const bool row_in = ARB_IN_RANGE(a.status, w.qrow0 + tok, a.rows);
            if (lone) {
                // The two groups hold O, max and sum over the even and over the odd KV tiles of the same rows.  They
                // exchange (max, sum) through the shared memory of Q tile B, which such an item does not use, and
                // each merges and writes 64 of the 128 dimensions: thread tg of either group owns TMEM lane tg and
                // reads that lane of both O.
                float2 *ml = reinterpret_cast<float2 *>(q_s + kTileBytes);
                ml[grp * kSoftmaxThreads + tg] = make_float2(m_used, l_sum);
                tc_fence_before();
                mbar_arrive(&bars->ml_full);
                mbar_wait(&bars->ml_full, nlone & 1u, abort, a.status);
                ++nlone;
                tc_fence_after();
                const float2 ml0 = ml[tg], ml1 = ml[kSoftmaxThreads + tg];
                const bool two = w.ntiles > 1;                       // else group B has worked on nothing: its O is undefined
                const float m = fmaxf(ml0.x, two ? ml1.x : -INFINITY);
                const float w0 = ml0.x == -INFINITY ? 0.f : fast_exp2(ml0.x - m);
                const float w1 = (!two || ml1.x == -INFINITY) ? 0.f : fast_exp2(ml1.x - m);
                const float l = ml0.y * w0 + (two ? ml1.y * w1 : 0.f);
                const bool slot_in = !w.split || ARB_IN_RANGE(a.status, w.slot, a.split_cap);
                float *po = a.split_ws + (size_t)(w.split && slot_in ? w.slot : 0) * kSlotFloats;
                const float norm = w.split ? (E4M3 ? a.v_scale : 1.0f) : (E4M3 ? a.v_scale : 1.0f) / l;
                const uint32_t oa = tmem + lane_base + kOCol, ob = oa + kBN;
                uint4 *dst = reinterpret_cast<uint4 *>(a.out + grow * 2);
#pragma unroll 1
                for (int c4 = 2 * grp; c4 < 2 * grp + 2; ++c4) {
                    uint32_t va[32];
                    float o[32];
                    tmem_ld32(oa + c4 * 32, va);
                    tmem_wait_ld();
                    const float n0 = w0 * norm, n1 = w1 * norm;
#pragma unroll
                    for (int k = 0; k < 32; ++k) o[k] = __uint_as_float(va[k]) * n0;
                    if (two) {
                        tmem_ld32(ob + c4 * 32, va);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 32; ++k) o[k] = fmaf(__uint_as_float(va[k]), n1, o[k]);
                    }
                    if (w.split) {
                        if (row_ok && slot_in) {
#pragma unroll
                            for (int qd = 0; qd < 8; ++qd)
                                *reinterpret_cast<float4 *>(po + ((size_t)(c4 * 8 + qd) * kBM + tg) * 4) =
                                    make_float4(o[qd * 4], o[qd * 4 + 1], o[qd * 4 + 2], o[qd * 4 + 3]);
                        }
                    } else if (row_ok && row_in) {
#pragma unroll
                        for (int qd = 0; qd < 4; ++qd) {
                            uint4 o4;
                            o4.x = pack_bf16(o[qd * 8 + 0], o[qd * 8 + 1]);
                            o4.y = pack_bf16(o[qd * 8 + 2], o[qd * 8 + 3]);
                            o4.z = pack_bf16(o[qd * 8 + 4], o[qd * 8 + 5]);
                            o4.w = pack_bf16(o[qd * 8 + 6], o[qd * 8 + 7]);
                            dst[c4 * 4 + qd] = o4;
                        }
                    }
                }
                if (w.split && grp == 0 && row_ok && slot_in)
                    *reinterpret_cast<float2 *>(po + (size_t)kBM * kD + tg * 2) = make_float2(m, l);
                tc_fence_before();
                continue;
            }
            if (w.split) {
                // one part of a split sequence: leave the un-normalised O row and its (max, sum)
                const bool slot_in = ARB_IN_RANGE(a.status, w.slot + grp, a.split_cap);
                float *po = a.split_ws + (size_t)(slot_in ? w.slot + grp : 0) * kSlotFloats;
#pragma unroll 1
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint32_t v[32];
                    tmem_ld32(o_tmem + c4 * 32, v);
                    tmem_wait_ld();
                    if (row_ok && slot_in) {
                        if constexpr (E4M3) {   // values of an E4M3 cache are v_scale * code
#pragma unroll
                            for (int k = 0; k < 32; ++k) v[k] = __float_as_uint(__uint_as_float(v[k]) * a.v_scale);
                        }
#pragma unroll
                        for (int qd = 0; qd < 8; ++qd)
                            *reinterpret_cast<uint4 *>(po + ((size_t)(c4 * 8 + qd) * kBM + tg) * 4) =
                                make_uint4(v[qd * 4], v[qd * 4 + 1], v[qd * 4 + 2], v[qd * 4 + 3]);
                    }
                }
                if (row_ok && slot_in) *reinterpret_cast<float2 *>(po + (size_t)kBM * kD + tg * 2) = make_float2(m_used, l_sum);
                tc_fence_before();
                continue;
            }
            const float inv_l = (E4M3 ? a.v_scale : 1.0f) / l_sum;
            uint4 *dst = reinterpret_cast<uint4 *>(a.out + grow * 2);
#pragma unroll 1
            for (int c4 = 0; c4 < 4; ++c4) {
                uint32_t v[32];
                tmem_ld32(o_tmem + c4 * 32, v);
                tmem_wait_ld();
                if (row_ok && row_in) {
#pragma unroll
                    for (int qd = 0; qd < 4; ++qd) {
                        uint4 o4;
                        o4.x = pack_bf16(__uint_as_float(v[qd * 8 + 0]) * inv_l, __uint_as_float(v[qd * 8 + 1]) * inv_l);
                        o4.y = pack_bf16(__uint_as_float(v[qd * 8 + 2]) * inv_l, __uint_as_float(v[qd * 8 + 3]) * inv_l);
                        o4.z = pack_bf16(__uint_as_float(v[qd * 8 + 4]) * inv_l, __uint_as_float(v[qd * 8 + 5]) * inv_l);
                        o4.w = pack_bf16(__uint_as_float(v[qd * 8 + 6]) * inv_l, __uint_as_float(v[qd * 8 + 7]) * inv_l);
                        dst[c4 * 4 + qd] = o4;
                    }
                }
            }
            tc_fence_before();
        }
    }

    // ---- teardown: everyone is done with TMEM before the allocating warp frees it ------------------
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// ---- merge of the parts of split sequences -------------------------------------------------------------
// Runs behind chunk_mma_kernel on the stream.  Every CTA rebuilds the plan, then takes jobs in turn: a job
// is a quarter (32 dimensions) of one row tile of a split sequence, one thread per query row:
//     m = max_p m_p,  w_p = 2^(m_p - m),  out = sum_p w_p O_p / sum_p w_p l_p.
// Partials are laid out so that the threads of a warp (consecutive rows) read consecutive 16-byte pieces.
constexpr int kCombineThreads = kBM;
constexpr int kCombineDims = 32;    // dimensions of a row per job

template <int G>
__global__ void __launch_bounds__(kCombineThreads)
chunk_combine_kernel(const MmaArgs a) {
    extern __shared__ int plan_smem[];
    const Plan pl = plan_arrays(plan_smem, a.batch);
    const int tid = threadIdx.x;
    const int B = a.batch, Hkv = a.Hkv;
    pdl_enter();
    make_plan<G>(a, pl, tid, kCombineThreads, nullptr);
    constexpr int kQuarters = kD / kCombineDims;
    int job = 0;
    for (int r = 0; r < B; ++r) {
        const int P = pl.parts[r];
        if (P <= 1) continue;
        const int sb = pl.sorted[r], pairs = pl.pairs[sb];
        const int n = a.q_lens[sb], L = a.seq_lens[sb], rows_total = n * G;
        const int T = part_tiles(L, P);
        const int njobs = Hkv * pairs * 2 * kQuarters;
        // the jobs of this sequence that fall to this CTA
        int j = (int)blockIdx.x - job % (int)gridDim.x;
        if (j < 0) j += (int)gridDim.x;
        job += njobs;
        for (; j < njobs; j += (int)gridDim.x) {
            const int qd = j % kQuarters, jt = j / kQuarters;
            const int g = jt & 1, pt = (jt >> 1) % pairs, kvh = (jt >> 1) / pairs;
            const int r_begin = pt * 2 * kBM;
            const int rows_here = max(0, min(kBM, rows_total - r_begin - g * kBM));
            if (tid >= rows_here) continue;
            const int nt_pair = (pair_kv_len<G>(L, n, rows_total, r_begin) + kBN - 1) / kBN;
            const int nparts = min(P, (nt_pair + T - 1) / T);   // parts the pair sees something of
            const float *slot0 = a.split_ws + (size_t)(pl.sslot[r] + ((kvh * pairs + pt) * P) * 2 + g) * kSlotFloats;
            const size_t part_stride = 2 * kSlotFloats;
            float m = -INFINITY;
            for (int p = 0; p < nparts; ++p)
                m = fmaxf(m, __ldcg(slot0 + p * part_stride + (size_t)kBM * kD + tid * 2));   // part 0 sees key 0: finite
            float l = 0.f;
            float4 acc[kCombineDims / 4];
#pragma unroll
            for (int c = 0; c < kCombineDims / 4; ++c) acc[c] = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int p = 0; p < nparts; ++p) {
                const float *sp = slot0 + p * part_stride;
                float4 o[kCombineDims / 4];
#pragma unroll
                for (int c = 0; c < kCombineDims / 4; ++c)
                    o[c] = __ldcg(reinterpret_cast<const float4 *>(sp + ((size_t)(qd * (kCombineDims / 4) + c) * kBM + tid) * 4));
                const float2 ml = __ldcg(reinterpret_cast<const float2 *>(sp + (size_t)kBM * kD + tid * 2));
                const float w = fast_exp2(ml.x - m);
                l = fmaf(w, ml.y, l);
#pragma unroll
                for (int c = 0; c < kCombineDims / 4; ++c) {
                    acc[c].x = fmaf(w, o[c].x, acc[c].x);
                    acc[c].y = fmaf(w, o[c].y, acc[c].y);
                    acc[c].z = fmaf(w, o[c].z, acc[c].z);
                    acc[c].w = fmaf(w, o[c].w, acc[c].w);
                }
            }
            const int rr = r_begin + g * kBM + tid;
            const int tok = rr / G, head = rr - tok * G;
            const size_t grow = ((size_t)(pl.row0[sb] + tok) * a.Hq + kvh * G + head) * kD + (size_t)qd * kCombineDims;
            const float inv = 1.0f / l;
            uint4 *dst = reinterpret_cast<uint4 *>(a.out + grow * 2);
#pragma unroll
            for (int c = 0; c < kCombineDims / 8; ++c) {
                uint4 o4;
                o4.x = pack_bf16(acc[2 * c].x * inv, acc[2 * c].y * inv);
                o4.y = pack_bf16(acc[2 * c].z * inv, acc[2 * c].w * inv);
                o4.z = pack_bf16(acc[2 * c + 1].x * inv, acc[2 * c + 1].y * inv);
                o4.w = pack_bf16(acc[2 * c + 1].z * inv, acc[2 * c + 1].w * inv);
                dst[c] = o4;
            }
        }
    }
}

template <int G, bool E4M3>
arb_status launch_one(Ctx *ctx, const MmaArgs &a, const CUtensorMap &km, const CUtensorMap &vm, int max_items,
                      cudaStream_t stream) {
    const size_t smem = mma_smem_bytes(a.batch, E4M3);
    static bool attr_set[64] = {};
    if (!attr_set[ctx->device & 63]) {
        if (cudaFuncSetAttribute(chunk_mma_kernel<G, E4M3>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)mma_smem_bytes(E4M3 ? kMaxBatchE4m3 : kMaxBatch, E4M3)) != cudaSuccess)
            return ARB_ERR_CUDA;
        attr_set[ctx->device & 63] = true;
    }
    const int grid = max_items < ctx->num_sms ? max_items : ctx->num_sms;
    const cudaError_t err = launch_pdl(chunk_mma_kernel<G, E4M3>, dim3(grid), dim3(threads_of(E4M3)), smem, stream, a, km, vm);
    ctx->launches++;
    if (err != cudaSuccess) return ARB_ERR_CUDA;
    // the merge of split sequences, when the block table is long enough for a sequence to be split at all
    if (a.split_cap > 0) {
        const size_t csmem = sizeof(int) * (7 * (size_t)a.batch + 2);
        const cudaError_t cerr = launch_pdl(chunk_combine_kernel<G>, dim3(4 * ctx->num_sms), dim3(kCombineThreads), csmem, stream, a);
        ctx->launches++;
        if (cerr != cudaSuccess) return ARB_ERR_CUDA;
    }
    return ARB_OK;
}

}  // namespace

bool chunk_mma_supported(const arb_attn_params &p) {
    const int g = p.num_q_heads / p.num_kv_heads;
    return p.dtype == ARB_BF16 && p.head_dim == kD && p.max_q_len >= 2 && p.max_q_len * g >= kChunkMmaMinRows &&
           tma_available();
}

namespace {

arb_status launch_chunk_tc(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages, const void *v_pages,
                           bool e4m3, float k_scale, float v_scale, const int32_t *block_table, const int32_t *seq_lens,
                           const int32_t *q_lens, void *out, cudaStream_t stream) {
    alignas(64) CUtensorMap km, vm;
    const PoolView view = e4m3 ? PoolView::kE4m3 : PoolView::kBf16HalfRows;
    if (!pool_map(ctx, &km, k_pages, p.num_pages, p.num_kv_heads, view) ||
        !pool_map(ctx, &vm, v_pages, p.num_pages, p.num_kv_heads, view))
        return ARB_ERR_CUDA;
    MmaArgs a;
    a.q = static_cast<const char *>(q);
    a.k_pool = static_cast<const char *>(k_pages);
    a.v_pool = static_cast<const char *>(v_pages);
    a.block_table = block_table;
    a.seq_lens = seq_lens;
    a.q_lens = q_lens;
    a.out = static_cast<char *>(out);
    a.status = ctx->status;
    a.batch = p.batch;
    a.Hq = p.num_q_heads;
    a.Hkv = p.num_kv_heads;
    a.num_pages = p.num_pages;
    a.max_pages = p.max_pages_per_seq;
    a.rows = p.total_q;
    a.min_rows = kChunkMmaMinRows;
    a.work_counter = ctx->rot + (size_t)kRotSets * kRotCounters + kRotSets + 1;
    a.split_ws = ctx->chunk_ws;
    a.split_cap = (int)(ctx->chunk_ws_bytes / (kSlotFloats * sizeof(float)));
    // Can a sequence of this call be split at all?  Long ones from kSplitMinTiles tiles on; shorter ones only in a call
    // whose work items may fail to fill the machine.  The host knows the rows: at most `batch` of them are decode rows,
    // the others sit in row-tile pairs of 256, one work item per pair and KV head.
    const long long max_tiles = ((long long)p.max_pages_per_seq * kPage + kBN - 1) / kBN;
    const long long least_items = (long long)p.num_kv_heads * (((long long)p.total_q - p.batch) * (p.num_q_heads / p.num_kv_heads) / (2 * kBM));
    a.fill_ctas = (2 * least_items <= ctx->num_sms && max_tiles >= kFillMinTiles) ? ctx->num_sms : 0;
    if (max_tiles <= kSplitMinTiles && a.fill_ctas == 0) a.split_cap = 0;
    if (cudaMemsetAsync(a.work_counter, 0, 2 * sizeof(int), stream) != cudaSuccess) return ARB_ERR_CUDA;
    const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.head_dim);
    a.scale_log2 = scale * k_scale * 1.4426950408889634f;
    a.v_scale = v_scale;
    const int g = p.num_q_heads / p.num_kv_heads;
    // upper bound of the work items from what the host knows: every row could sit in its own tile run
    long long bound = (long long)p.num_kv_heads * ((long long)p.total_q * g / kBM + p.batch);
    if (a.split_cap > 0) bound *= kSplitMaxParts;   // every item of a split sequence comes once per part
    const int max_items = (int)(bound < 1 ? 1 : (bound > (1 << 30) ? (1 << 30) : bound));
    switch (e4m3 ? g + 8 : g) {
        case 1: return launch_one<1, false>(ctx, a, km, vm, max_items, stream);
        case 2: return launch_one<2, false>(ctx, a, km, vm, max_items, stream);
        case 3: return launch_one<3, false>(ctx, a, km, vm, max_items, stream);
        case 4: return launch_one<4, false>(ctx, a, km, vm, max_items, stream);
        case 5: return launch_one<5, false>(ctx, a, km, vm, max_items, stream);
        case 6: return launch_one<6, false>(ctx, a, km, vm, max_items, stream);
        case 7: return launch_one<7, false>(ctx, a, km, vm, max_items, stream);
        case 8: return launch_one<8, false>(ctx, a, km, vm, max_items, stream);
        case 9: return launch_one<1, true>(ctx, a, km, vm, max_items, stream);
        case 10: return launch_one<2, true>(ctx, a, km, vm, max_items, stream);
        case 11: return launch_one<3, true>(ctx, a, km, vm, max_items, stream);
        case 12: return launch_one<4, true>(ctx, a, km, vm, max_items, stream);
        case 13: return launch_one<5, true>(ctx, a, km, vm, max_items, stream);
        case 14: return launch_one<6, true>(ctx, a, km, vm, max_items, stream);
        case 15: return launch_one<7, true>(ctx, a, km, vm, max_items, stream);
        case 16: return launch_one<8, true>(ctx, a, km, vm, max_items, stream);
        default: return ARB_ERR_UNSUPPORTED;
    }
}

}  // namespace

arb_status launch_chunk_mma(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages,
                            const void *v_pages, const int32_t *block_table, const int32_t *seq_lens,
                            const int32_t *q_lens, void *out, cudaStream_t stream) {
    return launch_chunk_tc(ctx, p, q, k_pages, v_pages, false, 1.0f, 1.0f, block_table, seq_lens, q_lens, out, stream);
}

// step chunks over an E4M3 cache (q, out bf16): keys are k_scale * code, values v_scale * code
arb_status launch_chunk_e4m3(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_codes,
                             const void *v_codes, float k_scale, float v_scale, const int32_t *block_table,
                             const int32_t *seq_lens, const int32_t *q_lens, void *out, cudaStream_t stream) {
    if (p.num_q_heads / p.num_kv_heads > 8 || p.batch > kMaxBatchE4m3 || !tma_available()) return ARB_ERR_UNSUPPORTED;
    return launch_chunk_tc(ctx, p, q, k_codes, v_codes, true, k_scale, v_scale, block_table, seq_lens, q_lens, out, stream);
}

}  // namespace arb

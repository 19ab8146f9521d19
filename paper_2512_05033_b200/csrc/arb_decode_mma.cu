// Split-KV decode attention (q_len = 1), bf16, head_dim 128: the group's query heads are padded to
// the 16 rows of a warp-level tensor-core tile.
//
// Why tensor cores for a bandwidth-bound kernel: with CUDA-core FMAs a decode launch of the
// draft-shaped workload (group size 6) executes 6.3 M warp instructions for 34 MB of KV, 10.7 k issue
// slots per SM sub-partition, i.e. 5.4 us at one instruction per cycle -- as long as the 5.3 us the
// bytes need at HBM speed.  The FMA form is issue-bound there.  Here one page (16 keys) costs a warp
// 8 ldmatrix + 16 mma for q.K and the same for P.V, about a tenth of the instructions, so the kernel
// goes back to being bound by memory and latency.  The rows 8..15 of the tile stay zero (g <= 8).
//
// The streaming part is the scheme of the CUDA-core decode kernel: flat page list cut into equal
// ranges per CTA, one producer warp feeding a 16-stage ring, pages owned by one consumer warp each
// with its own online softmax.  Differences: K/V tiles arrive through tiled TMA copies as two 128-byte-swizzled
// halves of 16 rows x 64 dims (one box of a 3-D view of the pool brings both) so that ldmatrix reads them
// without bank conflicts; P is rounded
// to bf16 for the second product (and summed after rounding, so numerator and denominator agree);
// results of a segment are parked in shared memory and written out after the CTA's last page, so
// the wait for the previous kernel (programmatic dependent launch) comes once, after all streaming.
//
// The split combine is a kernel of its own (decode_combine_kernel, below), launched right behind
// as a programmatic dependent.  Measured per-CTA timelines are the reason: with the combine inside
// the decode kernel (partials, fence, arrival counter, last arriver reads everything back) the
// CTAs of a 34 MB call spent 3 to 15 us after their last page in dependent round trips to a
// loaded memory system, each holding 86 KB of shared memory that the next call's CTAs were
// waiting for.  Now a decode CTA stores its partials and leaves; the kernel boundary makes them
// visible, and the few light CTAs of the combine kernel are already resident when it happens.
//
// The same kernel, compiled a second time (template parameter E4M3), reads an E4M3 KV cache: one byte per
// element, half the bytes of the bf16 cache per token -- the only way past the bf16 cache's HBM roofline.
//   - a (page, kv head) tile is 16 rows x 128 bytes = 2 KB, one TMA box (128-byte swizzle); the ring has 40
//     stages (80 KB in flight per CTA against 64 KB of bf16 tiles);
//   - the codes are widened to f16, which holds every E4M3 value exactly (cvt.rn.f16x2.e4m3x2), and the
//     products run as f16 MMAs (fp32 accumulate); q is converted bf16 -> f16 once per segment, P is rounded to
//     f16 (11 significant bits) and summed after rounding;
//   - ldmatrix moves 16-bit units, i.e. pairs of codes.  For q.K a thread receives four consecutive dimensions
//     of one key per 8 x 16-byte matrix; they serve as the B fragment of a k-slice whose sixteen "k" positions
//     are the matrix's sixteen dimensions in the order 4t, 4t+1 | 4t+2, 4t+3 (t = lane mod 4), and q's A
//     fragment is loaded in the same order (a dot product does not care).  For P.V the transposed load gives a
//     thread the codes (key 2t: dims d, d+1 | key 2t+1: dims d, d+1); one byte permute sorts them into the B
//     fragments of two n-tiles, the even and the odd dimensions of a 16-dimension group, so a thread ends up
//     owning four consecutive output dimensions per group;
//   - the key scale is folded into the softmax scale, the value scale into the segment result.
#include "arb_decode_tc.cuh"

namespace arb {

namespace {

constexpr int kMaxConsWarps = 5;
constexpr int kGroup = 1;       // pages per consumer work group: with 16 stages every warp has two groups in flight
constexpr int kBatch = 16;      // producer lanes issuing side by side
// what differs between the bf16 cache and the E4M3 cache: the ring, and the number of consumer warps.  The E4M3 path
// is bound by its consumers (every code is widened to f16 on the way to the tensor core), so large calls run five.
template <bool E4M3>
struct Fmt {
    static constexpr int kTileBytes = kPage * kD * (E4M3 ? 1 : 2);   // 4 KB (two halves of 16 rows x 64 bf16) or
                                                                     // 2 KB (one box of 16 rows x 128 codes)
    static constexpr int kHalfTile = kTileBytes / 2;
    // consumer warps of a large call (two CTAs per SM stream at the memory system's pace); a small call, whose
    // pace is set by latencies, runs four either way (five are slower there: 7.3 against 7.0 us per call)
    static constexpr int kLargeCallWarps = E4M3 ? 5 : 4;
    static constexpr int kStages = E4M3 ? 40 : 16;                   // 64 KB of bf16 tiles, 80 KB of E4M3 tiles
    static constexpr int kRingBytes = kStages * kTileBytes;
    static_assert(kLargeCallWarps <= kMaxConsWarps, "warp records are sized for kMaxConsWarps");
    // a ring stage must always belong to the same warp
    static_assert(kStages % (kLargeCallWarps * 2 * kGroup) == 0 && kStages % (4 * 2 * kGroup) == 0, "stage ownership");
};
constexpr int kCtasPerSm = 2;
constexpr int kParked = 2;      // segment results parked in shared memory before they are written
static_assert(kBatch <= Fmt<false>::kStages, "two producer lanes of one turn must never wait on the same stage: the later "
                                            "one would be two phases ahead of the barrier and a parity wait cannot tell");

struct Args {
    const char *q;
    const int32_t *block_table;
    const int32_t *seq_lens;
    const int32_t *q_lens;
    char *out;
    float *part_o;    // [slots][G][D]
    float *part_ml;   // [slots][GP][2]
    uint32_t *status;
    int batch, Hq, Hkv, num_pages, max_pages;
    int small_ctas;   // CTAs a small call spreads over
    int whole_rows;   // the tensor maps are 3-D: one copy per page instead of one per half
    float scale_log2;   // softmax scale (times the key scale of an E4M3 cache) * log2(e)
    float v_scale;      // value scale of an E4M3 cache, 1 otherwise
    // workspace rotation (see launch_decode_mma): this call's generation number, the number of
    // workspace sets, the generation of the newest completed call
    int slots, rows;  // partial slots of a workspace set; rows of q and out (bounds-check build)
    uint32_t gen;
    int sets;
    int force_wait;
    unsigned *done_gen;
};

template <bool E4M3>
struct Tail {
    uint64_t full[Fmt<E4M3>::kStages];
    uint64_t empty[Fmt<E4M3>::kStages];
    int abort;
    int early;            // the workspace set is free: partials may be written before the predecessor is done
};

struct Parked {  // host-side view of what a parked segment needs besides its record
    int bk, nparts, c_first;
    size_t out_base;
};

template <int G>
struct Cfg {
    static constexpr int GP = (G + 3) / 4 * 4;
    static constexpr int REC = G * kD + 2 * GP;            // [m[GP] | l[GP] | o[G][D]]
    static constexpr int OSM_BYTES = kMaxConsWarps * REC * 4;
    static constexpr int PARK_BYTES = kParked * REC * 4;
};

template <int G, bool E4M3>
size_t smem_bytes(int batch) {
    using C = Cfg<G>;
    return 1024 + Fmt<E4M3>::kRingBytes + C::OSM_BYTES + C::PARK_BYTES + sizeof(Tail<E4M3>) + sizeof(int) * (3 * (size_t)batch + 2);
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
// two E4M3 codes (low 16 bits of v) -> f16x2, exact; the low byte lands in the low half
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t v) {
    uint32_t r;
    asm("{\n\t.reg .b16 c;\n\tcvt.u16.u32 c, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, c;\n\t}" : "=r"(r) : "r"(v));
    return r;
}
__device__ __forceinline__ uint32_t byte_perm(uint32_t v, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %1, %2;" : "=r"(r) : "r"(v), "r"(sel));
    return r;
}

// byte offset of 16-byte chunk `c` of row `r` inside a swizzled tile: 16 chunks across the 256-byte row of a
// bf16 tile (two halves of 64 dims), 8 chunks across the 128-byte row of codes of an E4M3 tile
template <bool E4M3>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
    if constexpr (E4M3) return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4));
    else return (uint32_t)((c >> 3) * Fmt<false>::kHalfTile + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

template <int G, bool E4M3, int CW>
__global__ void __launch_bounds__(CW * 32 + 32, kCtasPerSm)
decode_mma_kernel(const Args a, const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map) {
    using C = Cfg<G>;
    using Tail = arb::Tail<E4M3>;
    constexpr int kStages = Fmt<E4M3>::kStages, kTileBytes = Fmt<E4M3>::kTileBytes, kHalfTile = Fmt<E4M3>::kHalfTile;
    constexpr int kRingBytes = Fmt<E4M3>::kRingBytes;
    constexpr int kCW = CW, kCT = CW * 32, kNT = kCT + 32;   // consumer warps, their threads, + the producer warp
    static_assert(CW <= kMaxConsWarps && kStages % (CW * 2 * kGroup) == 0, "stage ownership");
    constexpr int GP = C::GP, REC = C::REC;
    static_assert(G >= 1 && G <= 8, "query heads of a group occupy rows 0..7 of the 16-row tile");

    extern __shared__ char smem_raw[];
    char *base = reinterpret_cast<char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    char *ring = base;
    float *osm = reinterpret_cast<float *>(base + kRingBytes);
    float *park = reinterpret_cast<float *>(base + kRingBytes + C::OSM_BYTES);
    Tail *tail = reinterpret_cast<Tail *>(base + kRingBytes + C::OSM_BYTES + C::PARK_BYTES);
    int *pref = reinterpret_cast<int *>(tail + 1);
    int *row0 = pref + a.batch + 1;
    int *slen = row0 + a.batch + 1;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.batch, Hkv = a.Hkv;

    // Until wait_for_predecessor() only inputs are read; every write to out, the workspace or the
    // arrival counters comes after it (see the CUDA-core decode kernel for the ordering argument).
    let_successor_start();

    if (tid == kCT) {  // the producer warp's first lane: descriptors on their way before the first copy needs them
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&k_map)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&v_map)) : "memory");
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&tail->full[s], 1);
            mbar_init(&tail->empty[s], 1);
        }
        tail->abort = 0;
        mbar_fence_init();
        pref[0] = 0;
        row0[0] = 0;
    }
    for (int b = tid; b < B; b += kNT) {
        const int n = a.q_lens[b], L = a.seq_lens[b];
        int pages = 0;
        if (n == 1) {
            if (L >= 1 && L <= a.max_pages * kPage) {
                pages = (L + kPage - 1) / kPage;
            } else if (blockIdx.x == 0) {
                wait_for_predecessor();
                atomicOr(a.status, (uint32_t)ARB_DEV_BAD_SEQ_LEN);
                int row = 0;
                for (int i = 0; i < b; ++i) row += max(a.q_lens[i], 0);
                __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(a.out) + (size_t)row * a.Hq * kD;
                for (int i = 0; i < a.Hq * kD; ++i) o[i] = __float2bfloat16_rn(0.f);
            }
        }
        pref[b + 1] = pages * Hkv;
        row0[b + 1] = n > 0 ? n : 0;
        slen[b] = L;
    }
    __syncthreads();
    if (warp == 0) {
        int carry_p = 0, carry_r = 0;
        for (int b0 = 0; b0 < B; b0 += 32) {
            const int b = b0 + lane;
            int vp = b < B ? pref[b + 1] : 0;
            int vr = b < B ? row0[b + 1] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int tp = __shfl_up_sync(0xffffffffu, vp, off);
                const int tr = __shfl_up_sync(0xffffffffu, vr, off);
                if (lane >= off) { vp += tp; vr += tr; }
            }
            if (b < B) { pref[b + 1] = vp + carry_p; row0[b + 1] = vr + carry_r; }
            carry_p += __shfl_sync(0xffffffffu, vp, 31);
            carry_r += __shfl_sync(0xffffffffu, vr, 31);
        }
    }
    __syncthreads();

    // Small calls use the first small_ctas CTAs of the grid (see plan_chunk); the other CTAs leave at
    // once and their places are free for the next call, which -- launched as a programmatic
    // dependent -- then streams its KV while this call is still computing.  Large calls use every
    // CTA: two per SM keep more bytes in flight.
    const int total = pref[B];
    const int chunk = plan_chunk(total, (int)gridDim.x, a.small_ctas);
    const long long r0l = (long long)blockIdx.x * chunk;
    if (r0l >= total) {
        // (CTA 0 only gets here when the call has no decode rows.)  One thread of CTA 0 always waits
        // for the previous kernel, so that calls complete in stream order.
        if (blockIdx.x == 0 && tid == 0) wait_for_predecessor();
        return;
    }
    const int r0 = (int)r0l;
    const int r1 = min(total, r0 + chunk);
    volatile int *abort = &tail->abort;

    if (warp == kCW) {
        // ================================ producer warp ==========================================
        uint32_t c = 0;
        int cur = r0;
        Segment s;
        while (next_segment(cur, r1, pref, slen, B, Hkv, chunk, s)) {
            for (int sp0 = s.pg0; sp0 < s.pg1; sp0 += 32) {
                const int np = min(32, s.pg1 - sp0);
                int pid = 0;
                if (lane < np && ARB_IN_RANGE(a.status, sp0 + lane, a.max_pages)) {
                    pid = a.block_table[(size_t)s.b * a.max_pages + sp0 + lane];
                    if ((unsigned)pid >= (unsigned)a.num_pages) {
                        atomicOr(a.status, (uint32_t)ARB_DEV_BAD_PAGE);
                        pid = 0;
                    }
                }
                const int full_tiles = (np / kGroup) * 2 * kGroup;
                const int rem = np % kGroup;
                const int ntiles = 2 * np;
#pragma unroll 1
                for (int i0 = 0; i0 < ntiles; i0 += kBatch) {
                    const int i = i0 + lane;
                    int page, is_v;
                    if (i < full_tiles) {
                        const int g = i / (2 * kGroup), r = i - g * 2 * kGroup;
                        is_v = r / kGroup;
                        page = g * kGroup + (r - is_v * kGroup);
                    } else {
                        const int r = i - full_tiles, d = rem > 0 ? rem : 1;
                        is_v = r / d;
                        page = (np / kGroup) * kGroup + (r - is_v * d);
                    }
                    const int pg = __shfl_sync(0xffffffffu, pid, page & 31);
                    if (lane < kBatch && i < ntiles) {
                        const uint32_t cc = c + i, st = cc % kStages, par = (cc / kStages) & 1u;
                        const CUtensorMap *map = is_v ? &v_map : &k_map;
                        if (mbar_wait(&tail->empty[st], par ^ 1u, abort, a.status)) {
                            mbar_arrive_expect_tx(&tail->full[st], kTileBytes);
                            const int row = (pg * Hkv + s.kvh) * kPage;
                            if (!E4M3 && a.whole_rows) {
                                tma_box_load3(ring + st * kTileBytes, map, 0, row, 0, &tail->full[st]);
                            } else {
                                tma_box_load(ring + st * kTileBytes, map, 0, row, &tail->full[st]);
                                if constexpr (!E4M3) tma_box_load(ring + st * kTileBytes + kHalfTile, map, 64, row, &tail->full[st]);
                            }
                        }
                    }
                    __syncwarp();
                }
                c += ntiles;
            }
        }
        if (lane == 0 && *abort) {
            const uint32_t n = c < (uint32_t)kStages ? c : (uint32_t)kStages;
            for (uint32_t i = 0; i < n; ++i) {
                const uint32_t cc = c - 1 - i;
                const long long t0 = clock64();
                while (!mbar_try_wait(&tail->full[cc % kStages], (cc / kStages) & 1u) && clock64() - t0 < (1ll << 24)) {
                }
            }
        }
        return;
    }

    // ==================================== consumer warps ==========================================
    const int gq = lane >> 2, tq = lane & 3;   // fragment coordinates: row / column pair
    const bool row_ok = gq < G;                // this lane's row is a real query head
    const uint32_t ring_addr = smem_u32(ring);
    uint32_t seg_base = 0;
    int cur = r0;
    Segment s;
    int n_parked = 0;
    Parked pk[kParked];

    // Ordering against the previous kernel on the stream.  Writes to `out` always wait for it
    // (griddepcontrol.wait, once per CTA, and only in CTAs that have something to write there, plus
    // CTA 0, which keeps the calls completing in stream order).  Writes to the workspace wait for it
    // too, unless the call owns a workspace set that no unfinished call can still be reading: sets
    // rotate with the call's generation number, and the combine kernel of every call publishes the
    // generation in *done_gen when it is through.
    bool waited = false;
    auto ensure_wait = [&]() {
        if (!waited) { wait_for_predecessor(); waited = true; }
    };
    // The set is free when the newest completed call lies in [gen - sets, gen - 1]: calls complete in
    // stream order, so the set's previous user (gen - sets) is among the completed.  A value outside
    // the window -- in particular a newer generation left behind by an earlier replay of a captured
    // graph, whose generations repeat -- proves nothing and the CTA waits instead.
    const bool may_early = a.sets >= 3 && !a.force_wait;
    auto set_is_free = [&]() -> bool {
        unsigned d;
        asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(d) : "l"(a.done_gen) : "memory");
        return (uint32_t)(a.gen - 1u - d) < (uint32_t)a.sets;
    };
    bool early_known = false;   // thread 0 only; looked up now so that the answer is there when it is needed
    if (tid == 0 && may_early) early_known = set_is_free();
    // Publishes the parked segment results.  Parts of split (sequence, head)s go to the workspace as
    // partials (the combine kernel that follows merges them); results that are already final are
    // written to `out` -- at once in the middle of a range (`last_call` false), or left parked for
    // the epilogue, after the wait.
    auto flush = [&](bool last_call) {
        bool any_multi = false, any_single = false;
        for (int j = 0; j < n_parked; ++j) {
            any_multi = any_multi || pk[j].nparts > 1;
            any_single = any_single || pk[j].nparts == 1;
        }
        if (any_multi) {
            if (tid == 0) {
                if (may_early && !early_known) early_known = set_is_free();
                tail->early = early_known ? 1 : 0;
            }
            named_barrier(1, kCT);
            if (!tail->early) ensure_wait();
            for (int j = 0; j < n_parked; ++j) {
                if (pk[j].nparts == 1) continue;
                const float *rec = park + j * REC;
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
        if (!last_call) {
            if (any_single) ensure_wait();
            for (int j = 0; j < n_parked; ++j) {
                if (pk[j].nparts != 1) continue;
                const float *rec = park + j * REC;
                for (int idx = tid; idx < G * kD; idx += kCT)
                    reinterpret_cast<__nv_bfloat16 *>(a.out)[pk[j].out_base + idx] =
                        __float2bfloat16_rn(rec[2 * GP + idx] / rec[GP + idx / kD]);
            }
            named_barrier(1, kCT);  // parking slots are free again
            n_parked = 0;
        }
    };

    while (next_segment(cur, r1, pref, slen, B, Hkv, chunk, s)) {
        const int qrow = row0[s.b];
        if constexpr (!E4M3) {
            // ---- bf16 cache: the transposed products.  S^T = K q^T puts the 16 keys of a page on the rows of the
            //      m16n8k16 tile and the group's heads (padded to 8) on its columns, O^T += V^T P^T likewise: 8 + 8
            //      MMAs per page instead of 16 + 16 and half the accumulator registers.  P^T reaches the second
            //      product's B fragment through two movmatrix transposes; the row maximum is a reduction over the
            //      lanes that share a column pair (three shuffles).
            const bool head_ok = gq < G;               // as a B-fragment column: this lane's head is a real one
            const int h0 = 2 * tq, h1 = 2 * tq + 1;    // as accumulator columns: the two heads this lane holds
            uint32_t qb[8][2];                         // k-slice ks: dims 16 ks + 2 tq, + 1 and + 8 of head gq
            {
                const char *qh = a.q + ((size_t)qrow * a.Hq + s.kvh * G + (head_ok ? gq : 0)) * kD * 2;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    qb[ks][0] = head_ok ? __ldg(reinterpret_cast<const uint32_t *>(qh + ks * 32 + tq * 4)) : 0u;
                    qb[ks][1] = head_ok ? __ldg(reinterpret_cast<const uint32_t *>(qh + ks * 32 + 16 + tq * 4)) : 0u;
                }
            }
            // running max of heads h0, h1 (the same in the 8 lanes of a column pair), this lane's share of their sums,
            // and 8 m-tiles of O^T: o[mt][0..1] = dim 16 mt + gq of heads h0, h1; o[mt][2..3] = dim + 8
            float m_run0 = -INFINITY, m_run1 = -INFINITY, l_run0 = 0.f, l_run1 = 0.f;
            float o[8][4];
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) { o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f; }
            const int seg_pages = s.pg1 - s.pg0;
            for (int gi = warp; gi < seg_pages; gi += kCW) {
                const int pg = s.pg0 + gi;
                const int ntok = min(s.L - pg * kPage, kPage);
                const uint32_t ck = seg_base + 2u * (uint32_t)gi;
                float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};   // two chains, four deep
                {
                    const uint32_t st = ck % kStages, par = (ck / kStages) & 1u;
                    mbar_wait(&tail->full[st], par, abort, a.status);
                    const uint32_t tile = ring_addr + st * kTileBytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        uint32_t af[4];   // rows: keys; matrices: (keys 0-7 | 8-15) x (dims 16 ks + 0-7 | 8-15)
                        ldmatrix_x4(tile + tile_off<false>((lane & 7) + ((lane >> 3) & 1) * 8, 2 * ks + (lane >> 4)), af);
                        if (ks & 1) mma_16816<false>(sb, af, qb[ks][0], qb[ks][1]);
                        else mma_16816<false>(sa, af, qb[ks][0], qb[ks][1]);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tail->empty[st]);
                }
                const bool k0 = gq < ntok, k1 = gq + 8 < ntok;   // this lane has keys gq and gq + 8
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
                const float f0 = fast_exp2(m_run0 - mn0), f1 = fast_exp2(m_run1 - mn1);
                m_run0 = mn0;
                m_run1 = mn1;
                // P^T, rounded to bf16; the sums use the rounded weights, like the tensor core
                const uint32_t w0 = pack_bf16(fast_exp2(s00 - mn0), fast_exp2(s01 - mn1));   // key gq: heads h0, h1
                const uint32_t w1 = pack_bf16(fast_exp2(s10 - mn0), fast_exp2(s11 - mn1));   // key gq + 8
                l_run0 = fmaf(l_run0, f0, __uint_as_float(w0 << 16) + __uint_as_float(w1 << 16));
                l_run1 = fmaf(l_run1, f1, __uint_as_float(w0 & 0xffff0000u) + __uint_as_float(w1 & 0xffff0000u));
                const uint32_t pb0 = movmatrix_trans(w0), pb1 = movmatrix_trans(w1);   // keys 2 tq, + 1 (and + 8) of head gq
                if (__any_sync(0xffffffffu, f0 != 1.0f || f1 != 1.0f)) {
#pragma unroll
                    for (int mt = 0; mt < 8; ++mt) { o[mt][0] *= f0; o[mt][1] *= f1; o[mt][2] *= f0; o[mt][3] *= f1; }
                }
                {
                    const uint32_t cv = ck + 1u, st = cv % kStages, par = (cv / kStages) & 1u;
                    mbar_wait(&tail->full[st], par, abort, a.status);
                    if (ntok < kPage) {
                        // slots past the sequence end may hold anything; they must not reach the tensor core, not
                        // even times zero: blank them in shared memory
                        for (int i = lane; i < (kPage - ntok) * 16; i += 32)
                            *reinterpret_cast<uint4 *>(ring + st * kTileBytes + tile_off<false>(ntok + (i >> 4), i & 15)) = make_uint4(0, 0, 0, 0);
                        __syncwarp();
                    }
                    const uint32_t tile = ring_addr + st * kTileBytes;
#pragma unroll
                    for (int mt = 0; mt < 8; ++mt) {
                        uint32_t af[4];   // transposed on the way: rows dims (16 mt + 0-7 | 8-15), columns keys (0-7 | 8-15)
                        ldmatrix_x4_trans(tile + tile_off<false>((lane & 7) + (lane >> 4) * 8, 2 * mt + ((lane >> 3) & 1)), af);
                        mma_16816<false>(o[mt], af, pb0, pb1);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tail->empty[st]);
                }
            }
            seg_base += 2u * (uint32_t)seg_pages;
            // ---- segment end: every warp leaves (max, sum, accumulators) in the record layout the merge reads
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l_run0 += __shfl_xor_sync(0xffffffffu, l_run0, off);
                l_run1 += __shfl_xor_sync(0xffffffffu, l_run1, off);
            }
            float *rec = osm + warp * REC;
            if (gq == 0) {
                if (h0 < G) { rec[h0] = m_run0; rec[GP + h0] = l_run0; }
                if (h1 < G) { rec[h1] = m_run1; rec[GP + h1] = l_run1; }
            }
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
                const int d = 16 * mt + gq;
                if (h0 < G) { rec[2 * GP + h0 * kD + d] = o[mt][0]; rec[2 * GP + h0 * kD + d + 8] = o[mt][2]; }
                if (h1 < G) { rec[2 * GP + h1 * kD + d] = o[mt][1]; rec[2 * GP + h1 * kD + d + 8] = o[mt][3]; }
            }
        } else {
            // A fragments of q (16 x 128, rows >= G zero): 8 k-slices of 16 dims.  E4M3 cache: converted to f16, and
            // k-slice ks holds dims 16 ks .. 16 ks + 15 in the order the widened codes arrive in: this lane has dims
            // 16 ks + 4 tq + {0, 1} (k = 2 tq, + 1) and + {2, 3} (k = 8 + 2 tq, + 1)
            uint32_t qa[8][4];
            {
                const char *qh = a.q + ((size_t)qrow * a.Hq + s.kvh * G + gq) * kD * 2;
    #pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    if constexpr (E4M3) {
                        const uint2 raw = row_ok ? __ldg(reinterpret_cast<const uint2 *>(qh + ks * 32 + tq * 8)) : make_uint2(0u, 0u);
                        qa[ks][0] = pack_f16(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u));
                        qa[ks][2] = pack_f16(__uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u));
                    } else {
                        qa[ks][0] = row_ok ? __ldg(reinterpret_cast<const uint32_t *>(qh + ks * 32 + tq * 4)) : 0u;
                        qa[ks][2] = row_ok ? __ldg(reinterpret_cast<const uint32_t *>(qh + ks * 32 + 16 + tq * 4)) : 0u;
                    }
                    qa[ks][1] = 0u;
                    qa[ks][3] = 0u;
                }
            }
            // this lane's row (head gq): running max (the same in the 4 lanes of a row), its share of the
            // sum, and 16 n-tiles of the output row: o[n][0..1] = dims 8n + 2 tq, + 1 (o[n][2..3]: rows 8..15); with an E4M3
            // cache o[2c][0..1] = dims 16c + 4 tq, + 2 and o[2c+1][0..1] = dims 16c + 4 tq + 1, + 3
            float m_run = -INFINITY, l_run = 0.f;
            float o[16][4];
    #pragma unroll
            for (int n = 0; n < 16; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }

            const int seg_pages = s.pg1 - s.pg0;
            const int ngroups = (seg_pages + kGroup - 1) / kGroup;
            for (int gi = warp; gi < ngroups; gi += kCW) {
                const int p0 = s.pg0 + gi * kGroup;
                const int npg = min(kGroup, s.pg1 - p0);
                const int ntok = min(s.L - p0 * kPage, npg * kPage);
                const uint32_t gbase = seg_base + (uint32_t)gi * 2 * kGroup;

                // ---- S = q K^T for the group's pages: per page two n-tiles of 8 keys -----------------
                float sc[kGroup * 2][4];
    #pragma unroll
                for (int t = 0; t < kGroup; ++t) {
    #pragma unroll
                    for (int j = 0; j < 2; ++j) { sc[t * 2 + j][0] = sc[t * 2 + j][1] = sc[t * 2 + j][2] = sc[t * 2 + j][3] = 0.f; }
                    if (t < npg) {
                        const uint32_t cc = gbase + t, st = cc % kStages, par = (cc / kStages) & 1u;
                        mbar_wait(&tail->full[st], par, abort, a.status);
                        const uint32_t tile = ring_addr + st * kTileBytes;
    #pragma unroll
                        for (int j = 0; j < 2; ++j) {          // keys 8j .. 8j+7 of the page
                            if constexpr (E4M3) {
    #pragma unroll
                                for (int kq = 0; kq < 2; ++kq) {   // k-slices 4kq .. 4kq + 3: one 16-byte chunk of codes each
                                    uint32_t bfr[4];
                                    ldmatrix_x4(tile + tile_off<true>(8 * j + (lane & 7), 4 * kq + (lane >> 3)), bfr);
    #pragma unroll
                                    for (int i = 0; i < 4; ++i)
                                        mma_16816<true>(sc[t * 2 + j], qa[4 * kq + i], e4m3x2_to_f16x2(bfr[i]),
                                                        e4m3x2_to_f16x2(bfr[i] >> 16));
                                }
                            } else {
    #pragma unroll
                                for (int kp = 0; kp < 4; ++kp) {   // k-slices 2kp, 2kp+1
                                    uint32_t bfr[4];
                                    ldmatrix_x4(tile + tile_off<false>(8 * j + (lane & 7), 4 * kp + (lane >> 3)), bfr);
                                    mma_16816<false>(sc[t * 2 + j], qa[2 * kp], bfr[0], bfr[1]);
                                    mma_16816<false>(sc[t * 2 + j], qa[2 * kp + 1], bfr[2], bfr[3]);
                                }
                            }
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&tail->empty[st]);
                    }
                }

                // ---- online softmax on the fragments: this lane has 2 scores per n-tile of its row ------
                float mx = -INFINITY;
    #pragma unroll
                for (int nt = 0; nt < kGroup * 2; ++nt) {
    #pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int key = nt * 8 + tq * 2 + e;
                        const float v = (key < ntok) ? sc[nt][e] * a.scale_log2 : -INFINITY;
                        sc[nt][e] = v;
                        mx = fmaxf(mx, v);
                    }
                }
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run, mx);            // finite: the group has a visible key
                const float f = fast_exp2(m_run - m_new);        // 0 for the first group
                m_run = m_new;
                uint32_t pa[kGroup][4];                          // A fragments of P: one k-slice per page
                float lsum = 0.f;
    #pragma unroll
                for (int t = 0; t < kGroup; ++t) {
                    const float p00 = fast_exp2(sc[2 * t][0] - m_new), p01 = fast_exp2(sc[2 * t][1] - m_new);
                    const float p10 = fast_exp2(sc[2 * t + 1][0] - m_new), p11 = fast_exp2(sc[2 * t + 1][1] - m_new);
                    const uint32_t w0 = E4M3 ? pack_f16(p00, p01) : pack_bf16(p00, p01);
                    const uint32_t w1 = E4M3 ? pack_f16(p10, p11) : pack_bf16(p10, p11);
                    pa[t][0] = w0;   // row gq, keys 2 tq, +1
                    pa[t][2] = w1;   // row gq, keys 8 + 2 tq, +1
                    pa[t][1] = 0u;   // rows 8..15
                    pa[t][3] = 0u;
                    // the sum uses the rounded weights, like the tensor core
                    if constexpr (E4M3) {
                        const float2 r0 = unpack_f16(w0), r1 = unpack_f16(w1);
                        lsum += (r0.x + r0.y) + (r1.x + r1.y);
                    } else {
                        lsum += __uint_as_float(w0 << 16) + __uint_as_float(w0 & 0xffff0000u) +
                                __uint_as_float(w1 << 16) + __uint_as_float(w1 & 0xffff0000u);
                    }
                }
                l_run = fmaf(l_run, f, lsum);
                if (__any_sync(0xffffffffu, f != 1.0f)) {
    #pragma unroll
                    for (int n = 0; n < 16; ++n) { o[n][0] *= f; o[n][1] *= f; }
                }

                // ---- O += P V: per page 16 n-tiles of 8 dims, one k-slice of 16 keys ------------------
    #pragma unroll
                for (int t = 0; t < kGroup; ++t) {
                    if (t < npg) {
                        const uint32_t cc = gbase + npg + t, st = cc % kStages, par = (cc / kStages) & 1u;
                        mbar_wait(&tail->full[st], par, abort, a.status);
                        const uint32_t tile = ring_addr + st * kTileBytes;
                        const int nvalid = ntok - t * kPage;
                        if (nvalid < kPage) {
                            // slots past the sequence end may hold anything; they must not reach the
                            // tensor core, not even times zero: blank them in shared memory
                            constexpr int kRowChunks = kTileBytes / kPage / 16;   // 16-byte chunks of a row: 16 or 8
                            for (int i = lane; i < (kPage - nvalid) * kRowChunks; i += 32) {
                                const int r = nvalid + i / kRowChunks, c = i % kRowChunks;
                                *reinterpret_cast<uint4 *>(ring + st * kTileBytes + tile_off<E4M3>(r, c)) = make_uint4(0, 0, 0, 0);
                            }
                            __syncwarp();
                        }
    #pragma unroll
                        for (int np2 = 0; np2 < (E4M3 ? 4 : 8); ++np2) {    // two 16-byte chunks of a row: 16 dims, or 32 dims of codes
                            uint32_t bfr[4];
                            // blocks: (keys 0-7, chunk 2np2), (keys 8-15, 2np2), (keys 0-7, 2np2+1), (keys 8-15, 2np2+1)
                            ldmatrix_x4_trans(tile + tile_off<E4M3>((lane & 7) + ((lane >> 3) & 1) * 8, 2 * np2 + (lane >> 4)), bfr);
                            if constexpr (E4M3) {
                                // a lane has (key 2tq: dims d, d+1 | key 2tq+1: dims d, d+1) with d = 16 chunk + 2 gq
    #pragma unroll
                                for (int h = 0; h < 2; ++h) {      // chunk 2np2 + h
                                    // bytes -> (key 2tq, key 2tq+1) of dim d | the same of dim d + 1
                                    const uint32_t lo = byte_perm(bfr[2 * h], 0x3120u), hi = byte_perm(bfr[2 * h + 1], 0x3120u);
                                    mma_16816<true>(o[4 * np2 + 2 * h], pa[t], e4m3x2_to_f16x2(lo), e4m3x2_to_f16x2(hi));
                                    mma_16816<true>(o[4 * np2 + 2 * h + 1], pa[t], e4m3x2_to_f16x2(lo >> 16), e4m3x2_to_f16x2(hi >> 16));
                                }
                            } else {
                                mma_16816<false>(o[2 * np2], pa[t], bfr[0], bfr[1]);
                                mma_16816<false>(o[2 * np2 + 1], pa[t], bfr[2], bfr[3]);
                            }
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&tail->empty[st]);
                    }
                }
            }
            seg_base += 2u * (uint32_t)seg_pages;

            // ---- segment end: every warp leaves (max, sum, row accumulators); all threads merge them ------
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
            float *rec = osm + warp * REC;
            if (row_ok) {
    #pragma unroll
                if constexpr (E4M3) {
                    for (int c = 0; c < 8; ++c)   // four consecutive dims per 16-dim group
                        *reinterpret_cast<float4 *>(rec + 2 * GP + gq * kD + 16 * c + 4 * tq) =
                            make_float4(o[2 * c][0], o[2 * c + 1][0], o[2 * c][1], o[2 * c + 1][1]);
                } else {
                    for (int n = 0; n < 16; ++n)
                        *reinterpret_cast<float2 *>(rec + 2 * GP + gq * kD + 8 * n + tq * 2) = make_float2(o[n][0], o[n][1]);
                }
                if (tq == 0) { rec[gq] = m_run; rec[GP + gq] = l_run; }
            }
        }
        if (n_parked == kParked) flush(false);  // uniform across the consumer threads
        named_barrier(1, kCT);
        float *dst = park + n_parked * REC;
        for (int idx = tid; idx < G * kD; idx += kCT) {
            const int h = idx / kD;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kCW; ++w) M = fmaxf(M, osm[w * REC + h]);
            float l = 0.f, acc = 0.f;
#pragma unroll
            for (int w = 0; w < kCW; ++w) {
                const float ff = fast_exp2(osm[w * REC + h] - M);  // 0 for a warp that had no group
                l = fmaf(ff, osm[w * REC + GP + h], l);
                acc = fmaf(ff, osm[w * REC + 2 * GP + idx], acc);
            }
            dst[2 * GP + idx] = E4M3 ? acc * a.v_scale : acc;   // values of an E4M3 cache are v_scale * code
            if (idx - h * kD == 0) { dst[h] = M; dst[GP + h] = l; }
        }
        pk[n_parked].bk = s.bk;
        pk[n_parked].nparts = s.nparts;
        pk[n_parked].c_first = s.c_first;
        pk[n_parked].out_base = ((size_t)qrow * a.Hq + s.kvh * G) * kD;
        ++n_parked;
        named_barrier(1, kCT);  // warp records are free for the next segment
    }
    if (n_parked > 0) flush(true);  // final results stay parked until the epilogue

    // ---- epilogue: what goes to `out` waits for the previous kernel.  A CTA that only produced parts
    //      of split (sequence, head)s has nothing to write there and leaves at once, freeing its
    //      place on the SM for the next call.
    bool any_single = false;
    for (int j = 0; j < n_parked; ++j) any_single = any_single || pk[j].nparts == 1;
    if (any_single || blockIdx.x == 0) ensure_wait();
    for (int j = 0; j < n_parked; ++j) {
        if (pk[j].nparts != 1) continue;
        if (!ARB_IN_RANGE(a.status, pk[j].out_base + G * kD - 1, (size_t)a.rows * a.Hq * kD)) continue;
        const float *rec = park + j * REC;
        for (int idx = tid; idx < G * kD; idx += kCT)
            reinterpret_cast<__nv_bfloat16 *>(a.out)[pk[j].out_base + idx] =
                __float2bfloat16_rn(rec[2 * GP + idx] / rec[GP + idx / kD]);
    }
}

// ---- split combine ---------------------------------------------------------------------------------
// Launched right behind the decode kernel as its programmatic dependent: its CTAs come up while the
// decode kernel is still streaming, work out the same plan from the lengths, and then wait for the
// decode kernel to complete (griddepcontrol.wait), which makes every partial visible without a fence,
// an arrival counter or a CTA of the decode kernel staying behind.  One work item is a split
// (sequence, kv head); a thread merges one or two 4-dimension pieces of the group's G x 128 outputs
// over the parts,
//     m = max_p m_p,  w_p = 2^(m_p - m),  out = sum_p w_p o_p / sum_p w_p l_p.
// Few, light CTAs on purpose: they sit on the SMs, waiting, while decode CTAs of this and of the
// next call need the room.  The last CTA to finish publishes the call's generation (see the
// workspace rotation).
constexpr int kCombineThreads = 128;
constexpr int kCombinePreload = 4;   // parts whose values are asked for before the weights are known

struct CombineArgs {
    const int32_t *seq_lens;
    const int32_t *q_lens;
    char *out;
    const float *part_o;
    const float *part_ml;
    int batch, Hq, Hkv, max_pages;
    int small_ctas, decode_grid;
    uint32_t gen;
    unsigned *done_gen;
    int *exit_count;
};

template <int G>
__global__ void __launch_bounds__(kCombineThreads)
decode_combine_kernel(const CombineArgs a) {
    constexpr int GP = (G + 3) / 4 * 4;
    constexpr int VECS = G * kD / 4;                                       // float4 pieces of one partial output
    constexpr int NE = (VECS + kCombineThreads - 1) / kCombineThreads;     // pieces per thread (1 or 2)
    extern __shared__ int csm[];
    int *pref = csm;                      // [B + 1] pages (times kv heads) before sequence b
    int *row0 = pref + a.batch + 1;       // [B + 1] q rows before sequence b
    float2 *ml_s = reinterpret_cast<float2 *>(row0 + a.batch + 1);   // [parts][G] (max, sum); 2 (B + 1) ints before it
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.batch, Hkv = a.Hkv;

    let_successor_start();
    if (tid == 0) { pref[0] = 0; row0[0] = 0; }
    for (int b = tid; b < B; b += kCombineThreads) {
        const int n = a.q_lens[b], L = a.seq_lens[b];
        const int pages = (n == 1 && L >= 1 && L <= a.max_pages * kPage) ? (L + kPage - 1) / kPage : 0;
        pref[b + 1] = pages * Hkv;
        row0[b + 1] = n > 0 ? n : 0;
    }
    __syncthreads();
    if (warp == 0) {
        int carry_p = 0, carry_r = 0;
        for (int b0 = 0; b0 < B; b0 += 32) {
            const int b = b0 + lane;
            int vp = b < B ? pref[b + 1] : 0;
            int vr = b < B ? row0[b + 1] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int tp = __shfl_up_sync(0xffffffffu, vp, off);
                const int tr = __shfl_up_sync(0xffffffffu, vr, off);
                if (lane >= off) { vp += tp; vr += tr; }
            }
            if (b < B) { pref[b + 1] = vp + carry_p; row0[b + 1] = vr + carry_r; }
            carry_p += __shfl_sync(0xffffffffu, vp, 31);
            carry_r += __shfl_sync(0xffffffffu, vr, 31);
        }
    }
    __syncthreads();
    const int total = pref[B];
    const int chunk = plan_chunk(total, a.decode_grid, a.small_ctas);

    wait_for_predecessor();   // the decode kernel of this call, and with it every earlier call

    int ev[NE], eh[NE];       // this thread's pieces: index into a partial output, and its head
    bool eok[NE];
#pragma unroll
    for (int k = 0; k < NE; ++k) {
        const int e = tid + k * kCombineThreads;
        eok[k] = e < VECS;
        ev[k] = eok[k] ? e : 0;
        eh[k] = ev[k] / (kD / 4);
    }
    for (int bk = blockIdx.x; bk < B * Hkv; bk += gridDim.x) {
        const int b = bk / Hkv, kvh = bk - b * Hkv;
        const int pages = (pref[b + 1] - pref[b]) / Hkv;
        if (pages == 0) continue;
        const int s0 = pref[b] + kvh * pages, s1 = s0 + pages;
        const int c_first = s0 / chunk;
        const int nparts = (s1 - 1) / chunk - c_first + 1;   // at most one per CTA of the decode grid
        if (nparts <= 1) continue;       // the decode kernel wrote this one itself
        const size_t slot0 = (size_t)bk + c_first;
        const float4 *po = reinterpret_cast<const float4 *>(a.part_o + slot0 * G * kD);
        // the first partial values are asked for before the weights exist, so that the two round
        // trips to memory run side by side
        float4 v[NE][kCombinePreload];
#pragma unroll
        for (int u = 0; u < kCombinePreload; ++u)
#pragma unroll
            for (int k = 0; k < NE; ++k) v[k][u] = __ldcg(po + (size_t)min(u, nparts - 1) * VECS + ev[k]);
        __syncthreads();                 // ml_s of the previous item has been read by everyone
        for (int i = tid; i < nparts * G; i += kCombineThreads) {
            const int p = i / G, h = i - p * G;
            ml_s[i] = __ldcg(reinterpret_cast<const float2 *>(a.part_ml + ((slot0 + p) * GP + h) * 2));
        }
        __syncthreads();
        float m[NE], l[NE];
        float4 x[NE];
#pragma unroll
        for (int k = 0; k < NE; ++k) {
            m[k] = -INFINITY;
            for (int p = 0; p < nparts; ++p) m[k] = fmaxf(m[k], ml_s[p * G + eh[k]].x);
            l[k] = 0.f;
            x[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int p0 = 0; p0 < nparts; p0 += kCombinePreload) {
            if (p0 > 0) {
#pragma unroll
                for (int u = 0; u < kCombinePreload; ++u)
#pragma unroll
                    for (int k = 0; k < NE; ++k) v[k][u] = __ldcg(po + (size_t)min(p0 + u, nparts - 1) * VECS + ev[k]);
            }
#pragma unroll
            for (int u = 0; u < kCombinePreload; ++u) {
                if (p0 + u < nparts) {
#pragma unroll
                    for (int k = 0; k < NE; ++k) {
                        const float2 ml = ml_s[(p0 + u) * G + eh[k]];
                        const float w = fast_exp2(ml.x - m[k]);
                        l[k] = fmaf(w, ml.y, l[k]);
                        x[k].x = fmaf(w, v[k][u].x, x[k].x);
                        x[k].y = fmaf(w, v[k][u].y, x[k].y);
                        x[k].z = fmaf(w, v[k][u].z, x[k].z);
                        x[k].w = fmaf(w, v[k][u].w, x[k].w);
                    }
                }
            }
        }
        __nv_bfloat16 *orow = reinterpret_cast<__nv_bfloat16 *>(a.out) + ((size_t)row0[b] * a.Hq + kvh * G) * kD;
#pragma unroll
        for (int k = 0; k < NE; ++k) {
            if (eok[k]) {
                const float inv = 1.0f / l[k];
                uint2 o2;
                o2.x = pack_bf16(x[k].x * inv, x[k].y * inv);
                o2.y = pack_bf16(x[k].z * inv, x[k].w * inv);
                *reinterpret_cast<uint2 *>(orow + (size_t)ev[k] * 4) = o2;
            }
        }
    }
    // The last CTA through publishes this call's generation: its workspace set has been read for the
    // last time, and every earlier call has completed (every CTA here waited for the decode kernel,
    // whose CTA 0 waited for the kernel before it).
    __syncthreads();
    if (tid == 0) {
        const int old = atomicAdd(a.exit_count, 1);
        if (old == (int)gridDim.x - 1) {
            *a.exit_count = 0;
            __threadfence();
            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(a.done_gen), "r"(a.gen) : "memory");
        }
    }
}

template <int G, bool E4M3>
arb_status launch_one(Ctx *ctx, const Args &a, CombineArgs ca, const CUtensorMap &km, const CUtensorMap &vm,
                      bool overlap, cudaStream_t stream) {
    const size_t smem = smem_bytes<G, E4M3>(a.batch);
    constexpr int kLarge = Fmt<E4M3>::kLargeCallWarps;
    static bool attr_set[64] = {};
    if (!attr_set[ctx->device & 63]) {
        const int most = (int)smem_bytes<G, E4M3>(kMaxBatch);
        if (cudaFuncSetAttribute(decode_mma_kernel<G, E4M3, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess ||
            cudaFuncSetAttribute(decode_mma_kernel<G, E4M3, kLarge>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess)
            return ARB_ERR_CUDA;
        attr_set[ctx->device & 63] = true;
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    // A call that cannot be anything but small -- the block table has room for at most kSmallCallPages
    // pages per SM -- is launched with one CTA per SM outright: no CTA comes up only to leave.
    const long long page_bound = (long long)a.batch * a.max_pages * a.Hkv;
    const bool small = page_bound <= (long long)ctx->num_sms * kSmallCallPages;
    const int grid = small ? ctx->num_sms : ctx->num_sms * kCtasPerSm;
    cfg.gridDim = dim3(grid);
    const int cons_warps = small ? 4 : kLarge;
    cfg.blockDim = dim3(cons_warps * 32 + 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    const cudaError_t err = cons_warps == 4 ? cudaLaunchKernelEx(&cfg, decode_mma_kernel<G, E4M3, 4>, a, km, vm)
                                            : cudaLaunchKernelEx(&cfg, decode_mma_kernel<G, E4M3, kLarge>, a, km, vm);
    if (err != cudaSuccess) return ARB_ERR_CUDA;
    ctx->launches++;
    // the combine kernel, always a programmatic dependent of the decode kernel
    ca.decode_grid = grid;
    const long long items = (long long)a.batch * a.Hkv;
    cudaLaunchConfig_t ccfg = {};
    ccfg.gridDim = dim3((unsigned)(items < ctx->num_sms ? items : ctx->num_sms));
    ccfg.blockDim = dim3(kCombineThreads);
    ccfg.dynamicSmemBytes = sizeof(int) * (2 * (size_t)a.batch + 2) + sizeof(float2) * (size_t)grid * G;
    ccfg.stream = stream;
    ccfg.attrs = attr;
    ccfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&ccfg, decode_combine_kernel<G>, ca) != cudaSuccess) return ARB_ERR_CUDA;
    ctx->launches++;
    return ARB_OK;
}

}  // namespace

bool decode_mma_supported(const arb_attn_params &p) {
    const int g = p.num_q_heads / p.num_kv_heads;
    return p.dtype == ARB_BF16 && p.head_dim == kD && g >= kDecodeMmaMinGroup && g <= 8 && tma_available();
}

namespace {

// both caches: e4m3 selects the E4M3 form, whose keys are k_scale * code and values v_scale * code
arb_status launch_decode_tc(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages, const void *v_pages,
                            bool e4m3, float k_scale, float v_scale, const int32_t *block_table, const int32_t *seq_lens,
                            const int32_t *q_lens, void *out, cudaStream_t stream) {
    alignas(64) CUtensorMap km, vm;
    // bf16 pools: a page is fetched as one box of the 3-D view (both 64-element halves of its 16 rows), which
    // halves the number of TMA copies; the 2-D view with two boxes per page stays as the fallback should a
    // driver refuse the 3-D encoding, whose third stride is smaller than its second.
    bool whole_rows = false;
    if (!e4m3)
        whole_rows = pool_map(ctx, &km, k_pages, p.num_pages, p.num_kv_heads, PoolView::kBf16WholeRows) &&
                     pool_map(ctx, &vm, v_pages, p.num_pages, p.num_kv_heads, PoolView::kBf16WholeRows);
    const PoolView view = e4m3 ? PoolView::kE4m3 : PoolView::kBf16HalfRows;
    if (!whole_rows && (!pool_map(ctx, &km, k_pages, p.num_pages, p.num_kv_heads, view) ||
                        !pool_map(ctx, &vm, v_pages, p.num_pages, p.num_kv_heads, view)))
        return ARB_ERR_CUDA;
    const int g = p.num_q_heads / p.num_kv_heads;
    const int gp = (g + 3) / 4 * 4;
    const size_t slots = (size_t)p.batch * p.num_kv_heads + (size_t)ctx->num_sms * kCtasPerSm;
    // Workspace rotation.  The workspace is cut into kRotSets + 1 regions of one fixed size, whatever the
    // shape of the call: region 0 belongs to the decode kernels that take no generation number, regions
    // 1 .. kRotSets are the rotation sets.  Consecutive calls take consecutive generation numbers and use set
    // (generation mod kRotSets): partials and (max, sum) records of their own.  A call may write its set
    // without waiting for the previous call once the set's previous user (generation - kRotSets) has published
    // its completion.  Because a set always lies at the same place, that holds for any mix of shapes in a
    // series.  A call whose partials do not fit in one region takes the whole workspace and waits; it may lie
    // over every set, so the calls of the next kRotSets generations wait as well (until the window
    // [generation - kRotSets, generation - 1] no longer reaches back to it, a completion inside the window says
    // nothing about the large call).
    const size_t part_o_floats = (slots * g * p.head_dim + 63) & ~size_t(63);
    const size_t set_bytes = ((part_o_floats + slots * gp * 2) * sizeof(float) + 255) & ~size_t(255);
    if (set_bytes > ctx->workspace_bytes) return ARB_ERR_WORKSPACE;
    const size_t region = rot_region_bytes(ctx);
    const uint32_t gen = ctx->decode_gen++;
    const bool rotates = set_bytes <= region;
    const int sets = rotates ? kRotSets : 1;
    const int set = rotates ? (int)(gen % (uint32_t)kRotSets) : 0;
    const size_t set_offset = rotates ? (size_t)(1 + set) * region : 0;
    const bool force_wait = !rotates || (int32_t)(ctx->rot_wait_through - gen) >= 0;
    if (!rotates) ctx->rot_wait_through = gen + (uint32_t)kRotSets;
    Args a;
    a.q = static_cast<const char *>(q);
    a.block_table = block_table;
    a.seq_lens = seq_lens;
    a.q_lens = q_lens;
    a.out = static_cast<char *>(out);
    a.part_o = reinterpret_cast<float *>(ctx->workspace + set_offset);
    a.part_ml = a.part_o + part_o_floats;
    a.done_gen = reinterpret_cast<unsigned *>(ctx->rot + (size_t)kRotSets * kRotCounters + kRotSets);
    a.gen = gen;
    a.sets = sets;
    a.force_wait = force_wait ? 1 : 0;
    a.status = ctx->status;
    a.slots = (int)slots;
    a.rows = p.total_q;
    a.batch = p.batch;
    a.Hq = p.num_q_heads;
    a.Hkv = p.num_kv_heads;
    a.num_pages = p.num_pages;
    a.max_pages = p.max_pages_per_seq;
    a.whole_rows = whole_rows ? 1 : 0;
    // A small call streams at the pace of its CTAs' pipelines, not of the memory system, and every
    // CTA spends a fixed time before its first and after its last tile.  A call that declares itself
    // part of a back-to-back series (ARB_ATTN_OVERLAP_PREVIOUS) therefore takes only every second
    // SM's worth of CTAs: each lives longer, four calls are in flight instead of two, and the
    // series as a whole moves more bytes per second; a lone call gets one CTA on every SM, which
    // is what finishes it soonest.
    a.small_ctas = (p.flags & ARB_ATTN_OVERLAP_PREVIOUS) ? (ctx->num_sms + 1) / 2 : ctx->num_sms;
    const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.head_dim);
    a.scale_log2 = scale * k_scale * 1.4426950408889634f;
    a.v_scale = v_scale;
    const bool overlap = (p.flags & ARB_ATTN_OVERLAP_PREVIOUS) != 0;
    CombineArgs ca;
    ca.seq_lens = seq_lens;
    ca.q_lens = q_lens;
    ca.out = a.out;
    ca.part_o = a.part_o;
    ca.part_ml = a.part_ml;
    ca.batch = a.batch;
    ca.Hq = a.Hq;
    ca.Hkv = a.Hkv;
    ca.max_pages = a.max_pages;
    ca.small_ctas = a.small_ctas;
    ca.decode_grid = 0;  // set by launch_one
    ca.gen = gen;
    ca.done_gen = a.done_gen;
    ca.exit_count = ctx->rot + (size_t)kRotSets * kRotCounters + set;
    switch (e4m3 ? g + 8 : g) {
        case 1: return launch_one<1, false>(ctx, a, ca, km, vm, overlap, stream);
        case 2: return launch_one<2, false>(ctx, a, ca, km, vm, overlap, stream);
        case 3: return launch_one<3, false>(ctx, a, ca, km, vm, overlap, stream);
        case 4: return launch_one<4, false>(ctx, a, ca, km, vm, overlap, stream);
        case 5: return launch_one<5, false>(ctx, a, ca, km, vm, overlap, stream);
        case 6: return launch_one<6, false>(ctx, a, ca, km, vm, overlap, stream);
        case 7: return launch_one<7, false>(ctx, a, ca, km, vm, overlap, stream);
        case 8: return launch_one<8, false>(ctx, a, ca, km, vm, overlap, stream);
        case 9: return launch_one<1, true>(ctx, a, ca, km, vm, overlap, stream);
        case 10: return launch_one<2, true>(ctx, a, ca, km, vm, overlap, stream);
        case 11: return launch_one<3, true>(ctx, a, ca, km, vm, overlap, stream);
        case 12: return launch_one<4, true>(ctx, a, ca, km, vm, overlap, stream);
        case 13: return launch_one<5, true>(ctx, a, ca, km, vm, overlap, stream);
        case 14: return launch_one<6, true>(ctx, a, ca, km, vm, overlap, stream);
        case 15: return launch_one<7, true>(ctx, a, ca, km, vm, overlap, stream);
        case 16: return launch_one<8, true>(ctx, a, ca, km, vm, overlap, stream);
        default: return ARB_ERR_UNSUPPORTED;
    }
}

}  // namespace

arb_status launch_decode_mma(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages,
                             const void *v_pages, const int32_t *block_table, const int32_t *seq_lens,
                             const int32_t *q_lens, void *out, cudaStream_t stream) {
    return launch_decode_tc(ctx, p, q, k_pages, v_pages, false, 1.0f, 1.0f, block_table, seq_lens, q_lens, out, stream);
}

arb_status launch_decode_e4m3(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages,
                              const void *v_pages, float k_scale, float v_scale, const int32_t *block_table,
                              const int32_t *seq_lens, const int32_t *q_lens, void *out, cudaStream_t stream) {
    const int g = p.num_q_heads / p.num_kv_heads;
    if (g > 8 || !tma_available()) return ARB_ERR_UNSUPPORTED;
    return launch_decode_tc(ctx, p, q, k_pages, v_pages, true, k_scale, v_scale, block_table, seq_lens, q_lens, out, stream);
}

}  // namespace arb

// Split-KV decode attention (q_len = 1) over paged KV, one persistent launch.
//
// Work decomposition.  The (sequence, kv head, page) triples of every decoding sequence form one
// flat list, ordered sequence-major.  It is cut into gridDim.x equal ranges, one per CTA, so every
// CTA streams the same number of pages whatever the length mix is.  Where a range crosses a
// (sequence, kv head) boundary it splits into segments; a (sequence, kv head) whose pages span
// several CTAs is finished by whichever of them arrives last (arrival counter + fence, no waiting).
// The device derives all of this from seq_lens / q_lens in the kernel prologue, so the host never
// reads a length.
//
// Inside a CTA one producer warp walks its pages and issues one bulk (TMA) copy per (page, head)
// tile of K and of V -- 16 rows x head_dim, contiguous in the head-major page layout -- into a
// shared-memory ring guarded by full/empty mbarriers; up to sixteen lanes issue side by side, one
// ring stage each.  Pages are taken in groups of kGroup; group j of a segment belongs to consumer
// warp j mod 4, and its tiles enter the ring as K..K V..V.  Each consumer warp runs its own online
// softmax: q.K for the group's K tiles into a per-warp score buffer, running max / exp2 / running
// sum over those scores, then P.V over the group's V tiles into per-lane fp32 accumulators.  The
// warps never meet until the segment ends, where their (max, sum, accumulator) triples are merged.
//
// Arithmetic.  bf16 q.K uses the mixed-precision FMA of sm_100 (bf16 x bf16 + fp32 -> fp32, the
// product is exact), so neither operand is unpacked; eight lanes share a K row, each owning 16 of
// its 128 dims, and the lanes' partial dot products meet in a transposing shuffle reduction.  P.V
// keeps P in fp32: V is unpacked with one shift or mask per element, shared by the whole group.
//
// Split combine.  Partials of one (sequence, kv head) lie in consecutive workspace slots.  The CTA
// that arrives last notes the job and, once its own pages are done and the ring is idle, pulls the
// partials into shared memory with bulk copies and merges them there.
#include <mutex>

#include "arb_common.cuh"

namespace arb {

namespace {

constexpr int kConsWarps = 4;
constexpr int kConsThreads = kConsWarps * 32;
constexpr int kThreads = kConsThreads + 32;  // + producer warp
constexpr int kGroup = 2;                    // pages per consumer work group
constexpr int kGroupTokens = kGroup * kPage;
constexpr int kMinChunk = 4;                 // fewest pages worth giving a CTA
constexpr int kMaxCtasPerSm = 2;

struct DecodeArgs {
    const char *q;
    const char *k_pages;
    const char *v_pages;
    const int32_t *block_table;
    const int32_t *seq_lens;
    const int32_t *q_lens;
    char *out;
    float *part_o;    // [slots][G][D]    un-normalised partial outputs
    float *part_ml;   // [slots][GP][2]   running max (log2 domain) and sum
    int *counters;    // [batch * Hkv]
    uint32_t *status;
    int batch, Hq, Hkv, num_pages, max_pages;
    float scale_log2;  // softmax scale * log2(e)
};

template <typename T, int D, int G>
struct Cfg {
    static constexpr bool kBf16 = sizeof(T) == 2;
    static constexpr int EPL = Elt<T>::kPerVec;          // elements in one 16-byte vector
    static constexpr int ROW_BYTES = D * (int)sizeof(T);
    // P.V mapping: one 16-byte vector per lane
    static constexpr int LPR = ROW_BYTES / 16;           // lanes per V row: 8, 16 or 32
    static constexpr int RPP = 32 / LPR;                 // rows a warp reads per pass
    static constexpr int NPASS = kPage / RPP;
    // q.K mapping: bf16 rows are shared by 8 lanes (CPL vectors each); fp32 rows as for P.V
    static constexpr int QLPR = kBf16 ? 8 : LPR;
    static constexpr int CPL = kBf16 ? ROW_BYTES / 128 : 1;  // 16-byte vectors per lane and row
    static constexpr int QRPP = 32 / QLPR;
    static constexpr int QNPASS = kPage / QRPP;
    static constexpr int PB = QNPASS < 8 ? QNPASS : 8;   // passes per reduction batch
    static constexpr int NB = QNPASS / PB;
    static constexpr int NV = PB * G;                    // partial dot products per lane and batch
    static constexpr int NVP = (NV + QLPR - 1) / QLPR * QLPR;
    static constexpr int GP = (G + 3) / 4 * 4;           // heads padded to whole float4s
    static constexpr int TILE_BYTES = kPage * ROW_BYTES;
    // Ring stage = tile counter mod STAGES and owner warp = (tile counter / tiles per group) mod 4.
    // STAGES is a multiple of 4 groups, so a stage is only ever read by one warp: that warp has
    // consumed fill k-1 before it waits for fill k, which is what a parity wait needs (a waiter two
    // phases behind would pass at once).
    static constexpr int STAGES = 16;
    static constexpr int BATCH = 16;                         // producer lanes issuing side by side
    static constexpr int RING_BYTES = STAGES * TILE_BYTES;
    static constexpr int CTAS = RING_BYTES > 65536 ? 1 : 2;  // resident CTAs per SM aimed at
    static constexpr int SCORE_BYTES = kConsWarps * kGroupTokens * GP * 4;   // per-warp score buffers
    static constexpr int REC = G * D + 2 * GP;                               // floats of one warp record
    static constexpr int OSM_BYTES = kConsWarps * REC * 4;
    static_assert(LPR == 8 || LPR == 16 || LPR == 32, "row must be 128, 256 or 512 bytes");
    static_assert(STAGES % (kConsWarps * 2 * kGroup) == 0, "a ring stage must always belong to the same warp");
};

constexpr int kMaxStages = 16;

struct SmemTail {  // small fixed part after ring + buffers
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t cbar[2];  // split-combine staging, one per buffer
    float lsum[kMaxGroup];
    int abort;
    int is_last;
};

template <typename T, int D, int G>
size_t smem_bytes(int batch) {
    using C = Cfg<T, D, G>;
    return 128 + C::RING_BYTES + C::SCORE_BYTES + C::OSM_BYTES + sizeof(SmemTail) +
           sizeof(int) * (3 * (size_t)batch + 2);
}

struct Segment {
    int b, kvh, pg0, pg1, L, bk, nparts, c_first;
};

// Next segment of the flat range [cur, r1); advances cur.  pref[b] = kv heads * pages of all
// decoding sequences before b; slen[b] = seq_lens[b].
__device__ __forceinline__ bool next_segment(int &cur, int r1, const int *pref, const int *slen, int B, int Hkv,
                                             int chunk, Segment &s) {
    if (cur >= r1) return false;
    int lo = 0, hi = B;  // largest b with pref[b] <= cur
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (pref[mid] <= cur) lo = mid; else hi = mid;
    }
    const int b = lo;
    const int pages = (pref[b + 1] - pref[b]) / Hkv;
    const int r = cur - pref[b];
    const int kvh = r / pages;
    const int pg0 = r - kvh * pages;
    const int s0 = pref[b] + kvh * pages;  // flat range of this (sequence, kv head)
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

// acc += q.lo * k.lo + q.hi * k.hi for two packed bf16 pairs; products are exact, sums round in fp32
__device__ __forceinline__ float fma_bf16x2(uint32_t q, uint32_t k, float acc) {
    asm("{\n\t.reg .b16 ql, qh, kl, kh;\n\t"
        "mov.b32 {ql, qh}, %1;\n\t"
        "mov.b32 {kl, kh}, %2;\n\t"
        "fma.rn.f32.bf16 %0, ql, kl, %0;\n\t"
        "fma.rn.f32.bf16 %0, qh, kh, %0;\n\t}"
        : "+f"(acc)
        : "r"(q), "r"(k));
    return acc;
}

__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }


template <typename T, int D, int G>
__global__ void __launch_bounds__(kThreads, Cfg<T, D, G>::CTAS) decode_kernel(const DecodeArgs a) {
    using C = Cfg<T, D, G>;
    constexpr int EPL = C::EPL, LPR = C::LPR, RPP = C::RPP, GP = C::GP;
    constexpr int QLPR = C::QLPR, QRPP = C::QRPP, CPL = C::CPL, STAGES = C::STAGES;
    constexpr int QW = C::kBf16 ? CPL * 4 : EPL;  // 32-bit q registers per head and lane
    constexpr int REC = C::REC;

    extern __shared__ char smem_raw[];
    char *base = reinterpret_cast<char *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    char *ring = base;
    float *score_all = reinterpret_cast<float *>(base + C::RING_BYTES);
    float *osm = reinterpret_cast<float *>(base + C::RING_BYTES + C::SCORE_BYTES);
    SmemTail *tail = reinterpret_cast<SmemTail *>(base + C::RING_BYTES + C::SCORE_BYTES + C::OSM_BYTES);
    int *pref = reinterpret_cast<int *>(tail + 1);  // [B + 1]
    int *row0 = pref + a.batch + 1;                 // [B + 1]
    int *slen = row0 + a.batch + 1;                 // [B]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.batch, Hkv = a.Hkv;

    // Until wait_for_predecessor() this kernel only reads its inputs (and ORs error bits); every
    // write to out, the workspace or the arrival counters comes after it.  A successor launched as
    // a programmatic dependent does the same, so it can stream its KV under this kernel's tail and
    // still cannot touch the shared workspace before this kernel is complete.
    let_successor_start();

    // ---- prologue: lengths -> page counts and q row offsets, scanned by warp 0 -----------------
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&tail->full[s], 1);
            mbar_init(&tail->empty[s], 1);
        }
        mbar_init(&tail->cbar[0], 1);
        mbar_init(&tail->cbar[1], 1);
        tail->abort = 0;
        tail->is_last = 0;
        mbar_fence_init();
        pref[0] = 0;
        row0[0] = 0;
    }
    for (int b = tid; b < B; b += kThreads) {
        const int n = a.q_lens[b], L = a.seq_lens[b];
        int pages = 0;
        if (n == 1) {
            if (L >= 1 && L <= a.max_pages * kPage) {
                pages = (L + kPage - 1) / kPage;
            } else if (blockIdx.x == 0) {  // no defined result: flag it and zero the row
                wait_for_predecessor();
                atomicOr(a.status, (uint32_t)ARB_DEV_BAD_SEQ_LEN);
                int row = 0;
                for (int i = 0; i < b; ++i) row += max(a.q_lens[i], 0);
                T *o = reinterpret_cast<T *>(a.out) + (size_t)row * a.Hq * D;
                for (int i = 0; i < a.Hq * D; ++i) o[i] = Elt<T>::from_float(0.f);
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

    const int total = pref[B];
    int chunk = (total + (int)gridDim.x - 1) / (int)gridDim.x;
    if (chunk < kMinChunk) chunk = kMinChunk;
    const long long r0l = (long long)blockIdx.x * chunk;
    if (r0l >= total) return;  // whole CTA leaves together; no barrier is pending
    const int r0 = (int)r0l;
    const int r1 = min(total, r0 + chunk);
    volatile int *abort = &tail->abort;

    if (warp == kConsWarps) {
        // ================================ producer warp ==========================================
        // Tiles enter the ring group by group: K tiles of a group, then its V tiles.  Lanes
        // 0..BATCH-1 each own one ring stage at a time: wait until it is free, then issue the copy.
        // A batch never exceeds the ring, so a lane is at most one phase behind its barrier.
        uint32_t c = 0;
        int cur = r0;
        Segment s;
        while (next_segment(cur, r1, pref, slen, B, Hkv, chunk, s)) {
            for (int sp0 = s.pg0; sp0 < s.pg1; sp0 += 32) {
                const int np = min(32, s.pg1 - sp0);
                int pid = 0;
                if (lane < np) {
                    pid = a.block_table[(size_t)s.b * a.max_pages + sp0 + lane];
                    if ((unsigned)pid >= (unsigned)a.num_pages) {
                        atomicOr(a.status, (uint32_t)ARB_DEV_BAD_PAGE);
                        pid = 0;
                    }
                }
                const int full_tiles = (np / kGroup) * 2 * kGroup;  // tiles of the complete groups
                const int rem = np % kGroup;
                const int ntiles = 2 * np;
#pragma unroll 1
                for (int i0 = 0; i0 < ntiles; i0 += C::BATCH) {
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
                    if (lane < C::BATCH && i < ntiles) {
                        const uint32_t cc = c + i, st = cc % STAGES, par = (cc / STAGES) & 1u;
                        const char *pool = is_v ? a.v_pages : a.k_pages;
                        if (mbar_wait(&tail->empty[st], par ^ 1u, abort, a.status)) {
                            mbar_arrive_expect_tx(&tail->full[st], C::TILE_BYTES);
                            bulk_load(ring + st * C::TILE_BYTES, pool + ((size_t)pg * Hkv + s.kvh) * C::TILE_BYTES,
                                      C::TILE_BYTES, &tail->full[st]);
                        }
                    }
                    __syncwarp();
                }
                c += ntiles;
            }
        }
        // After a timeout the consumers may have left copies unconsumed: wait (bounded) for the
        // last ring's worth so that no copy is in flight into this CTA's memory when it exits.
        if (lane == 0 && *abort) {
            const uint32_t n = c < (uint32_t)STAGES ? c : (uint32_t)STAGES;
            for (uint32_t i = 0; i < n; ++i) {
                const uint32_t cc = c - 1 - i;
                const long long t0 = clock64();
                while (!mbar_try_wait(&tail->full[cc % STAGES], (cc / STAGES) & 1u) &&
                       clock64() - t0 < (1ll << 24)) {
                }
            }
        }
        return;
    }

    // ==================================== consumer warps ==========================================
    const int lg = lane % LPR, rg = lane / LPR;      // P.V: vector column within a row, row of a pass
    const int qlg = lane % QLPR, qrg = lane / QLPR;  // q.K: the same for its own row sharing
    float *sc = score_all + warp * kGroupTokens * GP;  // this warp's scores / probabilities
    uint32_t seg_base = 0;                             // ring counter of the segment's first tile
    int cur = r0;
    Segment s;
    // split-combine jobs this CTA has to finish (only the first and last segment of a range can be
    // part of a longer (sequence, kv head), so two slots are enough)
    int pend_n = 0;
    int pend_slot0[2], pend_parts[2];
    size_t pend_out[2];

    while (next_segment(cur, r1, pref, slen, B, Hkv, chunk, s)) {
        const int qrow = row0[s.b];
        // q of this kv head's group: packed bf16 pairs, or fp32 pre-multiplied by the scale
        uint32_t qp[G][QW];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            const char *qh = a.q + ((size_t)qrow * a.Hq + s.kvh * G + h) * D * sizeof(T);
            if constexpr (C::kBf16) {
#pragma unroll
                for (int cp = 0; cp < CPL; ++cp) {
                    const uint4 v = __ldg(reinterpret_cast<const uint4 *>(qh + (qlg + 8 * cp) * 16));
                    qp[h][4 * cp + 0] = v.x; qp[h][4 * cp + 1] = v.y;
                    qp[h][4 * cp + 2] = v.z; qp[h][4 * cp + 3] = v.w;
                }
            } else {
                const uint4 v = __ldg(reinterpret_cast<const uint4 *>(qh + qlg * 16));
                qp[h][0] = __float_as_uint(__uint_as_float(v.x) * a.scale_log2);
                qp[h][1] = __float_as_uint(__uint_as_float(v.y) * a.scale_log2);
                qp[h][2] = __float_as_uint(__uint_as_float(v.z) * a.scale_log2);
                qp[h][3] = __float_as_uint(__uint_as_float(v.w) * a.scale_log2);
            }
        }
        const float scl = C::kBf16 ? a.scale_log2 : 1.0f;
        // m_run is the same in every lane of the warp; l_run is this lane's share of the sum
        float m_run[G], l_run[G], o[G][EPL];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            m_run[h] = -INFINITY;
            l_run[h] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) o[h][e] = 0.f;
        }

        const int seg_pages = s.pg1 - s.pg0;
        const int ngroups = (seg_pages + kGroup - 1) / kGroup;
        for (int gi = warp; gi < ngroups; gi += kConsWarps) {
            const int p0 = s.pg0 + gi * kGroup;               // first page of the group
            const int npg = min(kGroup, s.pg1 - p0);
            const int ntok = min(s.L - p0 * kPage, npg * kPage);  // valid tokens of the group
            const uint32_t gbase = seg_base + (uint32_t)gi * 2 * kGroup;

            // ---- q.K: scores of the group's K tiles ----------------------------------------------
            for (int t = 0; t < npg; ++t) {
                const uint32_t cc = gbase + t, st = cc % STAGES, par = (cc / STAGES) & 1u;
                mbar_wait(&tail->full[st], par, abort, a.status);
                const char *tile = ring + st * C::TILE_BYTES;
#pragma unroll
                for (int nb = 0; nb < C::NB; ++nb) {
                    float acc[C::NVP];
#pragma unroll
                    for (int i = 0; i < C::NVP; ++i) acc[i] = 0.f;
#pragma unroll
                    for (int ps = 0; ps < C::PB; ++ps) {
                        const int r = (nb * C::PB + ps) * QRPP + qrg;
                        if constexpr (C::kBf16) {
#pragma unroll
                            for (int cp = 0; cp < CPL; ++cp) {
                                const uint4 kv = *reinterpret_cast<const uint4 *>(tile + r * C::ROW_BYTES +
                                                                                  (qlg + 8 * cp) * 16);
#pragma unroll
                                for (int h = 0; h < G; ++h) {
                                    float x = acc[ps * G + h];
                                    x = fma_bf16x2(qp[h][4 * cp + 0], kv.x, x);
                                    x = fma_bf16x2(qp[h][4 * cp + 1], kv.y, x);
                                    x = fma_bf16x2(qp[h][4 * cp + 2], kv.z, x);
                                    x = fma_bf16x2(qp[h][4 * cp + 3], kv.w, x);
                                    acc[ps * G + h] = x;
                                }
                            }
                        } else {
                            const uint4 kv = *reinterpret_cast<const uint4 *>(tile + r * C::ROW_BYTES + qlg * 16);
                            float kf[EPL];
                            Elt<T>::unpack(kv, kf);
#pragma unroll
                            for (int h = 0; h < G; ++h)
#pragma unroll
                                for (int e = 0; e < EPL; ++e)
                                    acc[ps * G + h] = fmaf(__uint_as_float(qp[h][e]), kf[e], acc[ps * G + h]);
                        }
                    }
                    transpose_reduce<C::NVP, QLPR>(acc, qlg);
#pragma unroll
                    for (int j = 0; j < C::NVP / QLPR; ++j) {
                        const int idx = j + (C::NVP / QLPR) * qlg;
                        if (idx < C::NV) {
                            const int ps = idx / G, h = idx - ps * G;
                            const int token = t * kPage + (nb * C::PB + ps) * QRPP + qrg;
                            sc[token * GP + h] = acc[j] * scl;
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&tail->empty[st]);
            }

            // ---- online softmax over the group's scores: one token per lane ---------------------
            static_assert(kGroupTokens == 32, "one token per lane");
            float sv[GP];
            const bool tok_ok = lane < ntok;
#pragma unroll
            for (int h4 = 0; h4 < GP; h4 += 4) {
                const float4 x = *reinterpret_cast<const float4 *>(sc + lane * GP + h4);
                sv[h4] = x.x; sv[h4 + 1] = x.y; sv[h4 + 2] = x.z; sv[h4 + 3] = x.w;
            }
            float mx[G];
#pragma unroll
            for (int h = 0; h < G; ++h) mx[h] = tok_ok ? sv[h] : -INFINITY;
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1)
#pragma unroll
                for (int h = 0; h < G; ++h) mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], off));
#pragma unroll
            for (int h = 0; h < G; ++h) {
                const float m = fmaxf(m_run[h], mx[h]);      // finite: the group has a valid token
                const float f = fast_exp2(m_run[h] - m);     // 0 for the first group
                m_run[h] = m;
                const float p = tok_ok ? fast_exp2(sv[h] - m) : 0.f;
                sv[h] = p;
                l_run[h] = fmaf(l_run[h], f, p);
#pragma unroll
                for (int e = 0; e < EPL; ++e) o[h][e] *= f;
            }
#pragma unroll
            for (int h4 = 0; h4 < GP; h4 += 4)
                *reinterpret_cast<float4 *>(sc + lane * GP + h4) = make_float4(sv[h4], sv[h4 + 1], sv[h4 + 2], sv[h4 + 3]);
            __syncwarp();

            // ---- P.V over the group's V tiles -----------------------------------------------------
            for (int t = 0; t < npg; ++t) {
                const uint32_t cc = gbase + npg + t, st = cc % STAGES, par = (cc / STAGES) & 1u;
                mbar_wait(&tail->full[st], par, abort, a.status);
                const char *tile = ring + st * C::TILE_BYTES;
                const float *pt = sc + t * kPage * GP;
                if ((t + 1) * kPage <= ntok) {  // every slot of the tile is a real token
#pragma unroll
                    for (int ps = 0; ps < C::NPASS; ++ps) {
                        const int r = ps * RPP + rg;
                        const uint4 vv = *reinterpret_cast<const uint4 *>(tile + r * C::ROW_BYTES + lg * 16);
                        float vf[EPL];
                        Elt<T>::unpack(vv, vf);
                        float pf[GP];
#pragma unroll
                        for (int h4 = 0; h4 < GP; h4 += 4) {
                            const float4 pv = *reinterpret_cast<const float4 *>(pt + r * GP + h4);
                            pf[h4] = pv.x; pf[h4 + 1] = pv.y; pf[h4 + 2] = pv.z; pf[h4 + 3] = pv.w;
                        }
#pragma unroll
                        for (int h = 0; h < G; ++h)
#pragma unroll
                            for (int e = 0; e < EPL; ++e) o[h][e] = fmaf(pf[h], vf[e], o[h][e]);
                    }
                } else {  // ragged last page: slots past the sequence end are never touched
#pragma unroll 1
                    for (int ps = 0; ps < C::NPASS; ++ps) {
                        const int r = ps * RPP + rg;
                        if (t * kPage + r < ntok) {
                            const uint4 vv = *reinterpret_cast<const uint4 *>(tile + r * C::ROW_BYTES + lg * 16);
                            float vf[EPL];
                            Elt<T>::unpack(vv, vf);
#pragma unroll
                            for (int h = 0; h < G; ++h) {
                                const float p = pt[r * GP + h];
#pragma unroll
                                for (int e = 0; e < EPL; ++e) o[h][e] = fmaf(p, vf[e], o[h][e]);
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&tail->empty[st]);
            }
        }
        seg_base += 2u * (uint32_t)seg_pages;

        // ---- segment end: every warp leaves (max, sum, accumulator); all threads merge them ----------
        wait_for_predecessor();  // first write of this CTA comes below; later calls return at once
#pragma unroll
        for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int e = 0; e < EPL; ++e) o[h][e] += __shfl_xor_sync(0xffffffffu, o[h][e], off);
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1)
#pragma unroll
            for (int h = 0; h < G; ++h) l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], off);
        float *rec = osm + warp * REC;  // [m[GP] | l[GP] | o[G][D]]
        if (rg == 0) {
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int e = 0; e < EPL; ++e) rec[2 * GP + h * D + lg * EPL + e] = o[h][e];
        }
        if (lane == 0) {
#pragma unroll
            for (int h = 0; h < G; ++h) { rec[h] = m_run[h]; rec[GP + h] = l_run[h]; }
        }
        named_barrier(1, kConsThreads);

        const size_t out_base = ((size_t)qrow * a.Hq + s.kvh * G) * D;
        const size_t slot = (size_t)s.bk + blockIdx.x;
        for (int idx = tid; idx < G * D; idx += kConsThreads) {
            const int h = idx / D;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kConsWarps; ++w) M = fmaxf(M, osm[w * REC + h]);
            float l = 0.f, acc = 0.f;
#pragma unroll
            for (int w = 0; w < kConsWarps; ++w) {
                const float f = fast_exp2(osm[w * REC + h] - M);  // 0 for a warp that had no group
                l = fmaf(f, osm[w * REC + GP + h], l);
                acc = fmaf(f, osm[w * REC + 2 * GP + idx], acc);
            }
            if (s.nparts == 1) {
                reinterpret_cast<T *>(a.out)[out_base + idx] = Elt<T>::from_float(acc / l);
            } else {
                a.part_o[slot * G * D + idx] = acc;
                if (idx - h * D == 0) {
                    a.part_ml[(slot * GP + h) * 2 + 0] = M;
                    a.part_ml[(slot * GP + h) * 2 + 1] = l;
                }
            }
        }
        if (s.nparts > 1) {
            __threadfence();
            fence_proxy_async_all();  // the partials are read back through bulk copies
            named_barrier(1, kConsThreads);
            if (tid == 0) {
                const int old = atomicAdd(&a.counters[s.bk], 1);
                const int last = (old == s.nparts - 1);
                if (last) a.counters[s.bk] = 0;  // everyone has arrived: ready for the next call
                tail->is_last = last;
            }
            named_barrier(1, kConsThreads);
            if (tail->is_last && pend_n < 2) {
                pend_slot0[pend_n] = s.bk + s.c_first;
                pend_parts[pend_n] = s.nparts;
                pend_out[pend_n] = out_base;
                ++pend_n;
            }
        }
        named_barrier(1, kConsThreads);  // records and is_last are free for the next segment
    }

    // ---- split combine of the (sequence, kv head)s this CTA was the last to reach -----------------
    // All tiles have been consumed and the producer issues nothing more, so the ring is free:
    // [ max/sum records of all parts | buffer A | buffer B ]; partial outputs stream through A and B
    // while the previous piece is being added up.
    uint32_t cph[2] = {0u, 0u};
    for (int j = 0; j < pend_n; ++j) {
        const int nparts = pend_parts[j];
        const size_t slot0 = (size_t)pend_slot0[j];
        __threadfence();
        const uint32_t ml_bytes = (uint32_t)nparts * GP * 8u;
        const uint32_t ml_area = (ml_bytes + 127u) & ~127u;
        constexpr int PART_BYTES = G * D * 4;
        float *ml = reinterpret_cast<float *>(ring);
        const int per_piece = ((C::RING_BYTES - (int)ml_area) / 2) / PART_BYTES;
        if (per_piece < 1) {
            // more parts than the ring can describe (far more CTAs than this part has SMs for):
            // merge straight from global memory
            for (int idx = tid; idx < G * D; idx += kConsThreads) {
                const int h = idx / D;
                float m = -INFINITY;
                for (int p = 0; p < nparts; ++p) m = fmaxf(m, __ldcg(&a.part_ml[((slot0 + p) * GP + h) * 2]));
                float l = 0.f, x = 0.f;
                for (int p = 0; p < nparts; ++p) {
                    const float w = fast_exp2(__ldcg(&a.part_ml[((slot0 + p) * GP + h) * 2]) - m);
                    l = fmaf(w, __ldcg(&a.part_ml[((slot0 + p) * GP + h) * 2 + 1]), l);
                    x = fmaf(w, __ldcg(&a.part_o[(slot0 + p) * G * D + idx]), x);
                }
                reinterpret_cast<T *>(a.out)[pend_out[j] + idx] = Elt<T>::from_float(x / l);
            }
            continue;
        }
        float *buf[2] = {reinterpret_cast<float *>(ring + ml_area),
                         reinterpret_cast<float *>(ring + ml_area + per_piece * PART_BYTES)};
        const int npieces = (nparts + per_piece - 1) / per_piece;
        auto issue_piece = [&](int i, uint32_t extra) {  // thread 0 only
            const int p0 = i * per_piece, np = min(per_piece, nparts - p0);
            const uint32_t bytes = (uint32_t)np * PART_BYTES;
            mbar_arrive_expect_tx(&tail->cbar[i & 1], bytes + extra);
            bulk_load(buf[i & 1], a.part_o + (slot0 + p0) * G * D, bytes, &tail->cbar[i & 1]);
        };
        if (tid == 0) {
            fence_proxy_async_all();
            issue_piece(0, ml_bytes);
            bulk_load(ml, a.part_ml + slot0 * GP * 2, ml_bytes, &tail->cbar[0]);
            if (npieces > 1) issue_piece(1, 0u);
        }
        __syncwarp();  // warp 0 reconverges before the wait and the weight phase
        mbar_wait(&tail->cbar[0], cph[0], abort, a.status);
        cph[0] ^= 1u;
        // weights: warp w owns heads w, w + 4; the max slot of every record is overwritten by its weight
        for (int h = warp; h < G; h += kConsWarps) {
            float m = -INFINITY;
            for (int p = lane; p < nparts; p += 32) m = fmaxf(m, ml[(p * GP + h) * 2]);
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
            float l = 0.f;
            for (int p = lane; p < nparts; p += 32) {
                const float w = fast_exp2(ml[(p * GP + h) * 2] - m);
                ml[(p * GP + h) * 2] = w;
                l = fmaf(w, ml[(p * GP + h) * 2 + 1], l);
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
            if (lane == 0) tail->lsum[h] = l;
        }
        named_barrier(1, kConsThreads);
        constexpr int NK = (G * D + kConsThreads - 1) / kConsThreads;
        float acc[NK];
        int hk[NK];
#pragma unroll
        for (int k = 0; k < NK; ++k) {
            const int idx = tid + k * kConsThreads;
            hk[k] = idx < G * D ? idx / D : 0;
            acc[k] = 0.f;
        }
        for (int i = 0; i < npieces; ++i) {
            const int p0 = i * per_piece, np = min(per_piece, nparts - p0);
            if (i > 0) {
                mbar_wait(&tail->cbar[i & 1], cph[i & 1], abort, a.status);
                cph[i & 1] ^= 1u;
            }
            const float *po = buf[i & 1];
#pragma unroll 2
            for (int p = 0; p < np; ++p) {
#pragma unroll
                for (int k = 0; k < NK; ++k) {
                    const int idx = tid + k * kConsThreads;
                    if (idx < G * D) acc[k] = fmaf(ml[((p0 + p) * GP + hk[k]) * 2], po[p * G * D + idx], acc[k]);
                }
            }
            named_barrier(1, kConsThreads);  // everyone is done with this buffer before it is refilled
            if (tid == 0 && i + 2 < npieces) issue_piece(i + 2, 0u);
        }
#pragma unroll
        for (int k = 0; k < NK; ++k) {
            const int idx = tid + k * kConsThreads;
            if (idx < G * D)
                reinterpret_cast<T *>(a.out)[pend_out[j] + idx] = Elt<T>::from_float(acc[k] / tail->lsum[hk[k]]);
        }
        named_barrier(1, kConsThreads);
    }
}

// first-use set-up (function attributes, the static scratch address) may be reached from several host threads
std::mutex g_setup_mutex;

template <typename T, int D, int G>
arb_status launch_one(Ctx *ctx, const DecodeArgs &args, bool overlap, cudaStream_t stream) {
    using C = Cfg<T, D, G>;
    const size_t smem = smem_bytes<T, D, G>(args.batch);
    static bool attr_set[64] = {};
    {
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!attr_set[ctx->device & 63]) {
            if (cudaFuncSetAttribute(decode_kernel<T, D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem_bytes<T, D, G>(kMaxBatch)) != cudaSuccess)
                return ARB_ERR_CUDA;
            attr_set[ctx->device & 63] = true;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctx->num_sms * C::CTAS);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, decode_kernel<T, D, G>, args);
    ctx->launches++;
    return err == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

template <typename T, int D>
arb_status launch_g(Ctx *ctx, int g, const DecodeArgs &args, bool overlap, cudaStream_t stream) {
    switch (g) {
        case 1: return launch_one<T, D, 1>(ctx, args, overlap, stream);
        case 2: return launch_one<T, D, 2>(ctx, args, overlap, stream);
        case 3: return launch_one<T, D, 3>(ctx, args, overlap, stream);
        case 4: return launch_one<T, D, 4>(ctx, args, overlap, stream);
        case 5: return launch_one<T, D, 5>(ctx, args, overlap, stream);
        case 6: return launch_one<T, D, 6>(ctx, args, overlap, stream);
        case 7: return launch_one<T, D, 7>(ctx, args, overlap, stream);
        case 8: return launch_one<T, D, 8>(ctx, args, overlap, stream);
        default: return ARB_ERR_UNSUPPORTED;
    }
}

inline size_t slot_count(const arb_attn_params &p, int num_sms) {
    return (size_t)p.batch * p.num_kv_heads + (size_t)num_sms * kMaxCtasPerSm;
}

// ---- scratch for arb_attn_decode_static ------------------------------------------------------------
// In host code `g_static_scratch` is only a stand-in for the symbol, not a device address; the
// address a kernel can use comes from cudaGetSymbolAddress, once per device.
constexpr size_t kStaticScratchBytes = 4u << 20;
constexpr int kStaticMaxBk = 1024;                              // batch * kv heads
constexpr size_t kStaticCounterBytes = sizeof(int) * kStaticMaxBk + 256;   // counters, then the status word
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticSetup {
    bool ready = false;
    unsigned char *base = nullptr;
    int num_sms = 0;
};
StaticSetup g_static_setup[64];

}  // namespace

arb_status launch_decode_static(const arb_attn_params &p, const void *q, const void *k_pages, const void *v_pages,
                                const int32_t *block_table, const int32_t *seq_lens, const int32_t *q_lens,
                                void *out, uint32_t *device_status, cudaStream_t stream) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ARB_ERR_CUDA;
    StaticSetup &su = g_static_setup[dev];
    std::unique_lock<std::mutex> setup_lock(g_setup_mutex);
    if (!su.ready) {  // first call on this device: it is current, so the symbol resolves to its copy
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return ARB_ERR_CUDA;
        }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
            return ARB_ERR_CUDA;
        su.base = static_cast<unsigned char *>(ptr);
        su.num_sms = sms;
        su.ready = true;
    }
    setup_lock.unlock();
    const int g = p.num_q_heads / p.num_kv_heads;
    const int gp = (g + 3) / 4 * 4;
    if ((long long)p.batch * p.num_kv_heads > kStaticMaxBk) return ARB_ERR_STATIC_LIMIT;
    const size_t slots = (size_t)p.batch * p.num_kv_heads + (size_t)su.num_sms * kMaxCtasPerSm;
    const size_t part_o_floats = (slots * g * p.head_dim + 63) & ~size_t(63);
    const size_t need = kStaticCounterBytes + (part_o_floats + slots * gp * 2) * sizeof(float);
    if (need > kStaticScratchBytes) return ARB_ERR_STATIC_LIMIT;

    // [counters | internal status word | pad to 256 B][partial outputs][partial max/sum records]
    int *counters = reinterpret_cast<int *>(su.base);
    uint32_t *own_status = reinterpret_cast<uint32_t *>(su.base + sizeof(int) * kStaticMaxBk);
    if (cudaMemsetAsync(su.base, 0, kStaticCounterBytes, stream) != cudaSuccess) return ARB_ERR_CUDA;

    Ctx tmp;  // launch bookkeeping only; owns nothing
    tmp.device = dev;
    tmp.num_sms = su.num_sms;
    DecodeArgs a;
    a.q = static_cast<const char *>(q);
    a.k_pages = static_cast<const char *>(k_pages);
    a.v_pages = static_cast<const char *>(v_pages);
    a.block_table = block_table;
    a.seq_lens = seq_lens;
    a.q_lens = q_lens;
    a.out = static_cast<char *>(out);
    a.part_o = reinterpret_cast<float *>(su.base + kStaticCounterBytes);
    a.part_ml = a.part_o + part_o_floats;
    a.counters = counters;
    a.status = device_status ? device_status : own_status;
    a.batch = p.batch;
    a.Hq = p.num_q_heads;
    a.Hkv = p.num_kv_heads;
    a.num_pages = p.num_pages;
    a.max_pages = p.max_pages_per_seq;
    const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.head_dim);
    a.scale_log2 = scale * 1.4426950408889634f;
    if (p.dtype == ARB_BF16) {
        if (p.head_dim == 128) return launch_g<__nv_bfloat16, 128>(&tmp, g, a, false, stream);
        if (p.head_dim == 64) return launch_g<__nv_bfloat16, 64>(&tmp, g, a, false, stream);
    } else if (p.dtype == ARB_F32) {
        if (p.head_dim == 128) return launch_g<float, 128>(&tmp, g, a, false, stream);
        if (p.head_dim == 64) return launch_g<float, 64>(&tmp, g, a, false, stream);
    }
    return ARB_ERR_UNSUPPORTED;
}

size_t decode_workspace_bytes(const arb_attn_params &p, int num_sms) {
    const int g = p.num_q_heads / p.num_kv_heads;
    const int gp = (g + 3) / 4 * 4;
    return slot_count(p, num_sms) * ((size_t)g * p.head_dim + 2 * (size_t)gp) * sizeof(float) + 256;
}

arb_status launch_decode(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages,
                         const void *v_pages, const int32_t *block_table, const int32_t *seq_lens,
                         const int32_t *q_lens, void *out, cudaStream_t stream) {
    const int g = p.num_q_heads / p.num_kv_heads;
    const size_t slots = slot_count(p, ctx->num_sms);
    DecodeArgs a;
    a.q = static_cast<const char *>(q);
    a.k_pages = static_cast<const char *>(k_pages);
    a.v_pages = static_cast<const char *>(v_pages);
    a.block_table = block_table;
    a.seq_lens = seq_lens;
    a.q_lens = q_lens;
    a.out = static_cast<char *>(out);
    a.part_o = reinterpret_cast<float *>(ctx->workspace);
    a.part_ml = a.part_o + ((slots * g * p.head_dim + 63) & ~size_t(63));  // keeps 256-byte alignment
    a.counters = ctx->counters;
    a.status = ctx->status;
    a.batch = p.batch;
    a.Hq = p.num_q_heads;
    a.Hkv = p.num_kv_heads;
    a.num_pages = p.num_pages;
    a.max_pages = p.max_pages_per_seq;
    const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.head_dim);
    a.scale_log2 = scale * 1.4426950408889634f;
    const bool overlap = (p.flags & ARB_ATTN_OVERLAP_PREVIOUS) != 0;
    if (p.dtype == ARB_BF16) {
        if (p.head_dim == 128) return launch_g<__nv_bfloat16, 128>(ctx, g, a, overlap, stream);
        if (p.head_dim == 64) return launch_g<__nv_bfloat16, 64>(ctx, g, a, overlap, stream);
    } else if (p.dtype == ARB_F32) {
        if (p.head_dim == 128) return launch_g<float, 128>(ctx, g, a, overlap, stream);
        if (p.head_dim == 64) return launch_g<float, 64>(ctx, g, a, overlap, stream);
    }
    return ARB_ERR_UNSUPPORTED;
}

}  // namespace arb

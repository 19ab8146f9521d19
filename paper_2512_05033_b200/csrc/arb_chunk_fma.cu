// Step-chunk attention, CUDA-core path: one CTA per (query row, kv head).
//
// This is the path for chunks the tensor-core kernel does not take: fp32 inputs (whose 1e-5 tolerance
// rules out tf32), head_dim 64, groups above 8, and every chunk when ARB_ATTN_NO_TENSOR_CORES is set.  It
// also zero-fills the rows of chunk sequences whose lengths are invalid, whatever their size.  Query token i of
// a chunk of n tokens sits at position pos = L - n + i and attends keys 0..pos; the causal mask is
// just each row's own key count.  K and V rows are read straight from global memory with 16-byte
// loads (the rows of one chunk are re-read by neighbouring CTAs out of L2); each group of lanes that
// shares a row keeps an online-softmax state (max, sum, accumulator), merged through shared memory
// at the end.
#include "arb_common.cuh"

namespace arb {

namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;

struct ChunkArgs {
    const char *q;
    const char *k_pages;
    const char *v_pages;
    const int32_t *block_table;
    const int32_t *seq_lens;
    const int32_t *q_lens;
    char *out;
    uint32_t *status;
    int batch, Hq, Hkv, num_pages, max_pages;
    int n_lo, n_hi;  // this kernel owns the sequences with n_lo <= q_len <= n_hi ...
    int skip_rows;   // ... except valid ones with q_len * group >= skip_rows (> 0): the tensor-core kernel has them
    const int *needed;  // with skip_rows > 0: written by the tensor-core kernel, 0 = nothing is left for this one
    int jobs;        // (query row, kv head) pairs: total_q * Hkv; the CTAs take them in turn
    float scale_log2;
};

// One (query row, kv head) pair; every thread of the block takes part.  rec: [NGROUPS][REC] floats of shared
// memory; row0: the prefix sums of the q_lens.
template <typename T, int D, int G>
__device__ void chunk_fma_job(const ChunkArgs &a, int job, float *rec, const int *row0) {
    constexpr int EPL = Elt<T>::kPerVec;
    constexpr int ROW_BYTES = D * (int)sizeof(T);
    constexpr int LPR = ROW_BYTES / 16;
    constexpr int RPP = 32 / LPR;
    constexpr int NGROUPS = kWarps * RPP;
    constexpr int REC = G * (D + 2);  // floats per group record: m[G], l[G], o[G][D]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.batch;
    const int row = job / a.Hkv, kvh = job - row * a.Hkv;
    if (row >= row0[B]) return;
    int lo = 0, hi = B;  // largest b with row0[b] <= row
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (row0[mid] <= row) lo = mid; else hi = mid;
    }
    const int b = lo;
    const int n = a.q_lens[b], L = a.seq_lens[b];
    if (n < a.n_lo || n > a.n_hi) return;  // another kernel owns this sequence
    T *orow = reinterpret_cast<T *>(a.out) + ((size_t)row * a.Hq + kvh * G) * D;
    if (L < n || L > a.max_pages * kPage) {
        if (tid == 0) atomicOr(a.status, (uint32_t)ARB_DEV_BAD_SEQ_LEN);
        for (int idx = tid; idx < G * D; idx += kThreads) orow[idx] = Elt<T>::from_float(0.f);
        return;
    }
    if (a.skip_rows > 0 && n * G >= a.skip_rows) return;
    const int i = row - row0[b];
    const int nkeys = L - n + i + 1;
    const int npages = (nkeys + kPage - 1) / kPage;

    const int lg = lane % LPR, rg = lane / LPR;
    float qf[G][EPL];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(
            a.q + (((size_t)row * a.Hq + kvh * G + h) * D + lg * EPL) * sizeof(T)));
        Elt<T>::unpack(v, qf[h]);
#pragma unroll
        for (int e = 0; e < EPL; ++e) qf[h][e] *= a.scale_log2;
    }
    float m[G], l[G], o[G][EPL];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        m[h] = -INFINITY;
        l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[h][e] = 0.f;
    }

    for (int pg = warp; pg < npages; pg += kWarps) {
        int pid = a.block_table[(size_t)b * a.max_pages + pg];
        if ((unsigned)pid >= (unsigned)a.num_pages) {
            if (lane == 0) atomicOr(a.status, (uint32_t)ARB_DEV_BAD_PAGE);
            pid = 0;
        }
        const size_t tile = ((size_t)pid * a.Hkv + kvh) * kPage * ROW_BYTES;
        for (int r = rg; r < kPage; r += RPP) {
            const int key = pg * kPage + r;
            const bool valid = key < nkeys;  // uniform within a row group
            float s[G];
            if (valid) {
                const uint4 kv = __ldg(reinterpret_cast<const uint4 *>(a.k_pages + tile + r * ROW_BYTES + lg * 16));
                float kf[EPL];
                Elt<T>::unpack(kv, kf);
#pragma unroll
                for (int h = 0; h < G; ++h) {
                    float acc = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc = fmaf(qf[h][e], kf[e], acc);
                    s[h] = acc;
                }
            } else {
#pragma unroll
                for (int h = 0; h < G; ++h) s[h] = 0.f;
            }
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int off = LPR / 2; off >= 1; off >>= 1) s[h] += __shfl_xor_sync(0xffffffffu, s[h], off);
            if (valid) {
                const uint4 vv = __ldg(reinterpret_cast<const uint4 *>(a.v_pages + tile + r * ROW_BYTES + lg * 16));
                float vf[EPL];
                Elt<T>::unpack(vv, vf);
#pragma unroll
                for (int h = 0; h < G; ++h) {
                    const float mn = fmaxf(m[h], s[h]);
                    const float f = fast_exp2(m[h] - mn);
                    const float p = fast_exp2(s[h] - mn);
                    l[h] = fmaf(l[h], f, p);
#pragma unroll
                    for (int e = 0; e < EPL; ++e) o[h][e] = fmaf(o[h][e], f, p * vf[e]);
                    m[h] = mn;
                }
            }
        }
    }

    // every row group leaves its record, then all threads merge them
    float *my = rec + (warp * RPP + rg) * REC;
#pragma unroll
    for (int h = 0; h < G; ++h) {
        if (lg == 0) { my[h] = m[h]; my[G + h] = l[h]; }
#pragma unroll
        for (int e = 0; e < EPL; ++e) my[2 * G + h * D + lg * EPL + e] = o[h][e];
    }
    __syncthreads();
    for (int idx = tid; idx < G * D; idx += kThreads) {
        const int h = idx / D;
        float M = -INFINITY;
        for (int gI = 0; gI < NGROUPS; ++gI) M = fmaxf(M, rec[gI * REC + h]);
        float ls = 0.f, acc = 0.f;
        for (int gI = 0; gI < NGROUPS; ++gI) {
            const float mg = rec[gI * REC + h];
            const float w = (mg == -INFINITY) ? 0.f : fast_exp2(mg - M);
            ls = fmaf(w, rec[gI * REC + G + h], ls);
            acc = fmaf(w, rec[gI * REC + 2 * G + idx], acc);
        }
        orow[idx] = Elt<T>::from_float(acc / ls);
    }
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kThreads) chunk_fma_kernel(const ChunkArgs a) {
    constexpr int ROW_BYTES = D * (int)sizeof(T);
    constexpr int LPR = ROW_BYTES / 16;
    constexpr int RPP = 32 / LPR;
    constexpr int NGROUPS = kWarps * RPP;
    constexpr int REC = G * (D + 2);

    extern __shared__ float sm[];
    float *rec = sm;                                      // [NGROUPS][REC]
    int *row0 = reinterpret_cast<int *>(sm + NGROUPS * REC);  // [B + 1]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.batch;
    pdl_enter();
    if (a.skip_rows > 0 && a.needed != nullptr && *a.needed == 0) return;  // the usual case: every chunk was large

    if (tid == 0) row0[0] = 0;
    for (int b = tid; b < B; b += kThreads) row0[b + 1] = max(a.q_lens[b], 0);
    __syncthreads();
    if (warp == 0) {
        int carry = 0;
        for (int b0 = 0; b0 < B; b0 += 32) {
            const int b = b0 + lane;
            int v = b < B ? row0[b + 1] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, v, off);
                if (lane >= off) v += t;
            }
            if (b < B) row0[b + 1] = v + carry;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
    }
    __syncthreads();
    // the grid is bounded (a call whose chunks all went to the tensor cores would otherwise start, and end at once,
    // one CTA per query row and kv head): the CTAs take the jobs in turn
    for (int job = blockIdx.x; job < a.jobs; job += gridDim.x) {
        chunk_fma_job<T, D, G>(a, job, rec, row0);
        __syncthreads();   // the records are free again
    }
}

template <typename T, int D, int G>
arb_status launch_one(Ctx *ctx, const ChunkArgs &a, int total_q, cudaStream_t stream) {
    constexpr int LPR = D * (int)sizeof(T) / 16;
    constexpr int NGROUPS = kWarps * (32 / LPR);
    const size_t smem = sizeof(float) * NGROUPS * G * (D + 2) + sizeof(int) * ((size_t)a.batch + 1);
    static bool attr_set[64] = {};
    if (!attr_set[ctx->device & 63]) {
        const size_t mx = sizeof(float) * NGROUPS * G * (D + 2) + sizeof(int) * (kMaxBatch + 1);
        if (cudaFuncSetAttribute(chunk_fma_kernel<T, D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mx) !=
            cudaSuccess)
            return ARB_ERR_CUDA;
        attr_set[ctx->device & 63] = true;
    }
    const int grid = a.jobs < 8 * ctx->num_sms ? a.jobs : 8 * ctx->num_sms;
    const cudaError_t err = launch_pdl(chunk_fma_kernel<T, D, G>, dim3(grid), dim3(kThreads), smem, stream, a);
    ctx->launches++;
    return err == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

template <typename T, int D>
arb_status launch_g(Ctx *ctx, int g, const ChunkArgs &a, int total_q, cudaStream_t stream) {
    switch (g) {
        case 1: return launch_one<T, D, 1>(ctx, a, total_q, stream);
        case 2: return launch_one<T, D, 2>(ctx, a, total_q, stream);
        case 3: return launch_one<T, D, 3>(ctx, a, total_q, stream);
        case 4: return launch_one<T, D, 4>(ctx, a, total_q, stream);
        case 5: return launch_one<T, D, 5>(ctx, a, total_q, stream);
        case 6: return launch_one<T, D, 6>(ctx, a, total_q, stream);
        case 7: return launch_one<T, D, 7>(ctx, a, total_q, stream);
        case 8: return launch_one<T, D, 8>(ctx, a, total_q, stream);
        default: return ARB_ERR_UNSUPPORTED;
    }
}

}  // namespace

arb_status launch_chunk_fma(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages,
                            const void *v_pages, const int32_t *block_table, const int32_t *seq_lens,
                            const int32_t *q_lens, void *out, int n_lo, int n_hi, int skip_rows,
                            cudaStream_t stream) {
    const int *needed = skip_rows > 0 ? ctx->rot + (size_t)kRotSets * kRotCounters + kRotSets + 2 : nullptr;
    ChunkArgs a;
    a.q = static_cast<const char *>(q);
    a.k_pages = static_cast<const char *>(k_pages);
    a.v_pages = static_cast<const char *>(v_pages);
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
    a.n_lo = n_lo;
    a.n_hi = n_hi;
    a.skip_rows = skip_rows;
    a.needed = needed;
    a.jobs = p.total_q * p.num_kv_heads;
    const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.head_dim);
    a.scale_log2 = scale * 1.4426950408889634f;
    const int g = p.num_q_heads / p.num_kv_heads;
    if (p.dtype == ARB_BF16) {
        if (p.head_dim == 128) return launch_g<__nv_bfloat16, 128>(ctx, g, a, p.total_q, stream);
        if (p.head_dim == 64) return launch_g<__nv_bfloat16, 64>(ctx, g, a, p.total_q, stream);
    } else if (p.dtype == ARB_F32) {
        if (p.head_dim == 128) return launch_g<float, 128>(ctx, g, a, p.total_q, stream);
        if (p.head_dim == 64) return launch_g<float, 64>(ctx, g, a, p.total_q, stream);
    }
    return ARB_ERR_UNSUPPORTED;
}

}  // namespace arb

// KV append: the keys and values of a step's new tokens go into the paged cache, right behind the
// tokens each sequence already holds (the write every "Sample ... step" line of Algorithm 1 of the
// paper implies before the next token, or the router's forward, attends to them).
//
// k_new, v_new are [total_new, Hkv, D], packed by sequence; token j of sequence b lands at position
// seq_lens[b] + j: page block_table[b][pos / 16], slot pos % 16 of the head-major pools
// [num_pages, Hkv, 16, D].  Plain memory movement: a (token, kv head) row of D elements is 256 or 512
// contiguous bytes on both sides, copied as 16-byte vectors, one row per half warp or warp.  Nothing
// is known on the host but the total number of new tokens; every CTA derives the row offsets from
// new_lens (scan in shared memory) and checks each sequence once: new tokens that do not fit under the
// block table, or that would land on a page outside the pool, leave that sequence untouched and set a
// status bit.  Lengths are advanced inside the same kernel by the CTA that finishes last (an arrival counter
// tells it, see advance_lens_when_last): by then every CTA has read the old lengths for the rows it placed.
//
// The quantising form writes an E4M3 cache (one byte per element: 1 sign, 4 exponent bits with bias 7, 3
// mantissa bits, largest finite value 448): code = e4m3(x * inv_scale), the product in fp32, the conversion
// to nearest with ties to even and saturation (cvt.rn.satfinite.e4m3x2.f32).  Same plan, same checks; a
// thread turns one 16-byte piece of a source row into 8 (bf16 source) or 4 (fp32 source) bytes.
#include "arb_common.cuh"

namespace arb {

namespace {

constexpr int kAppendThreads = 256;

struct AppendArgs {
    const char *k_new, *v_new;
    char *k_pages, *v_pages;
    const int32_t *block_table;
    int32_t *seq_lens;
    const int32_t *new_lens;
    uint32_t *status;
    int batch, Hkv, num_pages, max_pages;
    int row_bytes;   // D * element size: bytes of one (token, kv head) row
    int total_new;
    int update_lens;     // seq_lens += new_lens once every CTA has placed its rows
    int *done_counter;   // CTAs of this call that have; zero between calls
};

// 0 = append, otherwise the status bit that explains why not (new_len == 0 appends nothing and is fine)
__device__ __forceinline__ uint32_t append_check(const AppendArgs &a, int b) {
    const int n = a.new_lens[b], L = a.seq_lens[b];
    if (n == 0) return 0;
    if (n < 0 || L < 0 || (long long)L + n > (long long)a.max_pages * kPage) return ARB_DEV_BAD_SEQ_LEN;
    for (int pg = L / kPage; pg <= (L + n - 1) / kPage; ++pg) {
        const int page = a.block_table[(size_t)b * a.max_pages + pg];
        if ((unsigned)page >= (unsigned)a.num_pages) return ARB_DEV_BAD_PAGE;
    }
    return 0;
}

// The lengths move forward inside the append kernel: every CTA reads the old lengths for the rows it places, so
// the CTA that finishes last (a counter tells it) adds new_lens, and leaves the counter at zero for the next call.
// `okay` is this CTA's copy of the per-sequence checks, taken from the old lengths.
__device__ __forceinline__ void advance_lens_when_last(const AppendArgs &a, const int *okay) {
    if (!a.update_lens) return;
    __shared__ int is_last;
    __syncthreads();   // all rows of this CTA are placed, all its reads of seq_lens are done
    if (threadIdx.x == 0) {
        __threadfence();
        is_last = atomicAdd(a.done_counter, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (!is_last) return;
    for (int b = threadIdx.x; b < a.batch; b += kAppendThreads) {
        const int n = a.new_lens[b];
        if (n > 0 && okay[b]) a.seq_lens[b] += n;
    }
    if (threadIdx.x == 0) *a.done_counter = 0;
}

__global__ void __launch_bounds__(kAppendThreads)
kv_append_kernel(const AppendArgs a) {
    extern __shared__ int asm_[];
    int *pref = asm_;                  // [B + 1] new rows before sequence b
    int *okay = pref + a.batch + 1;    // [B] the sequence's new tokens may be written
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.batch;
    pdl_enter();
    if (tid == 0) pref[0] = 0;
    for (int b = tid; b < B; b += kAppendThreads) {
        const uint32_t bad = append_check(a, b);
        if (bad && blockIdx.x == 0) atomicOr(a.status, bad);
        okay[b] = bad == 0;
        const int n = a.new_lens[b];
        pref[b + 1] = n > 0 ? n : 0;
    }
    __syncthreads();
    if (warp == 0) {
        int carry = 0;
        for (int b0 = 0; b0 < B; b0 += 32) {
            const int b = b0 + lane;
            int v = b < B ? pref[b + 1] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, v, off);
                if (lane >= off) v += t;
            }
            if (b < B) pref[b + 1] = v + carry;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
    }
    __syncthreads();
    const int total = min(pref[B], a.total_new);
    const int vecs = a.row_bytes / 16;             // 16 (bf16, D 128 / fp32, D 64), 8 or 32
    const int rows_per_pass = kAppendThreads / vecs;
    const int sub = tid / vecs, vec = tid - sub * vecs;
    const long long nrows = (long long)total * a.Hkv;
    for (long long r = (long long)blockIdx.x * rows_per_pass + sub; r < nrows; r += (long long)gridDim.x * rows_per_pass) {
        const int tok = (int)(r / a.Hkv), h = (int)(r - (long long)tok * a.Hkv);
        int lo = 0, hi = B;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (pref[mid] <= tok) lo = mid; else hi = mid;
        }
        if (!okay[lo]) continue;
        const int pos = a.seq_lens[lo] + (tok - pref[lo]);
        const int page = a.block_table[(size_t)lo * a.max_pages + pos / kPage];
        const size_t dst = (((size_t)page * a.Hkv + h) * kPage + (pos % kPage)) * a.row_bytes + (size_t)vec * 16;
        const size_t src = (size_t)r * a.row_bytes + (size_t)vec * 16;
        if (!ARB_IN_RANGE(a.status, dst + 15, (size_t)a.num_pages * a.Hkv * kPage * a.row_bytes)) continue;
        const uint4 kx = __ldg(reinterpret_cast<const uint4 *>(a.k_new + src));
        const uint4 vx = __ldg(reinterpret_cast<const uint4 *>(a.v_new + src));
        *reinterpret_cast<uint4 *>(a.k_pages + dst) = kx;
        *reinterpret_cast<uint4 *>(a.v_pages + dst) = vx;
    }
    advance_lens_when_last(a, okay);
}

// two values -> two E4M3 codes; lo lands in the low byte
__device__ __forceinline__ uint32_t e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

template <typename T>
__global__ void __launch_bounds__(kAppendThreads)
kv_append_e4m3_kernel(const AppendArgs a, float k_inv_scale, float v_inv_scale) {
    constexpr int EPL = Elt<T>::kPerVec;   // source elements per 16-byte piece = code bytes written per thread
    extern __shared__ int asm_[];
    int *pref = asm_;
    int *okay = pref + a.batch + 1;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.batch;
    pdl_enter();
    if (tid == 0) pref[0] = 0;
    for (int b = tid; b < B; b += kAppendThreads) {
        const uint32_t bad = append_check(a, b);
        if (bad && blockIdx.x == 0) atomicOr(a.status, bad);
        okay[b] = bad == 0;
        const int n = a.new_lens[b];
        pref[b + 1] = n > 0 ? n : 0;
    }
    __syncthreads();
    if (warp == 0) {
        int carry = 0;
        for (int b0 = 0; b0 < B; b0 += 32) {
            const int b = b0 + lane;
            int v = b < B ? pref[b + 1] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, v, off);
                if (lane >= off) v += t;
            }
            if (b < B) pref[b + 1] = v + carry;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
    }
    __syncthreads();
    const int total = min(pref[B], a.total_new);
    const int vecs = a.row_bytes / 16;             // 16-byte pieces of a source row
    const int D = vecs * EPL;                      // = bytes of a row of codes
    const int rows_per_pass = kAppendThreads / vecs;
    const int sub = tid / vecs, vec = tid - sub * vecs;
    const long long nrows = (long long)total * a.Hkv;
    for (long long r = (long long)blockIdx.x * rows_per_pass + sub; r < nrows; r += (long long)gridDim.x * rows_per_pass) {
        const int tok = (int)(r / a.Hkv), h = (int)(r - (long long)tok * a.Hkv);
        int lo = 0, hi = B;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (pref[mid] <= tok) lo = mid; else hi = mid;
        }
        if (!okay[lo]) continue;
        const int pos = a.seq_lens[lo] + (tok - pref[lo]);
        const int page = a.block_table[(size_t)lo * a.max_pages + pos / kPage];
        const size_t dst = (((size_t)page * a.Hkv + h) * kPage + (pos % kPage)) * D + (size_t)vec * EPL;
        const size_t src = (size_t)r * a.row_bytes + (size_t)vec * 16;
        float kf[EPL], vf[EPL];
        Elt<T>::unpack(__ldg(reinterpret_cast<const uint4 *>(a.k_new + src)), kf);
        Elt<T>::unpack(__ldg(reinterpret_cast<const uint4 *>(a.v_new + src)), vf);
        uint32_t kc[EPL / 4], vc[EPL / 4];
#pragma unroll
        for (int w = 0; w < EPL / 4; ++w) {
            kc[w] = e4m3x2(kf[4 * w] * k_inv_scale, kf[4 * w + 1] * k_inv_scale) |
                    (e4m3x2(kf[4 * w + 2] * k_inv_scale, kf[4 * w + 3] * k_inv_scale) << 16);
            vc[w] = e4m3x2(vf[4 * w] * v_inv_scale, vf[4 * w + 1] * v_inv_scale) |
                    (e4m3x2(vf[4 * w + 2] * v_inv_scale, vf[4 * w + 3] * v_inv_scale) << 16);
        }
        if (EPL == 8) {
            *reinterpret_cast<uint2 *>(a.k_pages + dst) = make_uint2(kc[0], kc[EPL / 4 - 1]);
            *reinterpret_cast<uint2 *>(a.v_pages + dst) = make_uint2(vc[0], vc[EPL / 4 - 1]);
        } else {
            *reinterpret_cast<uint32_t *>(a.k_pages + dst) = kc[0];
            *reinterpret_cast<uint32_t *>(a.v_pages + dst) = vc[0];
        }
    }
    advance_lens_when_last(a, okay);
}

// The 4-bit cache's quantising append (bf16 rows of 128 values).  A row is held by 16 neighbouring threads, 8 values
// each: its scale is max|x| / 7 over the 16 threads (shuffles within the half warp), its codes rint(x * (7 / max|x|))
// clamped to -7 .. 7, both divisions IEEE; a thread's eight codes are one 32-bit word of nibbles (code + 8; nibbles
// 0..7 = dimensions 0, 2, 4, 6, 1, 3, 5, 7 of the eight).  Same plan, same checks as kv_append_kernel.
__device__ __forceinline__ uint32_t i4_word(const float (&x)[8], float m, float &scale) {
    scale = m > 0.f ? __fdiv_rn(m, 7.f) : 0.f;
    const float inv = m > 0.f ? __fdiv_rn(7.f, m) : 0.f;
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int c = max(-7, min(7, __float2int_rn(__fmul_rn(x[j], inv))));
        word |= (uint32_t)(c + 8) << (4 * ((j >> 1) + 4 * (j & 1)));
    }
    return word;
}

__global__ void __launch_bounds__(kAppendThreads)
kv_append_i4_kernel(const AppendArgs a, float *k_scales, float *v_scales) {
    extern __shared__ int asm_[];
    int *pref = asm_;
    int *okay = pref + a.batch + 1;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int B = a.batch;
    pdl_enter();
    if (tid == 0) pref[0] = 0;
    for (int b = tid; b < B; b += kAppendThreads) {
        const uint32_t bad = append_check(a, b);
        if (bad && blockIdx.x == 0) atomicOr(a.status, bad);
        okay[b] = bad == 0;
        const int n = a.new_lens[b];
        pref[b + 1] = n > 0 ? n : 0;
    }
    __syncthreads();
    if (warp == 0) {
        int carry = 0;
        for (int b0 = 0; b0 < B; b0 += 32) {
            const int b = b0 + lane;
            int v = b < B ? pref[b + 1] : 0;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, v, off);
                if (lane >= off) v += t;
            }
            if (b < B) pref[b + 1] = v + carry;
            carry += __shfl_sync(0xffffffffu, v, 31);
        }
    }
    __syncthreads();
    const int total = min(pref[B], a.total_new);
    constexpr int kVecs = 16;                      // 16-byte pieces of a bf16 row of 128 values
    constexpr int kRowsPerPass = kAppendThreads / kVecs;
    const int sub = tid / kVecs, vec = tid - sub * kVecs;
    const uint32_t half_mask = 0xffffu << (lane & 16);   // the 16 lanes that hold this row
    const long long nrows = (long long)total * a.Hkv;
    for (long long r = (long long)blockIdx.x * kRowsPerPass + sub; r < nrows; r += (long long)gridDim.x * kRowsPerPass) {
        const int tok = (int)(r / a.Hkv), h = (int)(r - (long long)tok * a.Hkv);
        int lo = 0, hi = B;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (pref[mid] <= tok) lo = mid; else hi = mid;
        }
        if (!okay[lo]) continue;   // (the same for the 16 lanes of the row)
        const int pos = a.seq_lens[lo] + (tok - pref[lo]);
        const int page = a.block_table[(size_t)lo * a.max_pages + pos / kPage];
        const size_t slot_row = ((size_t)page * a.Hkv + h) * kPage + (pos % kPage);
        const size_t src = (size_t)r * a.row_bytes + (size_t)vec * 16;
        float kf[8], vf[8];
        Elt<__nv_bfloat16>::unpack(__ldg(reinterpret_cast<const uint4 *>(a.k_new + src)), kf);
        Elt<__nv_bfloat16>::unpack(__ldg(reinterpret_cast<const uint4 *>(a.v_new + src)), vf);
        float mk = 0.f, mv = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) { mk = fmaxf(mk, fabsf(kf[j])); mv = fmaxf(mv, fabsf(vf[j])); }
#pragma unroll
        for (int off = 8; off >= 1; off >>= 1) {
            mk = fmaxf(mk, __shfl_xor_sync(half_mask, mk, off));
            mv = fmaxf(mv, __shfl_xor_sync(half_mask, mv, off));
        }
        float ks, vs;
        const uint32_t kw = i4_word(kf, mk, ks), vw = i4_word(vf, mv, vs);
        *reinterpret_cast<uint32_t *>(a.k_pages + slot_row * 64 + vec * 4) = kw;
        *reinterpret_cast<uint32_t *>(a.v_pages + slot_row * 64 + vec * 4) = vw;
        if (vec == 0) { k_scales[slot_row] = ks; v_scales[slot_row] = vs; }
    }
    advance_lens_when_last(a, okay);
}

}  // namespace

arb_status launch_kv_append(Ctx *ctx, const arb_attn_params &p, int total_new, const void *k_new, const void *v_new,
                            const int32_t *block_table, int32_t *seq_lens, const int32_t *new_lens, int update_lens,
                            void *k_pages, void *v_pages, cudaStream_t stream) {
    AppendArgs a;
    a.k_new = static_cast<const char *>(k_new);
    a.v_new = static_cast<const char *>(v_new);
    a.k_pages = static_cast<char *>(k_pages);
    a.v_pages = static_cast<char *>(v_pages);
    a.block_table = block_table;
    a.seq_lens = seq_lens;
    a.new_lens = new_lens;
    a.status = ctx->status;
    a.batch = p.batch;
    a.Hkv = p.num_kv_heads;
    a.num_pages = p.num_pages;
    a.max_pages = p.max_pages_per_seq;
    a.row_bytes = p.head_dim * (p.dtype == ARB_BF16 ? 2 : 4);
    a.total_new = total_new;
    a.update_lens = update_lens;
    a.done_counter = ctx->rot + (size_t)kRotSets * kRotCounters + kRotSets + 3;
    const int rows_per_pass = kAppendThreads / (a.row_bytes / 16);
    const long long nrows = (long long)total_new * p.num_kv_heads;
    long long want = (nrows + rows_per_pass - 1) / rows_per_pass;
    const long long cap = (long long)ctx->num_sms * 4;
    const int grid = (int)(want < 1 ? 1 : (want > cap ? cap : want));
    const size_t smem = sizeof(int) * (2 * (size_t)p.batch + 1);
    const cudaError_t err = launch_pdl(kv_append_kernel, dim3(grid), dim3(kAppendThreads), smem, stream, a);
    ctx->launches++;
    return err == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

arb_status launch_kv_append_e4m3(Ctx *ctx, const arb_attn_params &p, int total_new, const void *k_new,
                                 const void *v_new, float k_inv_scale, float v_inv_scale, const int32_t *block_table,
                                 int32_t *seq_lens, const int32_t *new_lens, int update_lens, void *k_codes,
                                 void *v_codes, cudaStream_t stream) {
    AppendArgs a;
    a.k_new = static_cast<const char *>(k_new);
    a.v_new = static_cast<const char *>(v_new);
    a.k_pages = static_cast<char *>(k_codes);
    a.v_pages = static_cast<char *>(v_codes);
    a.block_table = block_table;
    a.seq_lens = seq_lens;
    a.new_lens = new_lens;
    a.status = ctx->status;
    a.batch = p.batch;
    a.Hkv = p.num_kv_heads;
    a.num_pages = p.num_pages;
    a.max_pages = p.max_pages_per_seq;
    a.row_bytes = p.head_dim * (p.dtype == ARB_BF16 ? 2 : 4);   // of the source rows
    a.total_new = total_new;
    a.update_lens = update_lens;
    a.done_counter = ctx->rot + (size_t)kRotSets * kRotCounters + kRotSets + 3;
    const int rows_per_pass = kAppendThreads / (a.row_bytes / 16);
    const long long nrows = (long long)total_new * p.num_kv_heads;
    long long want = (nrows + rows_per_pass - 1) / rows_per_pass;
    const long long cap = (long long)ctx->num_sms * 4;
    const int grid = (int)(want < 1 ? 1 : (want > cap ? cap : want));
    const size_t smem = sizeof(int) * (2 * (size_t)p.batch + 1);
    const cudaError_t err =
        p.dtype == ARB_BF16
            ? launch_pdl(kv_append_e4m3_kernel<__nv_bfloat16>, dim3(grid), dim3(kAppendThreads), smem, stream, a, k_inv_scale, v_inv_scale)
            : launch_pdl(kv_append_e4m3_kernel<float>, dim3(grid), dim3(kAppendThreads), smem, stream, a, k_inv_scale, v_inv_scale);
    ctx->launches++;
    return err == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

arb_status launch_kv_append_i4(Ctx *ctx, const arb_attn_params &p, int total_new, const void *k_new, const void *v_new,
                               const int32_t *block_table, int32_t *seq_lens, const int32_t *new_lens, int update_lens,
                               void *k_codes, void *v_codes, float *k_scales, float *v_scales, cudaStream_t stream) {
    AppendArgs a;
    a.k_new = static_cast<const char *>(k_new);
    a.v_new = static_cast<const char *>(v_new);
    a.k_pages = static_cast<char *>(k_codes);
    a.v_pages = static_cast<char *>(v_codes);
    a.block_table = block_table;
    a.seq_lens = seq_lens;
    a.new_lens = new_lens;
    a.status = ctx->status;
    a.batch = p.batch;
    a.Hkv = p.num_kv_heads;
    a.num_pages = p.num_pages;
    a.max_pages = p.max_pages_per_seq;
    a.row_bytes = p.head_dim * 2;   // of the bf16 source rows
    a.total_new = total_new;
    a.update_lens = update_lens;
    a.done_counter = ctx->rot + (size_t)kRotSets * kRotCounters + kRotSets + 3;
    const int rows_per_pass = kAppendThreads / 16;
    const long long nrows = (long long)total_new * p.num_kv_heads;
    long long want = (nrows + rows_per_pass - 1) / rows_per_pass;
    const long long cap = (long long)ctx->num_sms * 4;
    const int grid = (int)(want < 1 ? 1 : (want > cap ? cap : want));
    const size_t smem = sizeof(int) * (2 * (size_t)p.batch + 1);
    const cudaError_t err = launch_pdl(kv_append_i4_kernel, dim3(grid), dim3(kAppendThreads), smem, stream, a, k_scales, v_scales);
    ctx->launches++;
    return err == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

}  // namespace arb

// Shared device helpers and the host-side context of the arb library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/arb.h"

namespace arb {

constexpr int kPage = 16;             // tokens per KV page
constexpr int kMaxBatch = 1024;       // sequences per call (prefix tables live in shared memory)
constexpr int kMaxGroup = 8;          // query heads per KV head
// q_len * group from which a bf16, head_dim-128 chunk goes to the tcgen05 kernel: every chunk.  A tile with few
// query rows wastes tensor-core rows, but the tile streams a sequence's keys once, at memory speed, where the
// CUDA-core kernel re-reads them per query row (measured on rounds of short steps: 0.76 ms against 0.12 ms per
// call; the threshold used to be 64 rows).
constexpr int kChunkMmaMinRows = 2;
constexpr int kDecodeMmaMinGroup = 1; // group size from which bf16 / head_dim 128 decode uses warp-level MMA
constexpr long long kWaitCycles = 1ll << 31;  // bound of every mbarrier wait (about a second)

// ---------------------------------------------------------------------------------------------
// Host-side context
// ---------------------------------------------------------------------------------------------
// One call of the pipelined host entry points in flight: its staging on both sides and the events that order its
// three parts (inputs in, kernels, result out) across the copy streams and the caller's stream.
struct HostSlot {
    char *dev = nullptr;     // [out | q | block table | seq_lens | q_lens]
    size_t dev_bytes = 0;
    char *host = nullptr;    // page-locked, [q | block table | seq_lens | q_lens]
    size_t host_bytes = 0;
    cudaEvent_t in_done = nullptr, kernels_done = nullptr, out_done = nullptr;
    bool busy = false;
};

constexpr int kHostSlots = 32;

struct Ctx {
    int device = 0;
    int num_sms = 0;
    size_t workspace_bytes = 0;
    char *workspace = nullptr;   // split-KV partials
    int *counters = nullptr;     // arrival counters, one per (sequence, kv head); zero between calls
    int counters_len = 0;
    uint32_t *status = nullptr;  // device status word
    uint64_t launches = 0;
    // staging for the *_host entry points
    char *stage = nullptr;
    size_t stage_bytes = 0;
    char *host_stage = nullptr;   // page-locked gather buffer of the *_host entry points
    size_t host_stage_bytes = 0;
    // pipelined host calls: a ring of slots and one copy stream per direction, created at the first such call
    HostSlot slots[kHostSlots];
    int next_slot = 0;
    cudaStream_t in_stream = nullptr, out_stream = nullptr;
    bool pipe_ready = false;
    void *map_cache = nullptr;      // tensor maps of the KV pools seen so far (arb_tma.cu)
    unsigned map_evictions = 0;
    // workspace rotation of the tensor-core decode kernel: kRotSets counter arrays, one exit counter
    // per set and the generation of the newest completed call, all in one allocation
    int *rot = nullptr;
    uint32_t decode_gen = 1000;          // generation of the next tensor-core decode call
    uint32_t rot_wait_through = 0;        // tensor-core decode calls up to this generation wait for their predecessor
    double *spearman_acc = nullptr;       // three fp64 accumulators of arb_spearman
    int *step_hint = nullptr;             // single-launch decode: the page tiles each CTA streamed last (arb_decode_step.cu)
    int step_min_chunk = 16;              // single-launch decode: fewest pages worth giving a CTA
    int step_boundary_pct = 100;          // single-launch decode: what a (sequence, kv head) boundary inside a CTA's range counts for
    float *chunk_ws = nullptr;            // partial results of split long sequences (step-chunk attention)
    size_t chunk_ws_bytes = 0;
    // bounds-check build: the guard zones around the buffers above (device addresses), their copy on the device,
    // and the counter the guard check adds up in
    const unsigned char *guards[16] = {};
    int n_guards = 0;
    const unsigned char **guards_dev = nullptr;
    unsigned long long *guard_bad = nullptr;
};

constexpr int kRotSets = 4;
constexpr int kRotCounters = 1 << 16;

// The decode workspace is cut into kRotSets + 1 regions of this size: region 0 for the decode kernels that take
// no generation number, regions 1 .. kRotSets for the rotation of the tensor-core decode kernel.
inline size_t rot_region_bytes(const Ctx *ctx) { return (ctx->workspace_bytes / (kRotSets + 1)) & ~size_t(255); }

// A decode kernel without a generation number is about to use `bytes` of the workspace from its start.  Inside
// region 0 it touches no rotation set.  Beyond it, it may lie over sets that later tensor-core calls would write
// early: those of the next kRotSets generations wait (a later completion, which they would otherwise trust,
// then implies this call's).
inline void note_unnumbered_decode(Ctx *ctx, size_t bytes) {
    if (bytes > rot_region_bytes(ctx)) ctx->rot_wait_through = ctx->decode_gen + (uint32_t)kRotSets - 1u;
}

// ---------------------------------------------------------------------------------------------
// Bounds-check build (-DARB_CHECKS): indices derived on the device are tested before use; a failing test raises
// ARB_DEV_CHECK_FAILED and the caller skips the access.  In the ordinary build the test is `true` and costs nothing.
// ---------------------------------------------------------------------------------------------
#ifdef ARB_CHECKS
#define ARB_IN_RANGE(status, idx, limit)                                  \
    (((unsigned long long)(idx) < (unsigned long long)(limit))            \
         ? true                                                           \
         : (atomicOr((status), (uint32_t)ARB_DEV_CHECK_FAILED), false))
constexpr size_t kGuardBytes = 4096;    // guard zone on either side of every buffer a ctx owns
#else
#define ARB_IN_RANGE(status, idx, limit) true
constexpr size_t kGuardBytes = 0;
#endif
constexpr unsigned char kGuardPattern = 0xA5;

// ---------------------------------------------------------------------------------------------
// Element types
// ---------------------------------------------------------------------------------------------
template <typename T>
struct Elt;

template <>
struct Elt<float> {
    static constexpr int kPerVec = 4;  // elements in one 16-byte vector
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x);
        f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z);
        f[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ float to_float(float x) { return x; }
    __device__ static __forceinline__ float from_float(float x) { return x; }
};

template <>
struct Elt<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    // bf16 -> fp32 is a 16-bit shift: low half << 16, high half masked in place
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[8]) {
        f[0] = __uint_as_float(v.x << 16);
        f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16);
        f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16);
        f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16);
        f[7] = __uint_as_float(v.w & 0xffff0000u);
    }
    __device__ static __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
    __device__ static __forceinline__ __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
};

// ---------------------------------------------------------------------------------------------
// mbarrier and bulk-copy (TMA) wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// The non-blocking form: true if the phase with the given parity has completed, else false at once.
__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Wait for the phase with the given parity.  Every wait is bounded: after `limit` cycles (kWaitCycles in
// every production kernel), or as soon as another thread of the block has given up (*abort != 0), it returns
// false and the caller carries on with whatever is in shared memory; the status word then carries
// ARB_DEV_WAIT_TIMEOUT.
__device__ __forceinline__ bool mbar_wait_limit(uint64_t *bar, uint32_t parity, volatile int *abort,
                                                uint32_t *status, long long limit) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort) return false;
        if (clock64() - t0 > limit) {
            *abort = 1;
            atomicOr(status, (uint32_t)ARB_DEV_WAIT_TIMEOUT);
            return false;
        }
    }
}

__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort,
                                          uint32_t *status) {
    return mbar_wait_limit(bar, parity, abort, status, kWaitCycles);
}

// One contiguous global -> shared copy by the TMA unit; completion is counted in bytes on `bar`.
// dst, src 16-byte aligned; bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src_gmem, uint32_t bytes, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void named_barrier(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Programmatic dependent launch.  Both are no-ops in a kernel launched the ordinary way.
//  - let_successor_start: the next kernel on the stream, if launched as a programmatic dependent, may come up
//    once every CTA of this grid has passed this point or exited.
//  - wait_for_predecessor: returns when the preceding kernel has completed and its writes are visible.
// Every kernel launched through launch_pdl passes wait_for_predecessor on all its paths before it touches global
// memory (so that its own completion implies that of everything before it on the stream), and calls
// let_successor_start at its top: a chain of small dependent kernels then pays no launch latency between them.
__device__ __forceinline__ void let_successor_start() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void wait_for_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() {
    let_successor_start();
    wait_for_predecessor();
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Transposing reduction of N per-lane values over an aligned group of W lanes (W a power of two,
// N a multiple of W).  On return v[j], j < N/W, holds the group-wide sum of the original value
// with index j + (N/W) * (lane % W).  N - N/W shuffles instead of N * log2(W).
template <int N, int W>
__device__ __forceinline__ void transpose_reduce(float (&v)[N], int lane_in_group) {
    static_assert(N % W == 0, "value count must be a multiple of the group width");
#pragma unroll
    for (int w = W / 2, n = N / 2; w >= 1; w >>= 1, n >>= 1) {
        const bool up = (lane_in_group & w) != 0;
#pragma unroll
        for (int i = 0; i < n; ++i) {
            const float send = up ? v[i] : v[i + n];
            const float keep = up ? v[i + n] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, w);
        }
    }
}

// Launchers (one per translation unit)
arb_status launch_decode(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages,
                         const void *v_pages, const int32_t *block_table, const int32_t *seq_lens,
                         const int32_t *q_lens, void *out, cudaStream_t stream);
arb_status launch_chunk_fma(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages,
                            const void *v_pages, const int32_t *block_table, const int32_t *seq_lens,
                            const int32_t *q_lens, void *out, int n_lo, int n_hi, int skip_rows,
                            cudaStream_t stream);
bool chunk_mma_supported(const arb_attn_params &p);
bool decode_mma_supported(const arb_attn_params &p);
arb_status launch_decode_mma(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages,
                             const void *v_pages, const int32_t *block_table, const int32_t *seq_lens,
                             const int32_t *q_lens, void *out, cudaStream_t stream);
arb_status launch_chunk_mma(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages,
                            const void *v_pages, const int32_t *block_table, const int32_t *seq_lens,
                            const int32_t *q_lens, void *out, cudaStream_t stream);
arb_status launch_chunk_e4m3(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_codes,
                             const void *v_codes, float k_scale, float v_scale, const int32_t *block_table,
                             const int32_t *seq_lens, const int32_t *q_lens, void *out, cudaStream_t stream);
arb_status launch_route(Ctx *ctx, int dtype, int n_steps, int hidden_dim, const void *hidden, const void *w,
                        float b, float tau, float *scores, uint8_t *decisions, cudaStream_t stream);
arb_status launch_rollback(Ctx *ctx, int batch, int32_t *seq_lens, const int32_t *step_lens,
                           const uint8_t *decisions, cudaStream_t stream);
arb_status launch_decode_static(const arb_attn_params &p, const void *q, const void *k_pages, const void *v_pages,
                                const int32_t *block_table, const int32_t *seq_lens, const int32_t *q_lens,
                                void *out, uint32_t *device_status, cudaStream_t stream);
arb_status launch_phase_lens(Ctx *ctx, int batch, const int32_t *step_lens, const uint8_t *decisions, int want, int t,
                             int32_t *out, cudaStream_t stream);
arb_status launch_phase_lens_tokens(Ctx *ctx, int batch, const int32_t *step_lens, const uint8_t *decisions, int want,
                                    int n_tokens, int32_t *out, cudaStream_t stream);
arb_status launch_spearman(Ctx *ctx, int n, const float *x, const float *y, double *rho, cudaStream_t stream);
arb_status launch_policy(Ctx *ctx, int kind, int n_steps, const float *s_d, const float *s_t, float tau, int budget,
                         uint8_t *decisions, arb_policy_stats *stats, cudaStream_t stream);
arb_status launch_route_classes(Ctx *ctx, int dtype, int mode, int n_steps, int hidden_dim, int n_classes,
                                const void *hidden, const void *w, const float *b_host, float tau, float *probs,
                                float *scores, uint8_t *decisions, cudaStream_t stream);
arb_status launch_kv_append(Ctx *ctx, const arb_attn_params &p, int total_new, const void *k_new, const void *v_new,
                            const int32_t *block_table, int32_t *seq_lens, const int32_t *new_lens, int update_lens,
                            void *k_pages, void *v_pages, cudaStream_t stream);
arb_status launch_kv_append_e4m3(Ctx *ctx, const arb_attn_params &p, int total_new, const void *k_new,
                                 const void *v_new, float k_inv_scale, float v_inv_scale, const int32_t *block_table,
                                 int32_t *seq_lens, const int32_t *new_lens, int update_lens, void *k_codes,
                                 void *v_codes, cudaStream_t stream);
arb_status launch_decode_e4m3(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_pages,
                              const void *v_pages, float k_scale, float v_scale, const int32_t *block_table,
                              const int32_t *seq_lens, const int32_t *q_lens, void *out, cudaStream_t stream);
arb_status launch_kv_append_i4(Ctx *ctx, const arb_attn_params &p, int total_new, const void *k_new, const void *v_new,
                               const int32_t *block_table, int32_t *seq_lens, const int32_t *new_lens, int update_lens,
                               void *k_codes, void *v_codes, float *k_scales, float *v_scales, cudaStream_t stream);
bool decode_step_supported(const arb_attn_params &p);
size_t decode_step_hint_bytes(int num_sms);
arb_status launch_decode_step(Ctx *ctx, const arb_attn_params &p, const void *q, const void *k_new, const void *v_new,
                              void *k_pages, void *v_pages, const float *scales, const int32_t *block_table,
                              int32_t *seq_lens, const int32_t *q_lens, void *out, cudaStream_t stream,
                              float *k_row_scales = nullptr, float *v_row_scales = nullptr);
arb_status launch_guard_count(Ctx *ctx, const unsigned char *const *zones, int n_zones, size_t zone_bytes,
                              unsigned long long *bad_dev, cudaStream_t stream);
arb_status launch_selftest_wait(Ctx *ctx, long long limit_cycles, int32_t *report, cudaStream_t stream);
size_t decode_workspace_bytes(const arb_attn_params &p, int num_sms);
int decode_grid(int num_sms);

}  // namespace arb

// C ABI of the arb library: argument validation, context and dispatch.  No arithmetic here.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>

#include "arb_tma.cuh"

using namespace arb;

namespace {

constexpr size_t kDefaultWorkspace = 48ull << 20;
constexpr int kCounters = 1 << 16;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

arb_status check_params(const arb_attn_params *p) {
    if (p == nullptr) return ARB_ERR_INVALID_ARG;
    if (p->batch < 1 || p->num_q_heads < 1 || p->num_kv_heads < 1 || p->num_pages < 1 || p->max_pages_per_seq < 1 ||
        p->total_q < 0 || p->max_q_len < 0)
        return ARB_ERR_INVALID_ARG;
    if (p->num_q_heads % p->num_kv_heads != 0) return ARB_ERR_INVALID_ARG;
    if (p->dtype != ARB_F32 && p->dtype != ARB_BF16) return ARB_ERR_UNSUPPORTED;
    if (p->head_dim != 64 && p->head_dim != 128) return ARB_ERR_UNSUPPORTED;
    if (p->page_size != kPage) return ARB_ERR_UNSUPPORTED;
    if (p->num_q_heads / p->num_kv_heads > kMaxGroup) return ARB_ERR_UNSUPPORTED;
    if (p->batch > kMaxBatch) return ARB_ERR_UNSUPPORTED;
    if ((long long)p->batch * p->num_kv_heads > kCounters) return ARB_ERR_UNSUPPORTED;
    if ((long long)p->max_pages_per_seq * kPage > (1ll << 30)) return ARB_ERR_UNSUPPORTED;
    if (p->flags & ~(uint32_t)(ARB_ATTN_OVERLAP_PREVIOUS | ARB_ATTN_NO_TENSOR_CORES)) return ARB_ERR_INVALID_ARG;
    return ARB_OK;
}

// Device allocations of a ctx.  In the bounds-check build each lies between two guard zones of kGuardBytes filled
// with kGuardPattern (kGuardBytes is 0 in the ordinary build and these are plain cudaMalloc / cudaFree).
template <typename T>
bool guarded_malloc(Ctx *c, T **ptr, size_t bytes) {
    const size_t body = (bytes + 255) & ~size_t(255);
    char *raw = nullptr;
    if (cudaMalloc(&raw, body + 2 * kGuardBytes) != cudaSuccess) return false;
    if (kGuardBytes > 0) {
        if (cudaMemset(raw, kGuardPattern, kGuardBytes) != cudaSuccess ||
            cudaMemset(raw + kGuardBytes + body, kGuardPattern, kGuardBytes) != cudaSuccess || c->n_guards + 2 > 16) {
            cudaFree(raw);
            return false;
        }
        c->guards[c->n_guards++] = reinterpret_cast<unsigned char *>(raw);
        c->guards[c->n_guards++] = reinterpret_cast<unsigned char *>(raw + kGuardBytes + body);
    }
    *ptr = reinterpret_cast<T *>(raw + kGuardBytes);
    return true;
}

void guarded_free(void *p) {
    if (p != nullptr) cudaFree(static_cast<char *>(p) - kGuardBytes);
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        ok = cudaGetDevice(&prev) == cudaSuccess;
        if (ok && prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

}  // namespace

namespace {

bool pipe_setup(Ctx *c) {
    if (c->pipe_ready) return true;
    bool ok = cudaStreamCreateWithFlags(&c->in_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->out_stream, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < kHostSlots; ++i) {
        HostSlot &h = c->slots[i];
        ok = cudaEventCreateWithFlags(&h.in_done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&h.kernels_done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&h.out_done, cudaEventDisableTiming) == cudaSuccess;
    }
    if (!ok) cudaGetLastError();
    c->pipe_ready = ok;
    return ok;
}

// Waits until the call in slot `h` has delivered its result; the slot becomes free.
arb_status slot_wait(HostSlot &h) {
    if (!h.busy) return ARB_OK;
    h.busy = false;
    if (cudaEventSynchronize(h.out_done) != cudaSuccess) {
        cudaGetLastError();
        return ARB_ERR_CUDA;
    }
    return ARB_OK;
}

// Waits for every call in flight; the slots become free.
arb_status pipe_drain(Ctx *c) {
    arb_status st = ARB_OK;
    for (int i = 0; i < kHostSlots; ++i)
        if (slot_wait(c->slots[i]) != ARB_OK) st = ARB_ERR_CUDA;
    return st;
}

void pipe_teardown(Ctx *c) {
    if (c->pipe_ready) pipe_drain(c);
    for (int i = 0; i < kHostSlots; ++i) {
        HostSlot &h = c->slots[i];
        if (h.in_done) cudaEventDestroy(h.in_done);
        if (h.kernels_done) cudaEventDestroy(h.kernels_done);
        if (h.out_done) cudaEventDestroy(h.out_done);
        cudaFree(h.dev);
        cudaFreeHost(h.host);
    }
    if (c->in_stream) cudaStreamDestroy(c->in_stream);
    if (c->out_stream) cudaStreamDestroy(c->out_stream);
}

}  // namespace

extern "C" {

arb_status arb_create(arb_ctx **out, int device, size_t workspace_bytes) {
    if (out == nullptr || device < 0) return ARB_ERR_INVALID_ARG;
    *out = nullptr;
    DeviceGuard guard(device);
    if (!guard.ok) return ARB_ERR_CUDA;
    Ctx *c = new (std::nothrow) Ctx();
    if (c == nullptr) return ARB_ERR_CUDA;
    c->device = device;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1) {
        delete c;
        return ARB_ERR_CUDA;
    }
    c->num_sms = sms;
    // tuning knob of the single-launch decode (see Plan in arb_decode_step.cu)
    if (const char *mc = std::getenv("ARB_STEP_MIN_CHUNK")) c->step_min_chunk = std::max(1, std::min(1024, std::atoi(mc)));
    if (const char *pct = std::getenv("ARB_STEP_BOUNDARY_PCT")) c->step_boundary_pct = std::max(0, std::min(400, std::atoi(pct)));
    c->workspace_bytes = workspace_bytes ? workspace_bytes : kDefaultWorkspace;
    c->counters_len = kCounters;
    bool ok = guarded_malloc(c, &c->workspace, c->workspace_bytes);
    ok = ok && guarded_malloc(c, &c->counters, sizeof(int) * (c->counters_len + 4));
    ok = ok && cudaMemset(c->counters, 0, sizeof(int) * (c->counters_len + 4)) == cudaSuccess;
    const size_t rot_ints = (size_t)kRotSets * kRotCounters + kRotSets + 8;
    ok = ok && guarded_malloc(c, &c->rot, sizeof(int) * rot_ints);
    ok = ok && cudaMemset(c->rot, 0, sizeof(int) * rot_ints) == cudaSuccess;
    ok = ok && guarded_malloc(c, &c->spearman_acc, 4 * sizeof(double));
    c->chunk_ws_bytes = 2 * c->workspace_bytes;   // partials of long step chunks that are split over their keys
    ok = ok && guarded_malloc(c, &c->chunk_ws, c->chunk_ws_bytes);
    ok = ok && guarded_malloc(c, &c->step_hint, decode_step_hint_bytes(sms));
    ok = ok && cudaMemset(c->step_hint, 0, decode_step_hint_bytes(sms)) == cudaSuccess;
    if (ok && c->n_guards > 0) {
        ok = cudaMalloc(&c->guards_dev, sizeof(c->guards)) == cudaSuccess &&
             cudaMalloc(&c->guard_bad, sizeof(unsigned long long)) == cudaSuccess &&
             cudaMemcpy(c->guards_dev, c->guards, sizeof(c->guards), cudaMemcpyHostToDevice) == cudaSuccess;
    }
    if (ok) {  // "everything before the first call has completed"
        const uint32_t done = c->decode_gen - 1;
        ok = cudaMemcpy(c->rot + (size_t)kRotSets * kRotCounters + kRotSets, &done, sizeof(done),
                        cudaMemcpyHostToDevice) == cudaSuccess;
    }
    if (!ok) {
        guarded_free(c->workspace);
        guarded_free(c->counters);
        guarded_free(c->rot);
        guarded_free(c->spearman_acc);
        guarded_free(c->chunk_ws);
        guarded_free(c->step_hint);
        cudaFree(c->guards_dev);
        cudaFree(c->guard_bad);
        delete c;
        cudaGetLastError();
        return ARB_ERR_CUDA;
    }
    c->status = reinterpret_cast<uint32_t *>(c->counters + c->counters_len);
    *out = reinterpret_cast<arb_ctx *>(c);
    return ARB_OK;
}

arb_status arb_destroy(arb_ctx *ctx) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    DeviceGuard guard(c->device);
    guarded_free(c->workspace);
    guarded_free(c->counters);
    guarded_free(c->rot);
    guarded_free(c->spearman_acc);
    guarded_free(c->chunk_ws);
    guarded_free(c->step_hint);
    cudaFree(c->guards_dev);
    cudaFree(c->guard_bad);
    cudaFree(c->stage);
    cudaFreeHost(c->host_stage);
    pipe_teardown(c);
    pool_map_cache_free(c);
    delete c;
    return ARB_OK;
}

size_t arb_attn_workspace_bytes(const arb_attn_params *params) {
    if (check_params(params) != ARB_OK) return 0;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaGetLastError();
    if (sms < 148) sms = 148;
    return decode_workspace_bytes(*params, sms);
}

arb_status arb_attn(arb_ctx *ctx, const arb_attn_params *params, const void *q, const void *k_pages,
                    const void *v_pages, const int32_t *block_table, const int32_t *seq_lens,
                    const int32_t *q_lens, void *out, arb_stream_t stream) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    arb_status st = check_params(params);
    if (st != ARB_OK) return st;
    if (!k_pages || !v_pages || !block_table || !seq_lens || !q_lens) return ARB_ERR_INVALID_ARG;
    if (params->total_q == 0 || params->max_q_len == 0) return ARB_OK;  // nothing to do
    if (!q || !out) return ARB_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(k_pages) || !aligned16(v_pages)) return ARB_ERR_INVALID_ARG;
    if (params->max_q_len > params->total_q) return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (decode_workspace_bytes(*params, c->num_sms) > c->workspace_bytes) return ARB_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

    // q_len == 1 rows: the split-KV decode kernel.  It is launched whenever decode rows may exist
    // (the host knows only the total and the maximum of q_lens).
    const bool maybe_decode = params->max_q_len == 1 || params->total_q > params->max_q_len;
    const bool tensor_cores = (params->flags & ARB_ATTN_NO_TENSOR_CORES) == 0;
    if (maybe_decode) {
        // bf16 / head_dim 128: a call that is one of a back-to-back series (ARB_ATTN_OVERLAP_PREVIOUS) takes the
        // two-kernel form, whose calls stream under one another's tails; a call on its own takes the single
        // launch, which is what finishes a lone call soonest.
        const bool series = (params->flags & ARB_ATTN_OVERLAP_PREVIOUS) != 0;
        if (tensor_cores && !series && decode_step_supported(*params))
            st = launch_decode_step(c, *params, q, nullptr, nullptr, const_cast<void *>(k_pages),
                                    const_cast<void *>(v_pages), nullptr, block_table, const_cast<int32_t *>(seq_lens), q_lens, out, s);
        else if (tensor_cores && decode_mma_supported(*params))
            st = launch_decode_mma(c, *params, q, k_pages, v_pages, block_table, seq_lens, q_lens, out, s);
        else {
            note_unnumbered_decode(c, decode_workspace_bytes(*params, c->num_sms));  // region 0, no generation number
            st = launch_decode(c, *params, q, k_pages, v_pages, block_table, seq_lens, q_lens, out, s);
        }
        if (st != ARB_OK) return st;
    }
    if (params->max_q_len >= 2) {
        // Step chunks: bf16 chunks of head_dim 128 go to the tcgen05 kernel (from kChunkMmaMinRows
        // rows on, i.e. all of them); the rest, and every fp32 chunk, to the CUDA-core kernel.  Both
        // kernels decide per sequence on the device.
        int skip_rows = 0;
        if (tensor_cores && chunk_mma_supported(*params)) {
            st = launch_chunk_mma(c, *params, q, k_pages, v_pages, block_table, seq_lens, q_lens, out, s);
            if (st != ARB_OK) return st;
            skip_rows = kChunkMmaMinRows;
        }
        st = launch_chunk_fma(c, *params, q, k_pages, v_pages, block_table, seq_lens, q_lens, out, 2,
                              params->max_q_len, skip_rows, s);
        if (st != ARB_OK) return st;
    }
    return ARB_OK;
}

arb_status arb_decode_step(arb_ctx *ctx, const arb_attn_params *params, const void *q, const void *k_new,
                           const void *v_new, void *k_pages, void *v_pages, const int32_t *block_table,
                           int32_t *seq_lens, const int32_t *q_lens, void *out, arb_stream_t stream) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    arb_status st = check_params(params);
    if (st != ARB_OK) return st;
    if (params->max_q_len != 1 || params->total_q < 0 || params->total_q > params->batch) return ARB_ERR_INVALID_ARG;
    if (params->flags & ARB_ATTN_OVERLAP_PREVIOUS) return ARB_ERR_INVALID_ARG;   // the call writes the cache it reads
    if (!k_pages || !v_pages || !block_table || !seq_lens || !q_lens) return ARB_ERR_INVALID_ARG;
    if (params->total_q == 0) return ARB_OK;
    if (!q || !out || !k_new || !v_new) return ARB_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(k_new) ||
        !aligned16(v_new))
        return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (decode_workspace_bytes(*params, c->num_sms) > c->workspace_bytes) return ARB_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if ((params->flags & ARB_ATTN_NO_TENSOR_CORES) == 0 && decode_step_supported(*params))
        return launch_decode_step(c, *params, q, k_new, v_new, k_pages, v_pages, nullptr, block_table, seq_lens, q_lens, out, s);
    // shapes the single launch does not serve (fp32, head_dim 64): the same step as two launches
    st = launch_kv_append(c, *params, params->total_q, k_new, v_new, block_table, seq_lens, q_lens, 1, k_pages, v_pages, s);
    if (st != ARB_OK) return st;
    note_unnumbered_decode(c, decode_workspace_bytes(*params, c->num_sms));
    return launch_decode(c, *params, q, k_pages, v_pages, block_table, seq_lens, q_lens, out, s);
}

arb_status arb_decode_step_e4m3(arb_ctx *ctx, const arb_attn_params *params, const void *q, const void *k_new,
                                const void *v_new, uint8_t *k_codes, uint8_t *v_codes, float k_scale, float v_scale,
                                float k_inv_scale, float v_inv_scale, const int32_t *block_table, int32_t *seq_lens,
                                const int32_t *q_lens, void *out, arb_stream_t stream) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    arb_status st = check_params(params);
    if (st != ARB_OK) return st;
    if (params->dtype != ARB_BF16 || params->head_dim != 128) return ARB_ERR_UNSUPPORTED;
    if (params->flags & ARB_ATTN_NO_TENSOR_CORES) return ARB_ERR_UNSUPPORTED;
    if (params->max_q_len != 1 || params->total_q < 0 || params->total_q > params->batch) return ARB_ERR_INVALID_ARG;
    if (params->flags & ARB_ATTN_OVERLAP_PREVIOUS) return ARB_ERR_INVALID_ARG;   // the call writes the cache it reads
    if (!(k_scale > 0.f) || !(v_scale > 0.f) || !(k_inv_scale > 0.f) || !(v_inv_scale > 0.f)) return ARB_ERR_INVALID_ARG;
    if (!k_codes || !v_codes || !block_table || !seq_lens || !q_lens) return ARB_ERR_INVALID_ARG;
    if (params->total_q == 0) return ARB_OK;
    if (!q || !out || !k_new || !v_new) return ARB_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(k_codes) || !aligned16(v_codes) || !aligned16(k_new) ||
        !aligned16(v_new))
        return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (decode_workspace_bytes(*params, c->num_sms) > c->workspace_bytes) return ARB_ERR_WORKSPACE;
    if (!decode_step_supported(*params)) return ARB_ERR_UNSUPPORTED;
    const float scales[4] = {k_scale, v_scale, k_inv_scale, v_inv_scale};
    return launch_decode_step(c, *params, q, k_new, v_new, k_codes, v_codes, scales, block_table, seq_lens, q_lens, out,
                              reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_decode_step_i4(arb_ctx *ctx, const arb_attn_params *params, const void *q, const void *k_new,
                              const void *v_new, uint8_t *k_codes, uint8_t *v_codes, float *k_scales, float *v_scales,
                              const int32_t *block_table, int32_t *seq_lens, const int32_t *q_lens, void *out,
                              arb_stream_t stream) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    arb_status st = check_params(params);
    if (st != ARB_OK) return st;
    if (params->dtype != ARB_BF16 || params->head_dim != 128) return ARB_ERR_UNSUPPORTED;
    if (params->flags & ARB_ATTN_NO_TENSOR_CORES) return ARB_ERR_UNSUPPORTED;
    if (params->max_q_len != 1 || params->total_q < 0 || params->total_q > params->batch) return ARB_ERR_INVALID_ARG;
    if (params->flags & ARB_ATTN_OVERLAP_PREVIOUS) return ARB_ERR_INVALID_ARG;   // the call writes the cache it reads
    if (!k_codes || !v_codes || !k_scales || !v_scales || !block_table || !seq_lens || !q_lens) return ARB_ERR_INVALID_ARG;
    if (params->total_q == 0) return ARB_OK;
    if (!q || !out || !k_new || !v_new) return ARB_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(k_codes) || !aligned16(v_codes) || !aligned16(k_new) ||
        !aligned16(v_new) || !aligned16(k_scales) || !aligned16(v_scales))
        return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (decode_workspace_bytes(*params, c->num_sms) > c->workspace_bytes) return ARB_ERR_WORKSPACE;
    if (!decode_step_supported(*params)) return ARB_ERR_UNSUPPORTED;
    return launch_decode_step(c, *params, q, k_new, v_new, k_codes, v_codes, nullptr, block_table, seq_lens, q_lens, out,
                              reinterpret_cast<cudaStream_t>(stream), k_scales, v_scales);
}

arb_status arb_attn_decode_static(const arb_attn_params *params, const void *q, const void *k_pages,
                                  const void *v_pages, const int32_t *block_table, const int32_t *seq_lens,
                                  const int32_t *q_lens, void *out, uint32_t *device_status, arb_stream_t stream) {
    arb_status st = check_params(params);
    if (st != ARB_OK) return st;
    if (params->max_q_len != 1 || params->total_q < 1 || params->total_q > params->batch) return ARB_ERR_INVALID_ARG;
    if (params->flags & ARB_ATTN_OVERLAP_PREVIOUS) return ARB_ERR_INVALID_ARG;  // calls share one scratch array
    if (!q || !out || !k_pages || !v_pages || !block_table || !seq_lens || !q_lens) return ARB_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(k_pages) || !aligned16(v_pages)) return ARB_ERR_INVALID_ARG;
    return launch_decode_static(*params, q, k_pages, v_pages, block_table, seq_lens, q_lens, out, device_status,
                                reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_attn_host(arb_ctx *ctx, const arb_attn_params *params, const void *q_host, const void *k_pages,
                         const void *v_pages, const int32_t *block_table_host, const int32_t *seq_lens_host,
                         const int32_t *q_lens_host, void *out_host, arb_stream_t stream) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    arb_status st = check_params(params);
    if (st != ARB_OK) return st;
    if (!q_host || !out_host || !block_table_host || !seq_lens_host || !q_lens_host) return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    DeviceGuard guard(c->device);
    if (!guard.ok) return ARB_ERR_CUDA;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t esz = params->dtype == ARB_BF16 ? 2 : 4;
    auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
    const size_t q_bytes = (size_t)params->total_q * params->num_q_heads * params->head_dim * esz;
    const size_t bt_bytes = sizeof(int32_t) * (size_t)params->batch * params->max_pages_per_seq;
    const size_t len_bytes = sizeof(int32_t) * (size_t)params->batch;
    const size_t need = 2 * up(q_bytes) + up(bt_bytes) + 2 * up(len_bytes);
    if (need > c->stage_bytes) {
        if (cudaStreamSynchronize(s) != cudaSuccess) return ARB_ERR_CUDA;
        cudaFree(c->stage);
        c->stage = nullptr;
        c->stage_bytes = 0;
        if (cudaMalloc(&c->stage, need) != cudaSuccess) {
            cudaGetLastError();
            return ARB_ERR_CUDA;
        }
        c->stage_bytes = need;
    }
    // device staging: [out | q | block table | seq_lens | q_lens]; the four inputs are gathered in a page-locked host
    // block of the same layout first, so that they cross the bus as one copy instead of four
    char *dout = c->stage, *dq = dout + up(q_bytes), *dbt = dq + up(q_bytes);
    char *dsl = dbt + up(bt_bytes), *dql = dsl + up(len_bytes);
    const size_t in_bytes = need - up(q_bytes);
    if (in_bytes > c->host_stage_bytes) {
        if (cudaStreamSynchronize(s) != cudaSuccess) return ARB_ERR_CUDA;
        cudaFreeHost(c->host_stage);
        c->host_stage = nullptr;
        c->host_stage_bytes = 0;
        if (cudaHostAlloc(&c->host_stage, in_bytes, cudaHostAllocDefault) != cudaSuccess) {
            cudaGetLastError();
            return ARB_ERR_CUDA;
        }
        c->host_stage_bytes = in_bytes;
    }
    char *hq = c->host_stage, *hbt = hq + up(q_bytes), *hsl = hbt + up(bt_bytes), *hql = hsl + up(len_bytes);
    memcpy(hq, q_host, q_bytes);
    memcpy(hbt, block_table_host, bt_bytes);
    memcpy(hsl, seq_lens_host, len_bytes);
    memcpy(hql, q_lens_host, len_bytes);
    if (cudaMemcpyAsync(dq, hq, in_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return ARB_ERR_CUDA;
    // a page-locked result buffer is written by the kernels themselves, row by row over the bus (posted
    // writes: nothing waits for them but the final synchronisation), which saves the copy back
    void *mapped_out = nullptr;
    if (!aligned16(out_host) || cudaHostGetDevicePointer(&mapped_out, out_host, 0) != cudaSuccess) {
        cudaGetLastError();
        mapped_out = nullptr;
    }
    st = arb_attn(ctx, params, dq, k_pages, v_pages, reinterpret_cast<int32_t *>(dbt),
                  reinterpret_cast<int32_t *>(dsl), reinterpret_cast<int32_t *>(dql), mapped_out ? mapped_out : dout,
                  stream);
    if (st != ARB_OK) return st;
    if (!mapped_out && cudaMemcpyAsync(out_host, dout, q_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return ARB_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return ARB_ERR_CUDA;
    return ARB_OK;
}

arb_status arb_attn_host_begin(arb_ctx *ctx, const arb_attn_params *params, const void *q_host, const void *k_pages,
                               const void *v_pages, const int32_t *block_table_host, const int32_t *seq_lens_host,
                               const int32_t *q_lens_host, void *out_host, arb_stream_t stream) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    arb_status st = check_params(params);
    if (st != ARB_OK) return st;
    if (!q_host || !out_host || !block_table_host || !seq_lens_host || !q_lens_host) return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    DeviceGuard guard(c->device);
    if (!guard.ok) return ARB_ERR_CUDA;
    if (!pipe_setup(c)) return ARB_ERR_CUDA;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t esz = params->dtype == ARB_BF16 ? 2 : 4;
    auto up = [](size_t x) { return (x + 255) & ~size_t(255); };
    const size_t q_bytes = (size_t)params->total_q * params->num_q_heads * params->head_dim * esz;
    const size_t bt_bytes = sizeof(int32_t) * (size_t)params->batch * params->max_pages_per_seq;
    const size_t len_bytes = sizeof(int32_t) * (size_t)params->batch;
    const size_t in_bytes = up(q_bytes) + up(bt_bytes) + 2 * up(len_bytes);
    const size_t need = up(q_bytes) + in_bytes;

    HostSlot &h = c->slots[c->next_slot];
    if (slot_wait(h) != ARB_OK) return ARB_ERR_CUDA;   // the ring is full: the oldest call has to finish first
    if (in_bytes > h.host_bytes) {
        cudaFreeHost(h.host);
        h.host = nullptr;
        h.host_bytes = 0;
        if (cudaHostAlloc(&h.host, in_bytes, cudaHostAllocDefault) != cudaSuccess) {
            cudaGetLastError();
            return ARB_ERR_CUDA;
        }
        h.host_bytes = in_bytes;
    }
    char *hq = h.host, *hbt = hq + up(q_bytes), *hsl = hbt + up(bt_bytes), *hql = hsl + up(len_bytes);
    memcpy(hq, q_host, q_bytes);
    memcpy(hbt, block_table_host, bt_bytes);
    memcpy(hsl, seq_lens_host, len_bytes);
    memcpy(hql, q_lens_host, len_bytes);
    // A call flagged ARB_ATTN_OVERLAP_PREVIOUS whose out_host is page-locked (and so mapped into the device's
    // address space) moves its operands itself: the kernels read the slot's page-locked copy of the inputs over
    // the bus and write the rows of out straight into out_host; no copy is enqueued, only the event that marks
    // the call complete.  Measured on the draft-shaped batch (34 MB of KV per call): 17 us per call against 24
    // with the copies below and unflagged kernels.  It pays for flagged calls only: every CTA reads lengths,
    // block-table entries and q rows over the bus in small requests, and an unflagged small call has twice the
    // CTAs (41 us per call).
    void *mapped_out = nullptr;
    if (!aligned16(out_host) || cudaHostGetDevicePointer(&mapped_out, out_host, 0) != cudaSuccess) {
        cudaGetLastError();   // out_host is ordinary memory
        mapped_out = nullptr;
    }
    if ((params->flags & ARB_ATTN_OVERLAP_PREVIOUS) && mapped_out) {
        void *mapped_in = nullptr;
        if (cudaHostGetDevicePointer(&mapped_in, h.host, 0) == cudaSuccess) {
            char *mq = static_cast<char *>(mapped_in), *mbt = mq + up(q_bytes);
            char *msl = mbt + up(bt_bytes), *mql = msl + up(len_bytes);
            st = arb_attn(ctx, params, mq, k_pages, v_pages, reinterpret_cast<int32_t *>(mbt),
                          reinterpret_cast<int32_t *>(msl), reinterpret_cast<int32_t *>(mql), mapped_out, stream);
            if (st != ARB_OK) {  // a part of the call may be in flight: the slot is not marked busy, so wait here
                cudaStreamSynchronize(s);
                cudaGetLastError();
                return st;
            }
            if (cudaEventRecord(h.out_done, s) != cudaSuccess) {
                cudaStreamSynchronize(s);
                cudaGetLastError();
                return ARB_ERR_CUDA;
            }
            h.busy = true;
            c->next_slot = (c->next_slot + 1) % kHostSlots;
            return ARB_OK;
        }
        cudaGetLastError();
    }
    if (need > h.dev_bytes) {  // the slot is idle, so nothing on the device still uses its buffers
        cudaFree(h.dev);
        h.dev = nullptr;
        h.dev_bytes = 0;
        if (cudaMalloc(&h.dev, need) != cudaSuccess) {
            cudaGetLastError();
            return ARB_ERR_CUDA;
        }
        h.dev_bytes = need;
    }
    char *dout = h.dev, *dq = dout + up(q_bytes), *dbt = dq + up(q_bytes);
    char *dsl = dbt + up(bt_bytes), *dql = dsl + up(len_bytes);
    // inputs in on one copy stream, kernels on the caller's stream, result out on the other copy stream:
    // the copies of neighbouring calls run beside the kernels instead of between them
    if (cudaMemcpyAsync(dq, hq, in_bytes, cudaMemcpyHostToDevice, c->in_stream) != cudaSuccess ||
        cudaEventRecord(h.in_done, c->in_stream) != cudaSuccess) {
        cudaStreamSynchronize(c->in_stream);
        cudaGetLastError();
        return ARB_ERR_CUDA;
    }
    if (cudaStreamWaitEvent(s, h.in_done, 0) == cudaSuccess)
        st = arb_attn(ctx, params, dq, k_pages, v_pages, reinterpret_cast<int32_t *>(dbt),
                      reinterpret_cast<int32_t *>(dsl), reinterpret_cast<int32_t *>(dql), dout, stream);
    else
        st = ARB_ERR_CUDA;
    if (st != ARB_OK) {  // nothing of this call may stay in flight on a slot that is not marked busy
        cudaStreamSynchronize(c->in_stream);
        cudaStreamSynchronize(s);
        cudaGetLastError();
        return st;
    }
    // (Letting these kernels write a page-locked out_host themselves was measured and is slower here, 27 against
    // 24 us per call: the writes over the bus have to drain before the kernel counts as complete, and that is on
    // the chain of serialised kernels, while the copy below is beside it.)
    bool ok = cudaEventRecord(h.kernels_done, s) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(c->out_stream, h.kernels_done, 0) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(out_host, dout, q_bytes, cudaMemcpyDeviceToHost, c->out_stream) == cudaSuccess;
    ok = ok && cudaEventRecord(h.out_done, c->out_stream) == cudaSuccess;
    if (!ok) {
        cudaStreamSynchronize(s);
        cudaStreamSynchronize(c->out_stream);
        cudaGetLastError();
        return ARB_ERR_CUDA;
    }
    h.busy = true;
    c->next_slot = (c->next_slot + 1) % kHostSlots;
    return ARB_OK;
}

arb_status arb_attn_host_wait(arb_ctx *ctx) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    DeviceGuard guard(c->device);
    if (!guard.ok) return ARB_ERR_CUDA;
    return pipe_drain(c);
}

arb_status arb_route(arb_ctx *ctx, int32_t dtype, int32_t n_steps, int32_t hidden_dim, const void *hidden,
                     const void *w, float b, float tau, float *scores, uint8_t *decisions, arb_stream_t stream) {
    if (ctx == nullptr || n_steps < 0 || hidden_dim < 1) return ARB_ERR_INVALID_ARG;
    if (dtype != ARB_F32 && dtype != ARB_BF16) return ARB_ERR_UNSUPPORTED;
    if (hidden_dim % 8 != 0) return ARB_ERR_UNSUPPORTED;
    if (n_steps == 0) return ARB_OK;
    if (!hidden || !w || !scores || !decisions) return ARB_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(w)) return ARB_ERR_INVALID_ARG;
    return launch_route(reinterpret_cast<Ctx *>(ctx), dtype, n_steps, hidden_dim, hidden, w, b, tau, scores,
                        decisions, reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_rollback(arb_ctx *ctx, int32_t batch, int32_t *seq_lens, const int32_t *step_lens,
                        const uint8_t *decisions, arb_stream_t stream) {
    if (ctx == nullptr || batch < 0) return ARB_ERR_INVALID_ARG;
    if (batch == 0) return ARB_OK;
    if (!seq_lens || !step_lens) return ARB_ERR_INVALID_ARG;
    return launch_rollback(reinterpret_cast<Ctx *>(ctx), batch, seq_lens, step_lens, decisions,
                           reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_spearman(arb_ctx *ctx, int32_t n, const float *x, const float *y, double *rho, arb_stream_t stream) {
    if (ctx == nullptr || n < 0 || rho == nullptr) return ARB_ERR_INVALID_ARG;
    if (n > 0 && (!x || !y)) return ARB_ERR_INVALID_ARG;
    if (n > 65536) return ARB_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(rho) & 7u) != 0) return ARB_ERR_INVALID_ARG;
    return launch_spearman(reinterpret_cast<Ctx *>(ctx), n, x, y, rho, reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_phase_lens(arb_ctx *ctx, int32_t batch, const int32_t *step_lens, const uint8_t *decisions, int32_t want,
                          int32_t t, int32_t *out, arb_stream_t stream) {
    if (ctx == nullptr || batch < 0) return ARB_ERR_INVALID_ARG;
    if (batch == 0) return ARB_OK;
    if (!step_lens || !out) return ARB_ERR_INVALID_ARG;
    return launch_phase_lens(reinterpret_cast<Ctx *>(ctx), batch, step_lens, decisions, want, t, out,
                             reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_phase_lens_tokens(arb_ctx *ctx, int32_t batch, const int32_t *step_lens, const uint8_t *decisions,
                                 int32_t want, int32_t n_tokens, int32_t *out, arb_stream_t stream) {
    if (ctx == nullptr || batch < 0 || n_tokens < 0) return ARB_ERR_INVALID_ARG;
    if (batch == 0 || n_tokens == 0) return ARB_OK;
    if (!step_lens || !out) return ARB_ERR_INVALID_ARG;
    if ((long long)batch * n_tokens > (1ll << 30)) return ARB_ERR_UNSUPPORTED;
    return launch_phase_lens_tokens(reinterpret_cast<Ctx *>(ctx), batch, step_lens, decisions, want, n_tokens, out,
                                    reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_policy(arb_ctx *ctx, int32_t kind, int32_t n_steps, const float *s_d, const float *s_t, float tau,
                      int32_t budget, uint8_t *decisions, arb_policy_stats *stats, arb_stream_t stream) {
    if (ctx == nullptr || n_steps < 0) return ARB_ERR_INVALID_ARG;
    if (kind < ARB_POLICY_RSD || kind > ARB_POLICY_ORACLE_BUDGET) return ARB_ERR_INVALID_ARG;
    if (n_steps == 0) return ARB_OK;
    if (!s_d || !decisions) return ARB_ERR_INVALID_ARG;
    if (!s_t && (kind != ARB_POLICY_RSD || stats != nullptr)) return ARB_ERR_INVALID_ARG;
    if (kind == ARB_POLICY_ORACLE_BUDGET && n_steps > 65536) return ARB_ERR_UNSUPPORTED;
    if (stats != nullptr && (reinterpret_cast<uintptr_t>(stats) & 7u) != 0) return ARB_ERR_INVALID_ARG;
    return launch_policy(reinterpret_cast<Ctx *>(ctx), kind, n_steps, s_d, s_t, tau, budget, decisions, stats,
                         reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_route_classes(arb_ctx *ctx, int32_t dtype, int32_t mode, int32_t n_steps, int32_t hidden_dim,
                             int32_t n_classes, const void *hidden, const void *w, const float *b_host, float tau,
                             float *probs, float *scores, uint8_t *decisions, arb_stream_t stream) {
    if (ctx == nullptr || n_steps < 0 || hidden_dim < 1) return ARB_ERR_INVALID_ARG;
    if (dtype != ARB_F32 && dtype != ARB_BF16) return ARB_ERR_UNSUPPORTED;
    if (mode != ARB_HEAD_SOFTMAX && mode != ARB_HEAD_ORDINAL) return ARB_ERR_INVALID_ARG;
    if (n_classes < 2 || n_classes > ARB_MAX_CLASSES || hidden_dim % 8 != 0) return ARB_ERR_UNSUPPORTED;
    if (n_steps == 0) return ARB_OK;
    if (!hidden || !w || !b_host || !scores || !decisions) return ARB_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(w)) return ARB_ERR_INVALID_ARG;
    return launch_route_classes(reinterpret_cast<Ctx *>(ctx), dtype, mode, n_steps, hidden_dim, n_classes, hidden, w,
                                b_host, tau, probs, scores, decisions, reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_kv_append(arb_ctx *ctx, const arb_attn_params *params, int32_t total_new, const void *k_new,
                         const void *v_new, const int32_t *block_table, int32_t *seq_lens, const int32_t *new_lens,
                         int32_t update_lens, void *k_pages, void *v_pages, arb_stream_t stream) {
    if (ctx == nullptr || params == nullptr || total_new < 0) return ARB_ERR_INVALID_ARG;
    if (params->batch < 1 || params->num_kv_heads < 1 || params->num_pages < 1 || params->max_pages_per_seq < 1)
        return ARB_ERR_INVALID_ARG;
    if (params->dtype != ARB_F32 && params->dtype != ARB_BF16) return ARB_ERR_UNSUPPORTED;
    if (params->head_dim != 64 && params->head_dim != 128) return ARB_ERR_UNSUPPORTED;
    if (params->page_size != kPage || params->batch > kMaxBatch) return ARB_ERR_UNSUPPORTED;
    if (!block_table || !seq_lens || !new_lens || !k_pages || !v_pages) return ARB_ERR_INVALID_ARG;
    if (total_new == 0) return ARB_OK;
    if (!k_new || !v_new) return ARB_ERR_INVALID_ARG;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_pages) || !aligned16(v_pages)) return ARB_ERR_INVALID_ARG;
    return launch_kv_append(reinterpret_cast<Ctx *>(ctx), *params, total_new, k_new, v_new, block_table, seq_lens,
                            new_lens, update_lens, k_pages, v_pages, reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_attn_decode_e4m3(arb_ctx *ctx, const arb_attn_params *params, const void *q, const uint8_t *k_codes,
                                const uint8_t *v_codes, float k_scale, float v_scale, const int32_t *block_table,
                                const int32_t *seq_lens, const int32_t *q_lens, void *out, arb_stream_t stream) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    arb_status st = check_params(params);
    if (st != ARB_OK) return st;
    if (params->dtype != ARB_BF16 || params->head_dim != 128) return ARB_ERR_UNSUPPORTED;
    if (params->max_q_len != 1 || params->total_q < 1 || params->total_q > params->batch) return ARB_ERR_INVALID_ARG;
    if (params->flags & ARB_ATTN_NO_TENSOR_CORES) return ARB_ERR_UNSUPPORTED;
    if (!(k_scale > 0.f) || !(v_scale > 0.f)) return ARB_ERR_INVALID_ARG;
    if (!q || !out || !k_codes || !v_codes || !block_table || !seq_lens || !q_lens) return ARB_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(k_codes) || !aligned16(v_codes)) return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (decode_workspace_bytes(*params, c->num_sms) > c->workspace_bytes) return ARB_ERR_WORKSPACE;
    return launch_decode_e4m3(c, *params, q, k_codes, v_codes, k_scale, v_scale, block_table, seq_lens, q_lens, out,
                              reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_attn_e4m3(arb_ctx *ctx, const arb_attn_params *params, const void *q, const uint8_t *k_codes,
                         const uint8_t *v_codes, float k_scale, float v_scale, const int32_t *block_table,
                         const int32_t *seq_lens, const int32_t *q_lens, void *out, arb_stream_t stream) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    arb_status st = check_params(params);
    if (st != ARB_OK) return st;
    if (params->dtype != ARB_BF16 || params->head_dim != 128) return ARB_ERR_UNSUPPORTED;
    if (params->flags & ARB_ATTN_NO_TENSOR_CORES) return ARB_ERR_UNSUPPORTED;
    if (!(k_scale > 0.f) || !(v_scale > 0.f)) return ARB_ERR_INVALID_ARG;
    if (!k_codes || !v_codes || !block_table || !seq_lens || !q_lens) return ARB_ERR_INVALID_ARG;
    if (params->total_q == 0 || params->max_q_len == 0) return ARB_OK;
    if (!q || !out) return ARB_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || !aligned16(k_codes) || !aligned16(v_codes)) return ARB_ERR_INVALID_ARG;
    if (params->max_q_len > params->total_q) return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    if (decode_workspace_bytes(*params, c->num_sms) > c->workspace_bytes) return ARB_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const bool maybe_decode = params->max_q_len == 1 || params->total_q > params->max_q_len;
    if (maybe_decode) {
        st = launch_decode_e4m3(c, *params, q, k_codes, v_codes, k_scale, v_scale, block_table, seq_lens, q_lens, out, s);
        if (st != ARB_OK) return st;
    }
    if (params->max_q_len >= 2) {
        st = launch_chunk_e4m3(c, *params, q, k_codes, v_codes, k_scale, v_scale, block_table, seq_lens, q_lens, out, s);
        if (st != ARB_OK) return st;
        // the CUDA-core chunk kernel reads no key here: every chunk of valid lengths has gone to the tensor cores; it
        // zero-fills the rows of sequences whose lengths are not (status bit) and otherwise leaves at once
        st = launch_chunk_fma(c, *params, q, k_codes, v_codes, block_table, seq_lens, q_lens, out, 2, params->max_q_len,
                              kChunkMmaMinRows, s);
        if (st != ARB_OK) return st;
    }
    return ARB_OK;
}

arb_status arb_kv_append_e4m3(arb_ctx *ctx, const arb_attn_params *params, int32_t total_new, const void *k_new,
                              const void *v_new, float k_inv_scale, float v_inv_scale, const int32_t *block_table,
                              int32_t *seq_lens, const int32_t *new_lens, int32_t update_lens, uint8_t *k_codes,
                              uint8_t *v_codes, arb_stream_t stream) {
    if (ctx == nullptr || params == nullptr || total_new < 0) return ARB_ERR_INVALID_ARG;
    if (params->batch < 1 || params->num_kv_heads < 1 || params->num_pages < 1 || params->max_pages_per_seq < 1)
        return ARB_ERR_INVALID_ARG;
    if (params->dtype != ARB_F32 && params->dtype != ARB_BF16) return ARB_ERR_UNSUPPORTED;
    if (params->head_dim != 64 && params->head_dim != 128) return ARB_ERR_UNSUPPORTED;
    if (params->page_size != kPage || params->batch > kMaxBatch) return ARB_ERR_UNSUPPORTED;
    if (!(k_inv_scale > 0.f) || !(v_inv_scale > 0.f)) return ARB_ERR_INVALID_ARG;
    if (!block_table || !seq_lens || !new_lens || !k_codes || !v_codes) return ARB_ERR_INVALID_ARG;
    if (total_new == 0) return ARB_OK;
    if (!k_new || !v_new) return ARB_ERR_INVALID_ARG;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_codes) || !aligned16(v_codes)) return ARB_ERR_INVALID_ARG;
    return launch_kv_append_e4m3(reinterpret_cast<Ctx *>(ctx), *params, total_new, k_new, v_new, k_inv_scale, v_inv_scale,
                                 block_table, seq_lens, new_lens, update_lens, k_codes, v_codes,
                                 reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_kv_append_i4(arb_ctx *ctx, const arb_attn_params *params, int32_t total_new, const void *k_new,
                            const void *v_new, const int32_t *block_table, int32_t *seq_lens, const int32_t *new_lens,
                            int32_t update_lens, uint8_t *k_codes, uint8_t *v_codes, float *k_scales, float *v_scales,
                            arb_stream_t stream) {
    if (ctx == nullptr || params == nullptr || total_new < 0) return ARB_ERR_INVALID_ARG;
    if (params->batch < 1 || params->num_kv_heads < 1 || params->num_pages < 1 || params->max_pages_per_seq < 1)
        return ARB_ERR_INVALID_ARG;
    if (params->dtype != ARB_BF16 || params->head_dim != 128) return ARB_ERR_UNSUPPORTED;
    if (params->page_size != kPage || params->batch > kMaxBatch) return ARB_ERR_UNSUPPORTED;
    if (!block_table || !seq_lens || !new_lens || !k_codes || !v_codes || !k_scales || !v_scales) return ARB_ERR_INVALID_ARG;
    if (total_new == 0) return ARB_OK;
    if (!k_new || !v_new) return ARB_ERR_INVALID_ARG;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_codes) || !aligned16(v_codes) || !aligned16(k_scales) ||
        !aligned16(v_scales))
        return ARB_ERR_INVALID_ARG;
    return launch_kv_append_i4(reinterpret_cast<Ctx *>(ctx), *params, total_new, k_new, v_new, block_table, seq_lens,
                               new_lens, update_lens, k_codes, v_codes, k_scales, v_scales,
                               reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_poll_status(arb_ctx *ctx, arb_stream_t stream, uint32_t *bits) {
    if (ctx == nullptr) return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    uint32_t host = 0;
    if (cudaMemcpyAsync(&host, c->status, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess) return ARB_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return ARB_ERR_CUDA;
    if (bits) *bits = host;
    if (host != 0) {  // a kernel that gave up may have left arrival counters behind
        if (cudaMemsetAsync(c->counters, 0, sizeof(int) * (c->counters_len + 4), s) != cudaSuccess) return ARB_ERR_CUDA;
        if (cudaMemsetAsync(c->rot, 0, sizeof(int) * ((size_t)kRotSets * kRotCounters + kRotSets), s) != cudaSuccess)
            return ARB_ERR_CUDA;
        if (cudaStreamSynchronize(s) != cudaSuccess) return ARB_ERR_CUDA;
        return ARB_ERR_DEVICE_STATUS;
    }
    return ARB_OK;
}

arb_status arb_selftest_wait_timeout(arb_ctx *ctx, int64_t limit_cycles, int32_t *report, arb_stream_t stream) {
    if (ctx == nullptr || report == nullptr) return ARB_ERR_INVALID_ARG;
    if (limit_cycles < 1 || limit_cycles > (1ll << 31)) return ARB_ERR_INVALID_ARG;   // at most about a second
    return launch_selftest_wait(reinterpret_cast<Ctx *>(ctx), limit_cycles, report, reinterpret_cast<cudaStream_t>(stream));
}

arb_status arb_selftest_guard_zones(arb_ctx *ctx, arb_stream_t stream, int64_t *bad, int64_t *checked) {
    if (ctx == nullptr || bad == nullptr) return ARB_ERR_INVALID_ARG;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    *bad = 0;
    if (checked) *checked = (int64_t)c->n_guards * (int64_t)kGuardBytes;
    if (c->n_guards == 0) return cudaStreamSynchronize(s) == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
    unsigned long long host = 0;
    if (cudaMemsetAsync(c->guard_bad, 0, sizeof(unsigned long long), s) != cudaSuccess) return ARB_ERR_CUDA;
    const arb_status st = launch_guard_count(c, c->guards_dev, c->n_guards, kGuardBytes, c->guard_bad, s);
    if (st != ARB_OK) return st;
    if (cudaMemcpyAsync(&host, c->guard_bad, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess) return ARB_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return ARB_ERR_CUDA;
    *bad = (int64_t)host;
    return ARB_OK;
}

#ifdef ARB_CHECKS
// Bounds-check build only, for the test of the guard check itself: overwrites the last `nbytes` bytes of the guard
// zone in front of the workspace (memory this ctx owns), as a store just below the buffer would.
int arb_debug_poke_guard(arb_ctx *ctx, int nbytes) {
    if (ctx == nullptr || nbytes < 1 || (size_t)nbytes > kGuardBytes) return 1;
    Ctx *c = reinterpret_cast<Ctx *>(ctx);
    return cudaMemset(c->workspace - nbytes, 0, (size_t)nbytes) == cudaSuccess ? 0 : 1;
}
#endif

uint64_t arb_launch_count(const arb_ctx *ctx) {
    return ctx ? reinterpret_cast<const Ctx *>(ctx)->launches : 0;
}

const char *arb_status_string(arb_status status) {
    switch (status) {
        case ARB_OK: return "ok";
        case ARB_ERR_INVALID_ARG: return "invalid argument";
        case ARB_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case ARB_ERR_WORKSPACE: return "workspace too small";
        case ARB_ERR_CUDA: return "CUDA runtime error";
        case ARB_ERR_DEVICE_STATUS: return "device status word is non-zero";
        case ARB_ERR_STATIC_LIMIT: return "call exceeds the built-in scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

}  // extern "C"

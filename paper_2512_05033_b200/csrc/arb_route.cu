// Router head with the threshold decision, and step rollback.
//
// Router (Section 4.2 and Algorithm 1 of the paper): score = sigmoid(hidden_last . w + b);
// decision = 1 (escalate to the target) iff score > tau, 0 (accept the draft step) otherwise.
// One warp per step: 16-byte loads of the hidden row and of w, fp32 FMAs, a shuffle reduction, and
// the sigmoid and the comparison in the same kernel.  The whole input is a few hundred KB, so the
// kernel is bound by launch and load latency; several loads are kept in flight per lane.
//
// Rollback: seq_lens[i] -= step_lens[i] where the step was escalated.  No KV bytes move.
#include "arb_common.cuh"

namespace arb {

namespace {

constexpr int kRouteWarps = 4;

template <typename T>
__global__ void __launch_bounds__(kRouteWarps * 32)
route_kernel(const char *__restrict__ hidden, const char *__restrict__ w, int n_steps, int hidden_dim, float b,
             float tau, float *__restrict__ scores, uint8_t *__restrict__ decisions) {
    constexpr int EPL = Elt<T>::kPerVec;
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int step = blockIdx.x * kRouteWarps + (threadIdx.x >> 5);
    if (step >= n_steps) return;
    const int nvec = hidden_dim / EPL;
    const uint4 *hrow = reinterpret_cast<const uint4 *>(hidden + (size_t)step * hidden_dim * sizeof(T));
    const uint4 *wv = reinterpret_cast<const uint4 *>(w);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    int v = lane;
    for (; v + 96 < nvec; v += 128) {  // four independent 16-byte loads of each operand in flight
        uint4 hx[4], wx[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            hx[u] = __ldg(hrow + v + 32 * u);
            wx[u] = __ldg(wv + v + 32 * u);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            float hf[EPL], wf[EPL];
            Elt<T>::unpack(hx[u], hf);
            Elt<T>::unpack(wx[u], wf);
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[u] = fmaf(hf[e], wf[e], acc[u]);
        }
    }
    for (; v < nvec; v += 32) {
        float hf[EPL], wf[EPL];
        Elt<T>::unpack(__ldg(hrow + v), hf);
        Elt<T>::unpack(__ldg(wv + v), wf);
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[0] = fmaf(hf[e], wf[e], acc[0]);
    }
    float z = (acc[0] + acc[1]) + (acc[2] + acc[3]);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
    if (lane == 0) {
        z += b;
        const float score = 1.0f / (1.0f + expf(-z));
        scores[step] = score;
        decisions[step] = score > tau ? 1 : 0;  // a tie accepts the draft step
    }
}

__global__ void rollback_kernel(int batch, int32_t *__restrict__ seq_lens, const int32_t *__restrict__ step_lens,
                                const uint8_t *__restrict__ decisions, uint32_t *status) {
    pdl_enter();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= batch) return;
    if (decisions != nullptr && decisions[i] == 0) return;
    const int L = seq_lens[i], s = step_lens[i];
    if (s < 0) {
        atomicOr(status, (uint32_t)ARB_DEV_ROLLBACK_UNDERFLOW);
        return;
    }
    int r = L - s;
    if (r < 0) {
        atomicOr(status, (uint32_t)ARB_DEV_ROLLBACK_UNDERFLOW);
        r = 0;
    }
    seq_lens[i] = r;
}

// Lengths of the next call of a phase of the step loop (see arb_phase_lens): one thread per sequence.
__global__ void phase_lens_kernel(int batch, const int32_t *__restrict__ step_lens, const uint8_t *__restrict__ decisions,
                                  int want, int t, int32_t *__restrict__ out) {
    pdl_enter();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const int n = max(step_lens[b], 0);
    const bool in = decisions == nullptr || ((decisions[b] != 0) == (want != 0));
    out[b] = !in ? 0 : (t < 0 ? n : (t < n ? 1 : 0));
}

// The same for every token of a step that is decoded token by token: out[t][b], t < n_tokens, in one launch.
__global__ void phase_lens_tokens_kernel(int batch, const int32_t *__restrict__ step_lens,
                                         const uint8_t *__restrict__ decisions, int want, int n_tokens,
                                         int32_t *__restrict__ out) {
    pdl_enter();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= batch * n_tokens) return;
    const int t = i / batch, b = i - t * batch;
    const bool in = decisions == nullptr || ((decisions[b] != 0) == (want != 0));
    out[i] = (in && t < step_lens[b]) ? 1 : 0;
}

}  // namespace

arb_status launch_phase_lens_tokens(Ctx *ctx, int batch, const int32_t *step_lens, const uint8_t *decisions, int want,
                                    int n_tokens, int32_t *out, cudaStream_t stream) {
    const long long n = (long long)batch * n_tokens;
    const cudaError_t err = launch_pdl(phase_lens_tokens_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, stream,
                                       batch, step_lens, decisions, want, n_tokens, out);
    ctx->launches++;
    return err == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

arb_status launch_phase_lens(Ctx *ctx, int batch, const int32_t *step_lens, const uint8_t *decisions, int want, int t,
                             int32_t *out, cudaStream_t stream) {
    const cudaError_t err = launch_pdl(phase_lens_kernel, dim3((batch + 127) / 128), dim3(128), 0, stream, batch,
                                       step_lens, decisions, want, t, out);
    ctx->launches++;
    return err == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

arb_status launch_route(Ctx *ctx, int dtype, int n_steps, int hidden_dim, const void *hidden, const void *w,
                        float b, float tau, float *scores, uint8_t *decisions, cudaStream_t stream) {
    const int grid = (n_steps + kRouteWarps - 1) / kRouteWarps;
    cudaError_t err;
    if (dtype == ARB_BF16)
        err = launch_pdl(route_kernel<__nv_bfloat16>, dim3(grid), dim3(kRouteWarps * 32), 0, stream,
                         static_cast<const char *>(hidden), static_cast<const char *>(w), n_steps, hidden_dim, b, tau,
                         scores, decisions);
    else if (dtype == ARB_F32)
        err = launch_pdl(route_kernel<float>, dim3(grid), dim3(kRouteWarps * 32), 0, stream,
                         static_cast<const char *>(hidden), static_cast<const char *>(w), n_steps, hidden_dim, b, tau,
                         scores, decisions);
    else
        return ARB_ERR_UNSUPPORTED;
    ctx->launches++;
    return err == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

arb_status launch_rollback(Ctx *ctx, int batch, int32_t *seq_lens, const int32_t *step_lens,
                           const uint8_t *decisions, cudaStream_t stream) {
    const cudaError_t err = launch_pdl(rollback_kernel, dim3((batch + 127) / 128), dim3(128), 0, stream, batch, seq_lens,
                                       step_lens, decisions, ctx->status);
    ctx->launches++;
    return err == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

}  // namespace arb

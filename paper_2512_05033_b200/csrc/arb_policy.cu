// Escalation policies on PRM scores, and C-way router heads.
//
// Policies (decision 1 = escalate the step to the target, 0 = keep the draft step):
//   RSD baseline (Section 3.1 of the paper): the step is accepted iff s_d > tau, so escalated iff s_d <= tau.
//   Oracle threshold (Section 4.1): escalate iff Delta = s_t - s_d > tau.
//   Oracle arg max (Section 4.1): keep the higher-scoring step; escalate iff s_t > s_d.
//   Budgeted oracle (Appendix B, Theorem): escalate the min(budget, #{Delta > 0}) steps with the largest
//   positive Delta; equal advantages go to the lower index.  Done by counting, not sorting: step i's
//   rank is the number of steps that come before it in (Delta descending, index ascending) order, and
//   every thread finds its own rank against tiles of Delta staged in shared memory.
// Each kernel also accumulates the escalation count, the wasted escalations of Section 3.2 (escalated
// although s_t <= s_d), the realised score sum_i (a_i ? s_t : s_d) and the gain sum_i a_i (s_t - s_d).
// Delta is one fp32 subtraction, not flushed to zero for subnormal results, so that the decision is
// the one an IEEE fp32 subtraction gives.
//
// C-way heads (Section 6.1, ablation): one warp per step computes the C logits (softmax head) or one
// logit against C - 1 ordered cut points (ordinal head), the class probabilities, the expected class
// level scaled to [0, 1] as the routing score, and the threshold decision (a tie accepts).
//
// Spearman's rho (the rank correlation the paper reports between router scores and the oracle advantage,
// Section 4.2 "Evaluation" and Tables 1-3): ranks by counting -- rank_i = #{x_j < x_i} + (#{x_j = x_i} + 1) / 2,
// ties sharing the mean of the ranks they span -- for both samples in one pass over shared-memory tiles,
// then the three centred sums of the Pearson formula in fp64 and a one-thread kernel for the quotient.
#include "arb_common.cuh"

namespace arb {

namespace {

constexpr int kPolicyThreads = 256;

__device__ __forceinline__ float sub_ieee(float a, float b) {
    float r;
    asm("sub.rn.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

// block-wide sums of the four statistics, then one atomic each
__device__ __forceinline__ void add_stats(arb_policy_stats *stats, unsigned esc, unsigned wasted, double realised,
                                          double gain) {
    __shared__ unsigned s_esc[kPolicyThreads / 32], s_wst[kPolicyThreads / 32];
    __shared__ double s_real[kPolicyThreads / 32], s_gain[kPolicyThreads / 32];
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        esc += __shfl_xor_sync(0xffffffffu, esc, off);
        wasted += __shfl_xor_sync(0xffffffffu, wasted, off);
        realised += __shfl_xor_sync(0xffffffffu, realised, off);
        gain += __shfl_xor_sync(0xffffffffu, gain, off);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { s_esc[warp] = esc; s_wst[warp] = wasted; s_real[warp] = realised; s_gain[warp] = gain; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kPolicyThreads / 32; ++w) {
            esc += s_esc[w]; wasted += s_wst[w]; realised += s_real[w]; gain += s_gain[w];
        }
        if (esc) atomicAdd(&stats->escalated, esc);
        if (wasted) atomicAdd(&stats->wasted, wasted);
        atomicAdd(&stats->realised, realised);
        atomicAdd(&stats->gain, gain);
    }
}

__global__ void __launch_bounds__(kPolicyThreads)
policy_kernel(int kind, int n, const float *__restrict__ s_d, const float *__restrict__ s_t, float tau, int budget,
              uint8_t *__restrict__ decisions, arb_policy_stats *stats) {
    __shared__ float tile[kPolicyThreads];
    const int i = blockIdx.x * kPolicyThreads + threadIdx.x;
    const bool live = i < n;
    const float sd = live ? s_d[i] : 0.f;
    const float st = (live && s_t != nullptr) ? s_t[i] : sd;
    const float delta = sub_ieee(st, sd);
    int a = 0;
    if (kind == ARB_POLICY_RSD) {
        a = live && !(sd > tau);
    } else if (kind == ARB_POLICY_ORACLE_THRESHOLD) {
        a = live && delta > tau;
    } else if (kind == ARB_POLICY_ORACLE_ARGMAX) {
        a = live && st > sd;
    } else {
        // rank of step i in (Delta descending, index ascending) order; uniform trip count per block
        int rank = 0;
        for (int j0 = 0; j0 < n; j0 += kPolicyThreads) {
            const int j = j0 + threadIdx.x;
            __syncthreads();
            tile[threadIdx.x] = j < n ? sub_ieee(s_t[j], s_d[j]) : -INFINITY;
            __syncthreads();
            const int m = min(kPolicyThreads, n - j0);
            for (int k = 0; k < m; ++k) {
                const float dj = tile[k];
                rank += (dj > delta) || (dj == delta && j0 + k < i);
            }
        }
        a = live && delta > 0.f && rank < budget;
    }
    if (live) decisions[i] = (uint8_t)a;
    if (stats != nullptr) {   // uniform: every thread of the block takes part in the reduction
        const bool w = a && !(st > sd);
        add_stats(stats, (unsigned)a, (unsigned)w, live ? (double)(a ? st : sd) : 0.0,
                  a ? (double)st - (double)sd : 0.0);
    }
}

__global__ void __launch_bounds__(kPolicyThreads)
spearman_rank_kernel(int n, const float *__restrict__ x, const float *__restrict__ y, double *__restrict__ acc) {
    __shared__ float xs[kPolicyThreads], ys[kPolicyThreads];
    __shared__ double red[3][kPolicyThreads / 32];
    const int i = blockIdx.x * kPolicyThreads + threadIdx.x;
    const bool live = i < n;
    const float xi = live ? x[i] : 0.f, yi = live ? y[i] : 0.f;
    int lx = 0, ex = 0, ly = 0, ey = 0;
    for (int j0 = 0; j0 < n; j0 += kPolicyThreads) {
        const int j = j0 + threadIdx.x;
        __syncthreads();
        xs[threadIdx.x] = j < n ? x[j] : 0.f;
        ys[threadIdx.x] = j < n ? y[j] : 0.f;
        __syncthreads();
        const int m = min(kPolicyThreads, n - j0);
        for (int k = 0; k < m; ++k) {
            lx += xs[k] < xi; ex += xs[k] == xi;
            ly += ys[k] < yi; ey += ys[k] == yi;
        }
    }
    const double mean = ((double)n + 1.0) * 0.5;
    const double dx = live ? (double)lx + ((double)ex + 1.0) * 0.5 - mean : 0.0;
    const double dy = live ? (double)ly + ((double)ey + 1.0) * 0.5 - mean : 0.0;
    double v[3] = {dx * dy, dx * dx, dy * dy};
#pragma unroll
    for (int q = 0; q < 3; ++q) {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) v[q] += __shfl_xor_sync(0xffffffffu, v[q], off);
        if ((threadIdx.x & 31) == 0) red[q][threadIdx.x >> 5] = v[q];
    }
    __syncthreads();
    if (threadIdx.x < 3) {
        double t = 0.0;
        for (int w = 0; w < kPolicyThreads / 32; ++w) t += red[threadIdx.x][w];
        atomicAdd(&acc[threadIdx.x], t);
    }
}

__global__ void spearman_finish_kernel(int n, const double *__restrict__ acc, double *__restrict__ rho) {
    const double sxy = acc[0], sxx = acc[1], syy = acc[2];
    *rho = (n < 2 || !(sxx > 0.0) || !(syy > 0.0)) ? __longlong_as_double(0x7ff8000000000000ll) : sxy / sqrt(sxx * syy);
}

constexpr int kHeadWarps = 4;

struct HeadArgs {
    const char *hidden;
    const char *w;
    float b[ARB_MAX_CLASSES];
    int n_steps, hidden_dim, n_classes, mode;
    float tau;
    float *probs, *scores;
    uint8_t *decisions;
};

template <typename T>
__global__ void __launch_bounds__(kHeadWarps * 32)
route_classes_kernel(const HeadArgs a) {
    constexpr int EPL = Elt<T>::kPerVec;
    // one CTA per step: its warps share the row (a single warp per step would walk the row in 14 dependent
    // round trips at the router's hidden size), partial sums meet in shared memory
    __shared__ float part[kHeadWarps][ARB_MAX_CLASSES];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int step = blockIdx.x;
    const int C = a.n_classes;
    const int nlog = a.mode == ARB_HEAD_SOFTMAX ? C : 1;   // dot products to take
    const int nvec = a.hidden_dim / EPL;
    const uint4 *hrow = reinterpret_cast<const uint4 *>(a.hidden + (size_t)step * a.hidden_dim * sizeof(T));
    float acc[ARB_MAX_CLASSES];
#pragma unroll
    for (int c = 0; c < ARB_MAX_CLASSES; ++c) acc[c] = 0.f;
    for (int v = threadIdx.x; v < nvec; v += kHeadWarps * 32) {
        float hf[EPL];
        Elt<T>::unpack(__ldg(hrow + v), hf);
#pragma unroll
        for (int c = 0; c < ARB_MAX_CLASSES; ++c) {
            if (c < nlog) {
                float wf[EPL];
                Elt<T>::unpack(__ldg(reinterpret_cast<const uint4 *>(a.w + (size_t)c * a.hidden_dim * sizeof(T)) + v), wf);
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc[c] = fmaf(hf[e], wf[e], acc[c]);
            }
        }
    }
#pragma unroll
    for (int c = 0; c < ARB_MAX_CLASSES; ++c) {
        if (c < nlog) {
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], off);
        }
    }
    if (lane == 0) {
#pragma unroll
        for (int c = 0; c < ARB_MAX_CLASSES; ++c)
            if (c < nlog) part[warp][c] = acc[c];
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
#pragma unroll
    for (int c = 0; c < ARB_MAX_CLASSES; ++c) {
        if (c < nlog) {
            float t = part[0][c];
            for (int w2 = 1; w2 < kHeadWarps; ++w2) t += part[w2][c];
            acc[c] = t;
        }
    }
    float p[ARB_MAX_CLASSES];
    if (a.mode == ARB_HEAD_SOFTMAX) {
        float mx = -INFINITY, z = 0.f;
#pragma unroll
        for (int c = 0; c < ARB_MAX_CLASSES; ++c)
            if (c < C) { acc[c] += a.b[c]; mx = fmaxf(mx, acc[c]); }
#pragma unroll
        for (int c = 0; c < ARB_MAX_CLASSES; ++c)
            if (c < C) { p[c] = expf(acc[c] - mx); z += p[c]; }
        const float inv = 1.0f / z;
#pragma unroll
        for (int c = 0; c < ARB_MAX_CLASSES; ++c)
            if (c < C) p[c] *= inv;
    } else {
        const float z = acc[0] + a.b[0];
        float ge_prev = 1.0f;   // P(y >= 0)
#pragma unroll
        for (int c = 0; c < ARB_MAX_CLASSES; ++c) {
            if (c < C) {
                const float ge_next = c + 1 < C ? 1.0f / (1.0f + expf(-(z - a.b[c + 1]))) : 0.f;   // P(y >= c + 1)
                p[c] = ge_prev - ge_next;
                ge_prev = ge_next;
            }
        }
    }
    float score = 0.f;
    const float step_level = 1.0f / (float)(C - 1);
#pragma unroll
    for (int c = 0; c < ARB_MAX_CLASSES; ++c) {
        if (c < C) {
            score = fmaf(p[c], (float)c * step_level, score);
            if (a.probs != nullptr) a.probs[(size_t)step * C + c] = p[c];
        }
    }
    a.scores[step] = score;
    a.decisions[step] = score > a.tau ? 1 : 0;   // a tie accepts the draft step
}

}  // namespace

arb_status launch_policy(Ctx *ctx, int kind, int n_steps, const float *s_d, const float *s_t, float tau, int budget,
                         uint8_t *decisions, arb_policy_stats *stats, cudaStream_t stream) {
    if (stats != nullptr && cudaMemsetAsync(stats, 0, sizeof(arb_policy_stats), stream) != cudaSuccess) return ARB_ERR_CUDA;
    const int grid = (n_steps + kPolicyThreads - 1) / kPolicyThreads;
    policy_kernel<<<grid, kPolicyThreads, 0, stream>>>(kind, n_steps, s_d, s_t, tau, budget, decisions, stats);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

arb_status launch_spearman(Ctx *ctx, int n, const float *x, const float *y, double *rho, cudaStream_t stream) {
    if (cudaMemsetAsync(ctx->spearman_acc, 0, 3 * sizeof(double), stream) != cudaSuccess) return ARB_ERR_CUDA;
    if (n > 0) {
        spearman_rank_kernel<<<(n + kPolicyThreads - 1) / kPolicyThreads, kPolicyThreads, 0, stream>>>(n, x, y, ctx->spearman_acc);
        ctx->launches++;
    }
    spearman_finish_kernel<<<1, 1, 0, stream>>>(n, ctx->spearman_acc, rho);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

arb_status launch_route_classes(Ctx *ctx, int dtype, int mode, int n_steps, int hidden_dim, int n_classes,
                                const void *hidden, const void *w, const float *b_host, float tau, float *probs,
                                float *scores, uint8_t *decisions, cudaStream_t stream) {
    HeadArgs a;
    a.hidden = static_cast<const char *>(hidden);
    a.w = static_cast<const char *>(w);
    for (int c = 0; c < ARB_MAX_CLASSES; ++c) a.b[c] = c < n_classes ? b_host[c] : 0.f;
    a.n_steps = n_steps;
    a.hidden_dim = hidden_dim;
    a.n_classes = n_classes;
    a.mode = mode;
    a.tau = tau;
    a.probs = probs;
    a.scores = scores;
    a.decisions = decisions;
    const int grid = n_steps;
    if (dtype == ARB_BF16)
        route_classes_kernel<__nv_bfloat16><<<grid, kHeadWarps * 32, 0, stream>>>(a);
    else if (dtype == ARB_F32)
        route_classes_kernel<float><<<grid, kHeadWarps * 32, 0, stream>>>(a);
    else
        return ARB_ERR_UNSUPPORTED;
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

}  // namespace arb

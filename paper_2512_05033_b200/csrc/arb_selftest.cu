// Self-test of the bounded wait: the path every production kernel takes when an asynchronous copy or MMA never
// signals its mbarrier.  Nothing arms the barrier of this kernel, so the wait runs out after the limit the
// caller passes, raises ARB_DEV_WAIT_TIMEOUT and the abort flag, and the kernel returns normally: no trap, no
// fault, the context stays usable.  It is the wait of arb_common.cuh itself (mbar_wait_limit), not a copy.
#include "arb_common.cuh"

namespace arb {

namespace {

constexpr int kSelftestThreads = 64;

// report[0] = 1 once the kernel has run to its end, report[1] = threads whose wait returned false,
// report[2] = cycles thread 0 waited (saturated to int32)
__global__ void __launch_bounds__(kSelftestThreads)
selftest_wait_kernel(long long limit, uint32_t *status, int32_t *report) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    __shared__ int gave_up;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
        abort_flag = 0;
        gave_up = 0;
    }
    __syncthreads();
    // warp 0 runs out its own limit; warp 1 is given a limit it cannot reach and must leave through the abort flag
    const long long mine = threadIdx.x < 32 ? limit : (1ll << 40);
    const long long t0 = clock64();
    const bool ok = mbar_wait_limit(&bar, 0u, &abort_flag, status, mine);
    const long long waited = clock64() - t0;
    if (!ok) atomicAdd(&gave_up, 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        report[1] = gave_up;
        report[2] = (int32_t)(waited > 0x7fffffffll ? 0x7fffffffll : waited);
        __threadfence();
        report[0] = 1;
    }
}

// counts the bytes of the guard zones that do not hold the pattern; zones: device array of n pointers
__global__ void guard_count_kernel(const unsigned char *const *zones, int n_zones, size_t zone_bytes,
                                   unsigned long long *bad) {
    unsigned long long mine = 0;
    for (int z = 0; z < n_zones; ++z)
        for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < zone_bytes; i += (size_t)gridDim.x * blockDim.x)
            mine += zones[z][i] != kGuardPattern;
    if (mine) atomicAdd(bad, mine);
}

}  // namespace

arb_status launch_guard_count(Ctx *ctx, const unsigned char *const *zones, int n_zones, size_t zone_bytes,
                              unsigned long long *bad_dev, cudaStream_t stream) {
    guard_count_kernel<<<8, 256, 0, stream>>>(zones, n_zones, zone_bytes, bad_dev);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

arb_status launch_selftest_wait(Ctx *ctx, long long limit_cycles, int32_t *report, cudaStream_t stream) {
    selftest_wait_kernel<<<1, kSelftestThreads, 0, stream>>>(limit_cycles, ctx->status, report);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? ARB_OK : ARB_ERR_CUDA;
}

}  // namespace arb

// A bounded wait that is made to run out on purpose, without touching any model kernel: one small CTA
// waits on an mbarrier that nothing signals (no arrival, no copy in flight), with the same wait routine
// and the same way out that the GEMM, attention and LayerNorm kernels use when a wait gives up: leave the
// loop, raise bit 1 of the status word, return normally.
#include "internal.h"
#include "ptx.cuh"

namespace kr {

namespace {

__global__ void __launch_bounds__(64, 1) wait_probe_kernel(uint32_t *status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_word;
    volatile uint32_t *abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_word = 0;
        fence_barrier_init();
    }
    __syncthreads();
    // warp 0 waits on the barrier itself; warp 1 stands for the other roles of a kernel, which learn of the
    // give-up through the abort flag on their own polls
    bool ok = mbar_wait(&bar, 0, abort_flag, limit_ns);
    ok = __all_sync(0xFFFFFFFFu, ok);
    __syncthreads();
    if (threadIdx.x == 0 && (!ok || *abort_flag) && status) atomicOr(status, STATUS_WAIT_LIMIT);
}

}  // namespace

}  // namespace kr

extern "C" int kraken_test_wait_limit(uint32_t *d_status, uint32_t limit_us, void *stream) {
    using namespace kr;
    if (!d_status || limit_us < 1 || limit_us > 1000000u) return KRAKEN_EINVAL;
    wait_probe_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(d_status, 1000ull * limit_us);
    return cuda_check(cudaGetLastError(), "wait probe: launch");
}

// Self-test of the bounded device-side wait: the way every tcgen05 kernel of this library reports a wait that cannot
// end.  One CTA initialises an mbarrier on which nothing will ever arrive and waits on it with a SHORT limit; the wait
// must give up, the kernel raises DEV_E_WAIT_TIMEOUT in the handle's sticky status word and returns normally (no trap,
// no endless loop), and the context stays usable.
#include "tc_common.cuh"

namespace anakin {

__global__ void __launch_bounds__(32) k_selftest_wait(int* status, long long limit_clocks, long long* waited_clocks) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        tc::mbar_fence_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        const bool ok = tc::mbar_wait(&bar, 0, limit_clocks);  // phase 0 never completes: nobody arrives
        if (waited_clocks) *waited_clocks = clock64() - t0;
        if (!ok) atomicOr(status, DEV_E_WAIT_TIMEOUT);
    }
}

cudaError_t launch_selftest_wait(int* status, long long limit_clocks, long long* waited_clocks, cudaStream_t s) {
    k_selftest_wait<<<1, 32, 0, s>>>(status, limit_clocks, waited_clocks);
    return cudaGetLastError();
}

}  // namespace anakin

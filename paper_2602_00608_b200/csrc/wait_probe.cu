// A one-block kernel that runs the library's bounded wait into its limit on purpose, for the test
// of the device-timeout path: it waits on an mbarrier that nothing ever arrives on, gives up after
// `limit_cycles` SM clocks, records the same kind of code in the status word that the tensor-core
// kernels record, and returns normally (no trap, no endless loop: the context stays usable).
#include "tc_common.cuh"
#include "vd_internal.h"

namespace vd {

namespace {

__global__ void wait_probe_kernel(unsigned int* status, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        tc::mbar_init(tc::smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // every thread waits, as the roles of the real kernels do; the first to reach the limit raises the flag
    const bool ok = tc::mbar_wait(tc::smem_u32(&bar), 0, &abort_flag, limit_cycles);
    __syncthreads();
    if (threadIdx.x == 0 && !ok && abort_flag && status) {
        if (atomicCAS(status, 0u, kStatusWaitProbe) == 0u) {
            status[1] = blockIdx.x;
            status[2] = (unsigned int)(limit_cycles & 0xffffffffll);
        }
    }
}

}  // namespace

cudaError_t launch_wait_probe(unsigned int* status_word, long long limit_cycles, cudaStream_t s) {
    wait_probe_kernel<<<1, 64, 0, s>>>(status_word, limit_cycles);
    return cudaGetLastError();
}

}  // namespace vd

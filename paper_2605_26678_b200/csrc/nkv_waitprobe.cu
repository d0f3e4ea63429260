// Test kernel for the bounded waits of the tcgen05 kernels: one warp waits, with the kernels' own polling
// loop, on an mbarrier that nothing ever arrives at, gives up after `limit` polls and records NKV_ERR_TIMEOUT.
// No copy, product or other thread is involved, so the wait ends by itself and leaves the context usable.
#include "nkv_sm100.cuh"

namespace nkv {

namespace {

__global__ void __launch_bounds__(32) wait_probe_kernel(int* status, uint32_t limit) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        sm100::mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    sm100::mbar_wait_poll(&bar, 0, status, kWaitProbeDetail, limit);
}

}  // namespace

cudaError_t launch_wait_probe(int* status, uint32_t limit, cudaStream_t stream, int64_t* launches) {
    wait_probe_kernel<<<1, 32, 0, stream>>>(status, limit);
    if (launches) ++*launches;
    return cudaGetLastError();
}

}  // namespace nkv

// Test hook for the failure path of the bounded waits: one CTA waits, with the configured limit, on an mbarrier that
// nothing ever arrives at. The wait runs out, the thread records JA_ERR_TIMEOUT in the stream's status word exactly as a
// product kernel would, the other lanes see the abort flag, and the kernel returns normally -- nothing faults, traps or
// spins without a limit. No product kernel is made to stall.
#include "ja_device.cuh"
#include "ja_ptx.cuh"

namespace {

using namespace ja_ptx;

__global__ void wait_timeout_kernel(int32_t* status, uint32_t cap_us, int32_t* polls_out) {
    __shared__ uint64_t barrier;
    __shared__ int ctl[2];
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&barrier), 1);
        wait_ctl_init(ctl, cap_us);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool ok = true;
    if (threadIdx.x == 0) ok = mbar_wait(smem_u32(&barrier), 0, ctl, status);         // runs out: records the error, raises the flag
    __syncthreads();
    if (threadIdx.x == 1) ok = mbar_wait(smem_u32(&barrier), 0, ctl, status);         // sees the flag at its first check and gives up
    if (threadIdx.x < 2 && polls_out) polls_out[threadIdx.x] = ok ? 1 : 0;
}

}  // namespace

// polls_out: optional DEVICE array of two ints: whether the first and the second waiter reported success (both must be 0)
extern "C" ja_status_t ja_debug_wait_timeout(void* cuda_stream, int32_t* polls_out) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int32_t* status = ja_device_status_word(st);
    if (!status) return ja_fail(JA_ERR_CUDA, "cannot resolve the device status word");
    wait_timeout_kernel<<<1, 32, 0, st>>>(status, (uint32_t)ja_config().wait_cap_us, polls_out);
    JA_CUDA(cudaGetLastError());
    ja_count_launch();
    return JA_OK;
}

// Test aid for the bounded waits: one warp waits on an mbarrier that nothing ever completes, with the same
// helper and the same sticky status word the attention kernels use.  The wait gives up after `limit_ns`, records
// kStatusTimeout and the kernel returns normally, so the context stays usable and the host can read the status.
#include "common.cuh"
#include "ptx.cuh"

namespace regenvc {

__global__ void __launch_bounds__(32) expire_wait_kernel(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t never;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&never), 1);
        fence_mbar_init();
        const WaitCtl ctl{&abort_flag, status, kStatusTimeout, limit_ns};
        (void)mbar_wait(smem_u32(&never), 0, ctl);
    }
    __syncwarp();
}

cudaError_t launch_expire_wait(int* status, unsigned long long limit_ns, cudaStream_t stream) {
    expire_wait_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
    return cudaGetLastError();
}

}  // namespace regenvc

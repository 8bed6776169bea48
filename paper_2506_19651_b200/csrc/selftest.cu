// Self-test of the bounded device-side wait: one thread waits, with the same wait routine the attention
// kernel uses, on an mbarrier that nothing ever arrives on.  The wait runs out after `limit_ns`, the thread
// records PEVLM_ETIMEOUT and the id of the wait in the workspace header exactly as the attention kernel does,
// and the kernel ends normally: no trap, no fault, the context stays usable.
#include "internal.h"
#include "ptx.cuh"

namespace pevlm {

constexpr int kWaitSelfTest = 99;  // wait id reported in the detail word: 99 * 1000000 + CTA index

__global__ void wait_selftest_kernel(WorkspaceHeader* hdr, uint64_t limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (!mbar_wait(smem_u32(&bar), 0, &abort_flag, limit_ns)) {
            if (atomicCAS(&hdr->status, 0, PEVLM_ETIMEOUT) == 0) hdr->detail = kWaitSelfTest * 1000000 + blockIdx.x;
        }
    }
    __syncthreads();
    // after the first expiry every later wait of the CTA gives up after the short grace period
    if (threadIdx.x == 1) (void)mbar_wait(smem_u32(&bar), 0, &abort_flag, limit_ns);
}

cudaError_t launch_wait_selftest(WorkspaceHeader* hdr, uint64_t limit_ns, cudaStream_t stream) {
    wait_selftest_kernel<<<1, 32, 0, stream>>>(hdr, limit_ns);
    return cudaGetLastError();
}

}  // namespace pevlm

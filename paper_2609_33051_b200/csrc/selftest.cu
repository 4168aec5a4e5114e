// Self-test of the library's failure reporting: a kernel whose bounded wait is certain to run out.
//
// Every wait in the hot-path kernels (mbarrier phases completed by bulk copies or by tensor-core commits) is
// bounded: when the limit is reached the kernel records a code in the caller's status block, stops waiting and
// returns, and the host finds the code with sketchssm_read_status.  Nothing in normal operation makes a wait run
// out, so this entry point exists to exercise that path end to end without a hang, a trap or a bad address: one
// warp waits, with a small poll limit, on a barrier phase that nothing will ever complete.  No copy is issued,
// so nothing is in flight when the warp gives up.
#include "internal.cuh"

namespace sketchssm {

namespace {

__global__ void __launch_bounds__(32, 1) wait_probe_kernel(int* status, uint32_t poll_limit, int where) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    __syncwarp();
    const bool ok = mbar_wait_bounded(&bar, 0u, poll_limit);       // phase 0 never completes: nobody arrives
    if (__any_sync(0xffffffffu, !ok)) {
        if (threadIdx.x == 0) record_fault(status, kFaultProbeWait, where);
    }
}

}  // namespace

int launch_wait_probe(Ctx* ctx, int poll_limit, int where, cudaStream_t stream) {
    wait_probe_kernel<<<1, 32, 0, stream>>>(static_cast<int*>(ctx->bufs.status), (uint32_t)poll_limit, where);
    if ((ctx->last_cuda_error = cudaGetLastError()) != cudaSuccess) return SKETCHSSM_CUDA_ERROR;
    ctx->last_launches = 1;
    return SKETCHSSM_OK;
}

}  // namespace sketchssm

// Self-test of the bounded device-side waits: one warp waits on an mbarrier that nothing ever arrives at, with the
// same wait routine and the same give-up path as the tensor-core kernels (flag in the status block, id of the
// wait, block index), then returns.  Nothing is left waiting and the context stays usable.
#include "tc_common.cuh"

namespace iptq {

constexpr int kSelftestWaitId = 99;

__global__ void __launch_bounds__(64) wait_timeout_selftest_kernel(StatusBlock* status)
{
    __shared__ uint64_t bar;
    __shared__ CtaControl ctl;
    grid_dep_launch();
    grid_dep_wait();
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        ctl.abort = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        // no thread and no copy ever arrives at this barrier: the wait can only run out
        if (elect_one()) mbar_wait(&bar, 0, &ctl, status, kSelftestWaitId);
        __syncwarp();
    }
    __syncthreads();          // the second warp sees the abort flag only after the wait has given up
}

}  // namespace iptq

using namespace iptq;

extern "C" {

int iptq_workspace_set_wait_limit(void* ws, size_t ws_bytes, int32_t microseconds, iptq_stream_t stream)
{
    if (!ws) return IPTQ_ERR_NULL;
    if (ws_bytes < kStatusBytes) return IPTQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return IPTQ_ERR_ALIGN;
    if (microseconds < 0) return IPTQ_ERR_SHAPE;
    StatusBlock* sb = static_cast<StatusBlock*>(ws);
    return cuda_status(cudaMemcpyAsync(&sb->wait_limit_us, &microseconds, sizeof(int32_t), cudaMemcpyHostToDevice, stream));
}

int iptq_selftest_wait_timeout(void* ws, size_t ws_bytes, iptq_stream_t stream)
{
    if (!ws) return IPTQ_ERR_NULL;
    if (ws_bytes < kStatusBytes) return IPTQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return IPTQ_ERR_ALIGN;
    launch_kernel(wait_timeout_selftest_kernel, 1, 64, 0, stream, static_cast<StatusBlock*>(ws));
    note_launch();
    return last_launch_status();
}

}  // extern "C"

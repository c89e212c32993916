// Self-test of the bounded-wait path, and the status check that turns a recorded time-out into a status.
//
// Every pipeline wait in the library's kernels gives up after a cycle budget, records a code in the status
// block and lets the kernel drain. That path cannot be reached by starving a production kernel (nothing here
// hangs or faults a GPU on purpose); instead one warp runs the same wait routine, with a short budget, on a
// barrier that nothing completes, and takes the same way out: flag, status word, normal return.
#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

__global__ void __launch_bounds__(32)
wait_expiry_kernel(unsigned *status, long long budget_cycles)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);                       // one arrival expected; none ever comes
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncwarp();
    // all lanes wait on phase 0, as the consumer warps of the decode kernels do
    const bool ok = mbar_wait_budget(&bar, 0, &abort_flag, budget_cycles);
    __syncwarp();
    if (threadIdx.x == 0 && (!ok || abort_flag)) {
        if (atomicOr(status + kStatusErrWord, kErrSelfTestWait) == 0u) status[kStatusInfoWord] = 0x40000u;
    }
}

}  // namespace

// l4l_decode.cu: device address of the library's own scratch array on the current device (nullptr on failure)
void *static_scratch_on_current_device();

}  // namespace l4l

extern "C" l4l_status l4l_selftest_wait_expiry(void *workspace, size_t ws_bytes, long long budget_cycles, l4l_stream stream)
{
    using namespace l4l;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (budget_cycles < 1000) budget_cycles = 1000;
    if (budget_cycles > (1ll << 24)) budget_cycles = 1ll << 24;
    wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<unsigned *>(workspace), budget_cycles);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

extern "C" l4l_status l4l_check_status(void *workspace, l4l_stream stream)
{
    using namespace l4l;
    void *block = workspace ? workspace : static_scratch_on_current_device();
    if (!block) return L4L_ERR_CUDA;
    const int code = l4l_last_device_error(block, stream);
    if (code < 0) return L4L_ERR_CUDA;
    return code == 0 ? L4L_OK : L4L_ERR_TIMEOUT;
}

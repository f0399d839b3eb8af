// Self-test of the bounded-wait protocol the tensor-core kernels share (tcgen05.cuh): one CTA allocates tensor
// memory, starts a bulk copy, and then waits on an mbarrier that nothing ever arrives at.  The wait runs out after
// a short, caller-given number of polls; the waiting role raises the CTA's abort flag and records
// AMX_ERR_TIMEOUT in the status word; the other roles, parked in waits of the normal length, leave through the
// flag; the copy in flight is drained with a bounded wait; tensor memory is released; the kernel returns and the
// context stays usable.  Nothing here faults, traps or spins without a limit.
#include "amx_common.cuh"
#include "tcgen05.cuh"

namespace amx {
namespace {

using namespace tc;

constexpr int kWarps = 4;
constexpr uint32_t kCopyBytes = 1024;

// trace[w]: what warp w saw - 1 its wait completed (never expected), 2 it gave up at its own limit, 3 it left
// because another role had raised the abort flag; trace[4]: 1 when the copy in flight was seen to land
__global__ void __launch_bounds__(kWarps * 32)
wait_timeout_kernel(const uint8_t* __restrict__ src, int* __restrict__ status, int* __restrict__ trace, uint32_t polls) {
    __shared__ __align__(128) uint8_t landing[kCopyBytes];
    __shared__ uint64_t never, copied;
    __shared__ uint32_t tmem_base;
    __shared__ volatile int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(&never, 1);
        mbar_init(&copied, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&tmem_base, 32);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) {
        if (lane == 0) {
            mbar_expect_tx(&copied, kCopyBytes);
            bulk_load(landing, src, kCopyBytes, &copied);
            const bool ok = mbar_wait(&never, 0, &abort_flag, status, polls);     // runs out
            trace[0] = ok ? 1 : 2;
            // after giving up: let the copy in flight land before shared memory is released
            bool landed = false;
            for (uint32_t n = 0; n < kSpinLimit && !landed; ++n) landed = mbar_try_wait(&copied, 0);
            trace[kWarps] = landed ? 1 : 0;
        }
    } else if (lane == 0) {
        const int before = abort_flag;
        const bool ok = mbar_wait(&never, 0, &abort_flag, status);               // leaves through the abort flag
        trace[warp] = ok ? 1 : (before || abort_flag) ? 3 : 2;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 32);
    }
}

}  // namespace
}  // namespace amx

extern "C" int amx_selftest_wait_timeout(void* workspace, size_t workspace_bytes, uint32_t polls, void* stream) {
    using namespace amx;
    if (!workspace) return AMX_ERR_NULL;
    if (workspace_bytes < 2048) return AMX_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return AMX_ERR_ALIGN;
    if (polls == 0 || polls > (1u << 16)) return AMX_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, 256 + kCopyBytes, st) != cudaSuccess) return AMX_ERR_CUDA;
    int* words = static_cast<int*>(workspace);
    wait_timeout_kernel<<<1, kWarps * 32, 0, st>>>(static_cast<const uint8_t*>(workspace) + 256, words, words + 8, polls);
    return launch_status();
}

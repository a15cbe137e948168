// Exercise of the give-up path of the bounded waits: one warp waits, with a small poll limit, on a
// barrier that nothing ever arrives at.  The wait runs out, sets the handle's status word and the
// kernel returns normally; accerl_policy_check then reports ACCERL_ERR_TIMEOUT and clears the word.
// Nothing traps, faults or waits without a limit, and the context stays usable.
#include "internal.h"
#include "tc_ptx.cuh"

namespace accerl {

namespace {

constexpr int kSelftestCode = 128;  // status bit of this kernel's wait

__global__ void __launch_bounds__(32) wait_giveup_kernel(int *status, int poll_limit)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    // phase 0 never completes: nobody arrives
    const bool ok = mbar_wait_limited(smem_u32(&bar), 0, &abort_flag, status, kSelftestCode, 0, poll_limit);
    if (ok) atomicOr(status, 1 << 30);  // cannot happen; would show as a different status word
}

}  // namespace

}  // namespace accerl

using namespace accerl;

extern "C" accerl_status accerl_policy_selftest_wait(accerl_policy *p, int32_t poll_limit, void *cuda_stream)
{
    if (!p) {
        set_error("selftest_wait: null handle");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (poll_limit < 1 || poll_limit > 100000) {
        set_error("selftest_wait: poll_limit must lie in 1..100000 (at most 256 ns a poll)");
        return ACCERL_ERR_INVALID_ARG;
    }
    int prev = -1;
    cudaGetDevice(&prev);
    struct Restore {
        int prev;
        ~Restore() { if (prev >= 0) cudaSetDevice(prev); }
    } restore{prev};
    ACCERL_CUDA_TRY(cudaSetDevice(p->device));
    p->last_stream = (cudaStream_t)cuda_stream;
    wait_giveup_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(p->status_word, poll_limit);
    ACCERL_CUDA_TRY(cudaGetLastError());
    return ACCERL_OK;
}

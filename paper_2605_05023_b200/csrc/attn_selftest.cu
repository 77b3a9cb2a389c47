// Self-test of the failure path that every kernel of this library shares: a bounded wait that gives up.
//
// The tensor-core kernels link their roles with mbarriers, and every wait on one is bounded (sm100_sync.cuh): when
// the limit passes, the waiting thread stores ATTN_ERR_TIMEOUT in the caller's status word, raises the CTA's abort
// flag, and the kernel drains and returns, so that the context stays usable.  In a correct launch no wait ever runs
// out, so this path is exercised here on purpose and harmlessly: a one-CTA kernel waits, with a short limit, on an
// mbarrier that nothing arrives on.  No trap, no fault, nothing is left spinning.
#include "../../include/attn.h"
#include "sm100_ptx.cuh"
#include "sm100_sync.cuh"

namespace b200attn {
namespace {

__global__ void __launch_bounds__(64, 1) bounded_wait_selftest_kernel(int32_t* status_word, unsigned long long limit_ns,
                                                                      int32_t* waited) {
    __shared__ uint64_t never_completes;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&never_completes), 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    // Warp 0, lane 0 waits and gives up after limit_ns; warp 1, lane 0 waits on the same barrier with the full
    // limit of the kernels and must leave as soon as the first one raises the abort flag.
    bool ok = true;
    if ((threadIdx.x & 31) == 0)
        ok = tc::bounded_wait_on<false>(ptx::smem_u32(&never_completes), 0u, &abort_flag, status_word,
                                        threadIdx.x == 0 ? (uint64_t)limit_ns : tc::kWaitLimitNs);
    __syncthreads();
    if (threadIdx.x == 32 && waited) *waited = ok ? 1 : 2;      // 2: the second waiter saw the abort and returned
}

}  // namespace
}  // namespace b200attn

extern "C" int attn_selftest_timeout(int32_t* status_word, uint64_t limit_ns, int32_t* second_waiter, void* stream) {
    if (!status_word) return ATTN_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(status_word) & 3u) || (second_waiter && (reinterpret_cast<uintptr_t>(second_waiter) & 3u)))
        return ATTN_ERR_ALIGN;
    if (limit_ns == 0 || limit_ns > 100000000ull) return ATTN_ERR_DESC;     // at most 0.1 s
    b200attn::bounded_wait_selftest_kernel<<<1, 64, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        status_word, (unsigned long long)limit_ns, second_waiter);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

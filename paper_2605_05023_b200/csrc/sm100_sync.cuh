// Device-side plumbing shared by every tensor-core kernel of this library (the three attention kernels and the
// GEMM + row-sum kernel): the bounded mbarrier wait, the work-item fetch through cluster launch control, the
// warp-level arrivals, and the check of a packed-document offset table.
//
// Nothing here spins for ever.  A wait that is not satisfied within its limit records ATTN_ERR_TIMEOUT in the
// caller's status word, raises the CTA's abort flag and returns false; every role tests the return value and
// drains to the kernel's common exit, where TMEM is released.
#pragma once
#include <cstdint>

#include "../../include/attn.h"
#include "sm100_ptx.cuh"

namespace b200attn {
namespace tc {

constexpr uint64_t kWaitLimitNs = 2000000000ull; // bounded waits give up after 2 s

// Waits until the phase with this parity of the mbarrier at shared-memory address `bar` has completed.
//   kCluster    the barrier is arrived on by the other CTA of a pair (acquire at cluster scope);
//   abort_flag  the CTA's abort flag in shared memory: raised by the first wait that gives up, polled by all;
//   limit_ns    how long to wait (the kernels use kWaitLimitNs; the self-test passes a short limit).
template <bool kCluster = false>
__device__ __forceinline__ bool bounded_wait_on(uint32_t bar, uint32_t parity, int* abort_flag, int32_t* status_word,
                                                uint64_t limit_ns = kWaitLimitNs) {
    auto attempt = [&]() { return kCluster ? ptx::mbar_try_wait_cluster(bar, parity) : ptx::mbar_try_wait(bar, parity); };
    if (attempt()) return true;
    uint64_t t0 = 0;
    uint32_t spins = 0;
    volatile int* aborted = abort_flag;
    while (true) {
        if (attempt()) return true;
        if ((++spins & 0x3Fu) == 0) {
            if (*aborted) return false;
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > limit_ns) {
                *aborted = 1;
                if (status_word) atomicExch(status_word, (int)ATTN_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

// One request to the hardware scheduler for the next not-yet-started CTA (cluster) of the grid, issued and read
// by ONE thread: the 16 response bytes are written through the async proxy, so the reader orders its reads
// before the next request with a proxy fence, and publishes what it learnt to the other roles with ordinary
// stores.  (With every role reading the response itself and no such fence, a late reader now and then saw the
// bytes of the following response.)  Returns false when the wait was abandoned; otherwise `got` tells whether a
// CTA was handed over and `ctaid_x` is its blockIdx.x.
__device__ __forceinline__ bool clc_fetch(uint32_t clc_bar, uint64_t* response, uint32_t& clc_phase, int* abort_flag,
                                          int32_t* status_word, bool& got, uint32_t& ctaid_x) {
    ptx::mbar_arrive_expect_tx(clc_bar, 16);
    ptx::clc_try_cancel(ptx::smem_u32(response), clc_bar);
    if (!bounded_wait_on<false>(clc_bar, clc_phase, abort_flag, status_word)) return false;
    clc_phase ^= 1u;
    const uint64_t lo = *reinterpret_cast<volatile uint64_t*>(&response[0]);
    const uint64_t hi = *reinterpret_cast<volatile uint64_t*>(&response[1]);
    got = ptx::clc_query(lo, hi, ctaid_x);
    ptx::fence_proxy_async_smem();
    return true;
}

// One arrival per warp: the warp converges first, so that every lane's earlier shared-memory / TMEM traffic is
// ordered before the arrival (the barriers count one arrival per warp).
__device__ __forceinline__ void warp_arrive(uint32_t bar) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) ptx::mbar_arrive(bar);
}
// Publishes this warp's TMEM stores to the MMA thread: every lane waits for its own stores first.
__device__ __forceinline__ void warp_arrive_after_tmem_st(uint32_t bar) {
    ptx::tmem_wait_st();
    ptx::tc_fence_before_sync();
    warp_arrive(bar);
}

// Packed documents (Appendix A.2, causal blockwise mask): the offset table must start at 0, end at `total` and
// never decrease.  Called by all 32 lanes of one warp of one CTA per launch; a table that breaks a rule is
// reported as ATTN_ERR_DESC in the status word.  (The kernels stay memory safe on any table: document look-ups
// are clamped to [0, num_docs - 1] and key intervals to [0, Sk - 1].)
__device__ __forceinline__ void check_offsets_warp(const int32_t* __restrict__ cu, int num_docs, int total, int32_t* status_word) {
    if (!cu || !status_word) return;
    const int lane = threadIdx.x & 31;
    bool bad = false;
    for (int d = lane; d < num_docs; d += 32) bad |= __ldg(cu + d) > __ldg(cu + d + 1);
    if (lane == 0) bad |= (__ldg(cu) != 0) || (__ldg(cu + num_docs) != total);
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicCAS(status_word, 0, (int)ATTN_ERR_DESC);
}

}  // namespace tc
}  // namespace b200attn

// bt_selftest_bounded_wait: shows on a live GPU that the bounded waits of the kernels give up.
//
// Every wait in the library's kernels is on a shared-memory barrier that a copy (or another warp)
// completes, and every one of them is bounded: by a poll count in the streaming decode kernels
// (mbar_wait_polls), by wall time in the prefill kernel (mbar_wait_walltime).  In production a wait
// only runs out if a copy is lost, which cannot be provoked without breaking something; here one
// small CTA calls the same two functions on barriers that were initialised and that nothing will
// ever complete.  No copy is issued and nothing is in flight, so there is nothing to drain: the waits
// return false after their (short) limits, the kernel records that, raises BT_DEV_TIMEOUT and ends.
#include "bt_common.cuh"
#include "bt_kernels.h"
#include "bt_mbarrier.cuh"

namespace bt {

constexpr uint32_t kSelftestPolls = 2048;          // poll-bounded wait: a few thousand polls
constexpr uint64_t kSelftestLimitNs = 200000ull;   // time-bounded wait: 0.2 ms
constexpr uint32_t kSelftestSpin = 1u << 22;       // and its poll cap (never reached before the time limit)

// report[0]: poll-bounded wait on a dead barrier gave up (1) / returned true (0)
// report[1]: time-bounded wait on a dead barrier gave up (1) / returned true (0)
// report[2]: control - a wait on a barrier whose phase was completed by an arrival returned true (1)
// report[3]: nanoseconds the time-bounded wait took (saturated at 2^32 - 1)
__global__ void selftest_bounded_wait_kernel(uint32_t* report, uint32_t* dev_status)
{
    __shared__ __align__(8) uint64_t bars[3];
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 3; ++i) mbar_init(smem_u32(&bars[i]), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_arrive(smem_u32(&bars[2]));  // the control barrier: its phase 0 completes right here
    }
    __syncthreads();
    if (warp == 0) {
        const bool ok = mbar_wait_polls(smem_u32(&bars[0]), 0, kSelftestPolls);
        const bool gave_up = !__any_sync(0xffffffffu, ok);
        if (lane == 0) {
            if (report) report[0] = gave_up ? 1u : 0u;
            if (gave_up) raise_status(dev_status, BT_DEV_TIMEOUT);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint64_t t0 = global_ns();
            const bool ok = mbar_wait_walltime(smem_u32(&bars[1]), 0, &abort_flag, kSelftestSpin, kSelftestLimitNs);
            const uint64_t dt = global_ns() - t0;
            if (report) {
                report[1] = ok ? 0u : 1u;
                report[3] = dt > 0xffffffffull ? 0xffffffffu : (uint32_t)dt;
            }
            if (!ok) raise_status(dev_status, BT_DEV_TIMEOUT);
        }
    } else if (warp == 2) {
        const bool ok = mbar_wait_polls(smem_u32(&bars[2]), 0, kSelftestPolls);
        if (lane == 0 && report) report[2] = ok ? 1u : 0u;
    }
}

cudaError_t launch_selftest_bounded_wait(uint32_t* report, uint32_t* dev_status, cudaStream_t stream)
{
    selftest_bounded_wait_kernel<<<1, 96, 0, stream>>>(report, dev_status);
    return cudaGetLastError();
}

}  // namespace bt

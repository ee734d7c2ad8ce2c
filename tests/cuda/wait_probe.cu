// Test-only kernel: a bounded wait that is made to run out, without hanging anything.
//
// One thread waits on an mbarrier at which nobody ever arrives, through the library's own bounded-wait
// routine (csrc/tc_common.cuh) with a small poll limit. The wait must give up, write its code into the status
// word it was given (the first word of a handle's workspace, which lococo_get_last_device_status reads), and
// raise the CTA's `failed` flag, after which a second wait gives up after 64 polls. The kernel always ends by
// itself within microseconds; the limit is capped on the host.
#include <cuda_runtime.h>
#include <stdint.h>

#include "tc_common.cuh"

namespace {

using namespace lococo::tc;

__global__ void wait_probe_kernel(int* status, uint32_t limit, long long* out) {
    __shared__ uint64_t bar;
    __shared__ int failed;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        failed = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t b = smem_u32(&bar);
        const long long t0 = clock64();
        const bool ok1 = mbar_wait_slow(b, 0, status, &failed, 42, limit);   // phase 0 never completes
        const long long t1 = clock64();
        const bool ok2 = mbar_wait_slow(b, 0, status, &failed, 43, limit);   // `failed` is set: 64 polls
        const long long t2 = clock64();
        out[0] = ok1;
        out[1] = ok2;
        out[2] = t1 - t0;
        out[3] = t2 - t1;
        out[4] = failed;
        mbar_inval(b);
    }
}

}  // namespace

// status_word, out (5 x int64): device pointers. Returns 0, -1 for a limit above 4096 polls, -2 for a launch error.
extern "C" int wait_probe_run(void* status_word, unsigned limit, void* out, void* stream) {
    if (!status_word || !out || limit < 65 || limit > 4096) return -1;
    wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<int*>(status_word), limit,
                                                                        static_cast<long long*>(out));
    return cudaGetLastError() == cudaSuccess ? 0 : -2;
}

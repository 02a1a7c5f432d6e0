// Self-test of the bounded device-side waits: a one-CTA kernel waits on an mbarrier that nothing ever arrives at,
// with a limit of one millisecond, and must come back with the time-out recorded -- first wait by running out,
// second wait by finding the CTA's latch set.  Then the same for the flag wait of the one-launch forms: a flag that
// nobody sets, one millisecond, and once more with the launch's status word already showing a failure (that wait must
// return at once).  Nothing here faults, traps or waits without a limit.
#include "kernels.h"
#include "tc_common.cuh"

namespace harts {
namespace {

using namespace tc;

__device__ int selftest_flag;       // stays zero

__global__ void selftest_timeout_kernel(int* status, int* report) {
    __shared__ uint64_t bar;
    __shared__ int dead, dead2, dead3;
    if (threadIdx.x == 0) {
        dead = dead2 = dead3 = 0;
        mbar_init(&bar, 1);
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned long long t0 = global_ns();
        const bool first = mbar_wait(&bar, 0, status, &dead, 1000ull * 1000);    // runs out after ~1 ms
        const unsigned long long t1 = global_ns();
        const bool second = mbar_wait(&bar, 0, status, &dead, 1000ull * 1000);   // latch set: returns at once
        const unsigned long long t2 = global_ns();
        if (report) {
            report[0] = first ? 1 : 0;
            report[1] = second ? 1 : 0;
            report[2] = (int)min((unsigned long long)INT32_MAX, (t1 - t0) / 1000);   // microseconds spent in each wait
            report[3] = (int)min((unsigned long long)INT32_MAX, (t2 - t1) / 1000);
        }
        const bool f1 = flag_wait(&selftest_flag, nullptr, &dead2, 1000ull * 1000);   // runs out after ~1 ms
        const unsigned long long t3 = global_ns();
        const bool f2 = flag_wait(&selftest_flag, status, &dead3);                     // status already set: at once
        const unsigned long long t4 = global_ns();
        if (report) {
            report[5] = (f1 ? 1 : 0) | (f2 ? 2 : 0) | (dead2 ? 4 : 0) | (dead3 ? 8 : 0);
            report[6] = (int)min((unsigned long long)INT32_MAX, (t3 - t2) / 1000);
            report[7] = (int)min((unsigned long long)INT32_MAX, (t4 - t3) / 1000);
        }
    }
    const int gave_up = __syncthreads_or(dead);
    if (report && threadIdx.x == 0) report[4] = gave_up ? 1 : 0;
}

}  // namespace
}  // namespace harts

extern "C" int32_t harts_la_selftest_timeout(int32_t* dev_status, int32_t* dev_report, void* stream) {
    if (!dev_status) return HARTS_EINVAL;
    harts::selftest_timeout_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(dev_status, dev_report);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

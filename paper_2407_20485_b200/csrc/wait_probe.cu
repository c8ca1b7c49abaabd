// Self-test of the bounded device-side wait: one CTA waits on an mbarrier that nobody arrives
// at, through the same tc::mbar_wait the production kernels use, with a caller-chosen limit.
// The wait gives up, the CTA is poisoned (a second wait returns at once) and the sticky status
// word is raised the way the prefill and generation-step kernels raise it.  Nothing traps and
// nothing waits without a bound.
#include "common.cuh"
#include "tc_sm100.cuh"

namespace a2sf {

namespace {

__global__ void wait_probe_kernel(int *status_word, long long limit, long long *report)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        abort_flag = 0;
        tc::fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        const bool first = tc::mbar_wait(&bar, 0, &abort_flag, limit);        // nobody arrives
        const long long t1 = clock64();
        // what the kernels' wait wrappers do once a CTA is poisoned: no further spinning
        const bool second = abort_flag ? false : tc::mbar_wait(&bar, 0, &abort_flag, limit);
        const long long t2 = clock64();
        report[0] = first ? 0 : 1;
        report[1] = t1 - t0;
        report[2] = t2 - t1;
        report[3] = second ? 0 : 1;
        if (abort_flag) *status_word = A2SF_ERR_TIMEOUT;
    }
}

}  // namespace

cudaError_t launch_wait_probe(int *status_word, long long limit_cycles, long long *report, cudaStream_t s)
{
    wait_probe_kernel<<<1, 32, 0, s>>>(status_word, limit_cycles, report);
    count_launch();
    return cudaGetLastError();
}

}  // namespace a2sf

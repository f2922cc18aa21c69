// Self-test of the bounded waits: a kernel waits, with a short limit, on a shared-memory barrier that nothing
// ever completes.  The wait has to give up, raise its bit in the status word and let the kernel return, which
// is what every pipeline of the tensor-core kernels relies on when a copy or a partner never arrives.
#include "tc_common.cuh"
#include "tc_host.cuh"

namespace castling {
namespace tc {
namespace {

__global__ void __launch_bounds__(64)
selftest_wait_kernel(unsigned* status, unsigned long long limit_ns, unsigned* reached_end) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);   // one arrival expected; none will come
        abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    // warp 0 waits on the barrier itself; warp 1 waits too and must notice that warp 0 has given up (the CTA's
    // abort flag) or run into its own limit: either way every thread gets out
    const bool ok = mbar_wait(&bar, 0, &abort_flag, status, kStatusSelfTestTimeout, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0) *reached_end = ok ? 2u : 1u;
}

}  // namespace

cudaError_t launch_selftest_wait(unsigned* status, unsigned long long limit_ns, unsigned* reached_end, cudaStream_t st) {
    selftest_wait_kernel<<<1, 64, 0, st>>>(status, limit_ns, reached_end);
    return cudaGetLastError();
}

}  // namespace tc
}  // namespace castling

// rapid_selftest_bounded_wait: lets a caller (and the test-suite) see the library's time-out path work
// without anything being broken for it.  Every wait of the pipelined kernels goes through
// mbar_wait_bounded; here one thread waits, with a caller-chosen limit of at most a second, on a
// barrier that nothing ever arrives at, gives up when the limit has passed, and reports
// RAPID_ERR_TIMEOUT through the statistics block exactly as the real kernels do.  The kernel then
// ends normally: no trap, no fault, the context stays usable.
#include "rapid_common.cuh"
#include "tma_pipe.cuh"

namespace rapid {
namespace {

__global__ void __launch_bounds__(32) bounded_wait_probe_kernel(unsigned long long limit_ns, rapid_stats_t* stats) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);  // one arrival expected; none will come
        abort_flag = 0;
        mbar_init_fence();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const unsigned long long t0 = global_timer_ns();
        const bool got = mbar_wait_bounded(&bar, 0u, &abort_flag, limit_ns);
        const unsigned long long waited = global_timer_ns() - t0;
        rapid_stats_t st = {};
        st.status = (!got && abort_flag) ? (int)RAPID_ERR_TIMEOUT : (int)RAPID_OK;
        st.n_tokens = (long long)waited;  // nanoseconds the wait lasted
        *stats = st;
    }
}

}  // namespace
}  // namespace rapid

extern "C" rapid_status_t rapid_selftest_bounded_wait(uint64_t limit_ns, rapid_stats_t* stats, void* stream) {
    if (!stats || limit_ns == 0) return RAPID_ERR_INVALID_ARG;
    if (limit_ns > 1000000000ull) return RAPID_ERR_UNSUPPORTED;  // a self-test may hold an SM for a second at most
    rapid::bounded_wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(limit_ns, stats);
    return cudaGetLastError() == cudaSuccess ? RAPID_OK : RAPID_ERR_CUDA;
}

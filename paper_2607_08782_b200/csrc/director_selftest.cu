// Self-test of the failure-detection plumbing: the bounded mbarrier wait every pipeline role of the GEMM
// kernels uses, the abort flag it raises, and the sticky device status word the host reads afterwards.
//
// The kernel below waits - with the SAME helper, but a caller-chosen limit - on an mbarrier that nobody ever
// arrives at.  Nothing else is involved (no TMA, no tensor memory, no cluster), so the wait simply runs out: the
// helper returns false, the kernel records DIRECTOR_ERR_TIMEOUT and exits, and the context stays usable.
#include "director_common.cuh"
#include "director_umma.cuh"

namespace director {
namespace {

__global__ void __launch_bounds__(32)
bounded_wait_selftest_kernel(unsigned long long limit_ns, int32_t* status, unsigned long long* waited_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        umma::mbar_init(umma::smem_u32(&bar), 1);        // one arrival expected, none will come
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned long long t0 = umma::global_ns();
        const bool ok = umma::mbar_wait_limit(umma::smem_u32(&bar), 0u, &abort_flag, limit_ns);
        if (waited_ns) *waited_ns = umma::global_ns() - t0;
        // the same two steps the GEMM kernels take on their way out: the flag was raised by the helper ...
        if (!ok && abort_flag) director_set_status(status, DIRECTOR_ERR_TIMEOUT);
    }
    __syncthreads();
    // ... and every other role sees it on its next check and leaves as well
    if (threadIdx.x == 1 && abort_flag == 0) director_set_status(status, DIRECTOR_ERR_CUDA);
}

}  // namespace
}  // namespace director

extern "C" int director_selftest_bounded_wait(director_ctx* ctx, uint64_t limit_ns, uint64_t* waited_ns, void* stream) {
    using namespace director;
    if (ctx == nullptr) return DIRECTOR_ERR_INVALID_ARG;
    // a test must not park an SM for long: 1 us .. 100 ms
    if (limit_ns < 1000ull || limit_ns > 100000000ull) return DIRECTOR_ERR_INVALID_ARG;
    if (waited_ns != nullptr && (reinterpret_cast<uintptr_t>(waited_ns) & 7u)) return DIRECTOR_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    LaunchScope scope(ctx, st, "bounded_wait_selftest_kernel");
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>((unsigned long long)limit_ns, ctx->d_status,
                                                   reinterpret_cast<unsigned long long*>(waited_ns));
    return cuda_status(cudaGetLastError());
}

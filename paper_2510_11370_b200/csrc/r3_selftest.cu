// Self-test of the bounded wait that every pipeline of the tensor-core kernels is built on.
//
// The GEMM, weight-gradient and router kernels wait on shared-memory barriers for copies and
// tensor-core completions.  Each such wait gives up after a clock limit, raises the CTA's abort
// flag and reports R3_DEV_TIMEOUT through dev_status instead of spinning for ever.  In a healthy
// run no wait ever runs out, so this entry point exercises the path on purpose, in the one form
// that is harmless: a single small CTA waits on a barrier of its own that nothing will ever
// signal (no copy in flight, no tensor memory held), with a limit chosen by the caller.
#include "r3_common.cuh"
#include "r3_tc.cuh"

namespace r3 {

__global__ void __launch_bounds__(32)
bounded_wait_selftest_kernel(long long limit_clocks, int32_t* dev_status, int32_t* out) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    const uint32_t b = tc::smem_u32(&bar);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        tc::mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        // phase 0 of a fresh barrier with one expected arrival that never comes
        const bool ok = tc::mbar_wait(b, 0u, &abort_flag, dev_status, limit_clocks);
        out[0] = ok ? 1 : 0;
        out[1] = abort_flag;
        const long long waited = clock64() - t0;
        out[2] = (int32_t)(waited > 0x7fffffffLL ? 0x7fffffffLL : waited);
    }
    __syncwarp();
    // a second thread that arrives late finds the CTA aborting and leaves at once
    if (threadIdx.x == 1) out[3] = tc::mbar_wait(b, 0u, &abort_flag, dev_status, limit_clocks) ? 1 : 0;
}

}  // namespace r3

extern "C" r3_status r3_selftest_bounded_wait(int64_t limit_clocks, int32_t* dev_status,
                                              int32_t* out, void* stream) {
    // at most about a second at 2 GHz: a self-test must never look like a hang
    if (limit_clocks <= 0 || limit_clocks > 2000000000LL || !out) return R3_ERR_INVALID_ARG;
    r3::bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        (long long)limit_clocks, dev_status, out);
    return r3::launch_status();
}

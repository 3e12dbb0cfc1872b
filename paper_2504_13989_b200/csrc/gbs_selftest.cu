// gbs_selftest_wait_expiry: exercises the expiry path of the bounded barrier waits the tensor-core kernels use.
//
// Every wait in those kernels gives up after a time limit, records a code in a status word and returns, so that
// a lost arrival can never hang the device.  In normal operation that path does not run.  This self-test runs
// it on purpose, harmlessly: one thread waits, with a short limit, on a barrier nothing will ever arrive at;
// the wait must run out, the code must be recorded, the kernel must end and the context must stay usable.
// Nothing faults, traps or spins without a bound.
#include "gbs_internal.h"
#include "gbs_tc_common.cuh"

namespace {

constexpr int SELFTEST_CODE = 7;

// [0]: status word, [1]: nanoseconds the wait lasted, [2]: 1 if the wait (wrongly) reported success
__device__ unsigned long long g_selftest[3];

__global__ void k_wait_expiry(unsigned long long limit_ns)
{
    __shared__ unsigned long long bar;
    __shared__ int abort_flag;
    __shared__ int status;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        status = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const unsigned long long t0 = global_ns();
        const bool ok = mbar_try_wait(&bar, 0) || mbar_wait_slow(&abort_flag, &bar, 0, &status, SELFTEST_CODE, false, limit_ns);
        g_selftest[1] = global_ns() - t0;
        g_selftest[2] = ok ? 1ull : 0ull;
        g_selftest[0] = (unsigned long long)(unsigned)status + ((unsigned long long)(unsigned)abort_flag << 32);
    }
}

}  // namespace

extern "C" int gbs_selftest_wait_expiry(int limit_us, int* code_out, int* abort_out, int* waited_us_out)
{
    if (limit_us < 1 || limit_us > 1000000 || !code_out || !abort_out || !waited_us_out) return GBS_ERR_INVALID_ARG;
    k_wait_expiry<<<1, 32>>>((unsigned long long)limit_us * 1000ull);
    if (cudaGetLastError() != cudaSuccess) return GBS_ERR_CUDA;
    unsigned long long h[3] = {0, 0, 0};
    if (cudaMemcpyFromSymbol(h, g_selftest, sizeof(h)) != cudaSuccess) { cudaGetLastError(); return GBS_ERR_CUDA; }
    if (h[2] != 0) return GBS_ERR_CUDA;           // a wait on a barrier nobody arrives at may not succeed
    *code_out = (int)(h[0] & 0xffffffffull);
    *abort_out = (int)(h[0] >> 32);
    *waited_us_out = (int)(h[1] / 1000ull);
    return GBS_OK;
}

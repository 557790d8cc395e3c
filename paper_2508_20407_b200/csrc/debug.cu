// Diagnostic entry point: lets a test see the bounded-wait path of the tensor-core kernels run to its end without
// touching those kernels.  The kernel below waits, with the very routine they use (ptx::mbar_wait), on an mbarrier
// that nothing ever arrives on; the wait gives up after the given number of clocks, raises the CTA's abort flag,
// the other threads' waits then return at once, and the CTA reports TLIN_ERR_TIMEOUT through the status word exactly
// as the attention kernels do.  Nothing faults or hangs: the wait ends by itself.
#include "tlin_internal.h"
#include "sm100_ptx.cuh"

namespace tlin {
namespace {

__global__ void __launch_bounds__(64)
wait_expires_kernel(int* status, long long limit_cycles, long long* waited_cycles) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ptx::mbar_init(&bar, 1);
        ptx::fence_mbar_init();
    }
    __syncthreads();
    volatile int* abort_p = &abort_flag;
    const long long t0 = clock64();
    bool ok = true;
    if (threadIdx.x == 0) ok = ptx::mbar_wait(&bar, 0, abort_p, limit_cycles);      // phase 0 never completes
    __syncthreads();
    // every other role of a kernel finds the flag raised and leaves its own wait without serving the limit again
    if (threadIdx.x != 0) ok = ptx::mbar_wait(&bar, 0, abort_p, limit_cycles);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (waited_cycles != nullptr) *waited_cycles = clock64() - t0;
        if (abort_flag) atomicExch(status, (int)TLIN_ERR_TIMEOUT);
    }
    (void)ok;
}

}  // namespace
}  // namespace tlin

extern "C" int tlin_debug_wait_expires(long long limit_cycles, long long* waited_cycles, tlin_stream_t stream) {
    using namespace tlin;
    reset_launches();
    if (limit_cycles <= 0 || limit_cycles > 2000000000LL) return TLIN_ERR_INVALID_ARG;   // at most about a second
    int* status = status_word();
    if (!status) return TLIN_ERR_CUDA;
    wait_expires_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(status, limit_cycles, waited_cycles);
    TLIN_CUDA_CHECK(cudaGetLastError());
    count_launch();
    return TLIN_OK;
}

// A wait that runs out, on purpose and cheaply: the one way to see the library's handling of a
// device-side time-out (bounded wait -> outcome shared over a barrier -> bit in the context's error
// word -> eosq_check_status) without a kernel that hangs or faults.  The kernel waits on an mbarrier
// that nothing ever arrives at, with a poll budget the caller gives (a few milliseconds at most),
// through the same helper the tensor-core kernels wait with.
#include "eosq_common.cuh"
#include "eosq_sm100.cuh"

namespace eosq {

using namespace sm100;

namespace {

constexpr int ST_THREADS = 64;
constexpr int ST_ERR_TIMEOUT = 32;

__global__ void __launch_bounds__(ST_THREADS) wait_timeout_kernel(int *err, uint32_t polls) {
    __shared__ __align__(8) uint64_t never;
    __shared__ volatile int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&never, 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    const bool ok = mbar_wait_limited(&never, 0, &abort_flag, polls);
    // a wait ends per thread: the group learns of it together, as in the pipelines
    if (__syncthreads_or(!ok) && threadIdx.x == 0) atomicOr(err, ST_ERR_TIMEOUT);
}

}  // namespace

void launch_wait_timeout(int *err, uint32_t polls, cudaStream_t s) { wait_timeout_kernel<<<1, ST_THREADS, 0, s>>>(err, polls); }

}  // namespace eosq

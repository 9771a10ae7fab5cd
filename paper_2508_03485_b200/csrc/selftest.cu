// Diagnostic for the bounded device-side waits.  Every wait of the tensor-core kernels goes through
// lrq_tc::mbar_wait*, which gives up after a cycle budget, records a code in the library's status word and lets
// the kernel unwind.  This file holds the one kernel in which such a wait is made to run out on purpose, in the
// only safe form: a single CTA, one mbarrier on which nothing ever arrives, no TMA copy and no TMEM allocation in
// flight, and a budget of a fraction of a millisecond.  The kernel returns normally; the context stays usable.
#include "lrq_internal.cuh"
#include "tc_ptx.cuh"

namespace {
using namespace lrq_tc;

__global__ void __launch_bounds__(32)
wait_timeout_kernel(int* status, int code, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ volatile int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        mbar_init_fence();
    }
    __syncwarp();
    // the whole warp waits, as the decode warps of the contraction do; phase 0 never completes
    const bool ok = mbar_wait_warp<64>(smem_u32(&bar), 0, &abort_flag, status, code, limit_cycles);
    if (ok && threadIdx.x == 0 && status) atomicCAS(status, 0, -code);      // unreachable: the wait cannot succeed
}
}  // namespace

extern "C" lrq_status lrq_selftest_wait_timeout(long long limit_cycles, void* cuda_stream) {
    if (limit_cycles < 1 || limit_cycles > 100000000ll) return LRQ_ERR_INVALID_ARG;      // at most ~50 ms
    int* status = lrq_status_word();
    if (!status) return LRQ_ERR_CUDA;
    wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(status, LRQ_SELFTEST_WAIT_CODE, limit_cycles);
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}

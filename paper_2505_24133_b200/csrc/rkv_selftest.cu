// rkv_selftest_wait_expiry: runs the error path of the tcgen05 kernels' bounded waits on purpose, without any
// other work in flight.  One small block allocates tensor memory and sets up two mbarriers that nothing ever arrives
// at.  One thread waits on the first with the given (short) limit: the wait runs out, raises the block's abort flag
// and records RKV_ERR_TIMEOUT.  A thread of another warp waits on the second with the default limit: it must notice
// the abort flag and give up long before its own limit.  Both then leave through the same kind of exit the scoring
// kernels have (block barrier, tensor memory freed).  Nothing faults, traps or spins without a bound; the context
// stays usable.  See include/rkv.h for the contract.
#include "rkv_sm100.cuh"

namespace rkv {

namespace {

using namespace sm100;

constexpr uint32_t kSelfTestTmemCols = 32;

__global__ void __launch_bounds__(64, 1) wait_expiry_kernel(int32_t *status, unsigned long long *report_words,
                                                            long long limit_cycles, long long other_limit_cycles)
{
    __shared__ __align__(8) unsigned long long bars[2];
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t bar0 = smem_u32(&bars[0]), bar1 = smem_u32(&bars[1]);
    if (threadIdx.x == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar1, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_holder)), "r"(kSelfTestTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;

    if (warp == 0 && lane == 0) {
        // the wait that runs out: nobody ever arrives at bar0
        const ErrSink sink{status, report_words, limit_cycles};
        const long long t0 = clock64();
        const bool ok = mbar_wait(bar0, 0, abort_flag, sink);
        report_words[1] = (unsigned long long)(clock64() - t0);
        report_words[2] = ok ? 1ull : 0ull;
    } else if (warp == 1 && lane == 0) {
        // the wait that is called off: nobody arrives at bar1 either, but the abort flag ends it
        const ErrSink sink{status, report_words, other_limit_cycles};
        const long long t0 = clock64();
        const bool ok = mbar_wait(bar1, 0, abort_flag, sink);
        const long long waited = clock64() - t0;
        report_words[3] = (unsigned long long)waited;
        report_words[4] = (!ok && waited < other_limit_cycles) ? 1ull : 0ull;
    }
    __syncwarp();

    // the scoring kernels' common exit
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag) __nanosleep(20000);
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kSelfTestTmemCols) : "memory");
    }
    if (threadIdx.x == 0) report_words[5] = 1ull;       // the block reached its end
}

}  // namespace
}  // namespace rkv

extern "C" {

int rkv_selftest_wait_expiry(int32_t *device_status, unsigned long long *report_words, int64_t limit_cycles,
                             void *stream)
{
    using namespace rkv;
    if (!device_status || !report_words) return RKV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(report_words) & 7u) || (reinterpret_cast<uintptr_t>(device_status) & 3u))
        return RKV_ERR_INVALID_ARG;
    // between a thousand ticks and the default limit: the wait must run out quickly but not before it has polled
    if (limit_cycles < 1000 || limit_cycles > sm100::kWaitCycles) return RKV_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(report_words, 0, 8 * sizeof(unsigned long long), s);
    if (e != cudaSuccess) return RKV_ERR_CUDA;
    wait_expiry_kernel<<<1, 64, 0, s>>>(device_status, report_words, (long long)limit_cycles, sm100::kWaitCycles);
    return cudaGetLastError() == cudaSuccess ? RKV_OK : RKV_ERR_CUDA;
}

}  // extern "C"

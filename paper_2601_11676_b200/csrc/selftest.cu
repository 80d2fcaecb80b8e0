// halo_selftest_bounded_wait: shows, without hanging or faulting anything, what a device-side wait of this
// library does when the event it waits for never comes.  One thread block waits on an mbarrier phase that
// nothing completes and spins on a global flag that nothing sets, each with a short limit; both waits must
// give up, the kernel records where, raises HALO_DEV_TIMEOUT and returns normally, and the context stays usable.
#include "common.cuh"
#include "tma.cuh"

namespace halo {

__global__ void __launch_bounds__(128)
bounded_wait_selftest_kernel(const unsigned* __restrict__ never_set_flag, long long limit_cycles, uint32_t* report,
                             uint32_t* dev_status) {
    __shared__ uint64_t bar;
    __shared__ int give_up;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);   // one arrival expected; nobody will arrive
        give_up = 0;
        mbar_fence_init();
    }
    __syncthreads();
    // every thread waits on the mbarrier, as consumer threads of the FFN kernels do
    const bool completed = mbar_wait_bounded(&bar, 0, &give_up, limit_cycles);
    const int gave_up_threads = __syncthreads_count(!completed);
    if (threadIdx.x == 0) {
        // and one thread polls a global word, as the grid barrier and the selection flag are polled
        bool flag_seen = false;
        const long long t0 = clock64();
        while (clock64() - t0 <= limit_cycles) {
            if (ld_acquire_gpu(never_set_flag) != 0u) { flag_seen = true; break; }
        }
        report[0] = static_cast<uint32_t>(gave_up_threads);   // threads whose mbarrier wait ran out
        report[1] = flag_seen ? 0u : 1u;                      // 1 = the flag wait ran out
        if (gave_up_threads > 0 || !flag_seen) flag_status(dev_status, HALO_DEV_TIMEOUT);
    }
}

}  // namespace halo

extern "C" halo_status halo_selftest_bounded_wait(const uint32_t* never_set_flag, long long limit_cycles,
                                                  uint32_t* report, uint32_t* dev_status, void* stream) {
    if (!never_set_flag || !report || !dev_status) return HALO_ERR_ARG;
    if (limit_cycles <= 0 || limit_cycles > halo::kWaitLimitCycles) return HALO_ERR_ARG;
    halo::bounded_wait_selftest_kernel<<<1, 128, 0, static_cast<cudaStream_t>(stream)>>>(never_set_flag, limit_cycles,
                                                                                      report, dev_status);
    return cudaGetLastError() == cudaSuccess ? HALO_OK : HALO_ERR_CUDA;
}

// Self-test of the bounded device wait (not part of the paper's method): one CTA waits, with the
// helper every tensor-core kernel uses and a caller-given limit, on a barrier nothing ever arrives
// on, and reports the give-up the way those kernels do.
#include "tc_common.cuh"

namespace gc {
namespace {

__global__ void __launch_bounds__(64)
wait_limit_kernel(uint64_t limit_ns, int* dev_status, unsigned long long* waited_ns) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_s;
    volatile int* abort_flag = &abort_s;
    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // warp 0 runs out of time; warp 1 polls the same barrier and leaves through the abort flag
    const uint64_t t0 = global_ns();
    const bool ok = mbar_wait_limit(smem_u32(&bar), 0, abort_flag,
                                    threadIdx.x < 32 ? limit_ns : 8 * limit_ns + 1000000ull);
    const uint64_t waited = global_ns() - t0;
    __syncthreads();
    if (threadIdx.x == 0) {
        if (!ok && *abort_flag && dev_status) atomicOr(dev_status, GC_DEV_WAIT_LIMIT);
        if (waited_ns) *waited_ns = waited;
    }
}

}  // namespace
}  // namespace gc

extern "C" int gc_selftest_wait_limit(uint64_t limit_ns, int* dev_status,
                                      unsigned long long* waited_ns, void* cuda_stream) {
    if (!dev_status) return GC_ERR_NULL;
    if (limit_ns == 0 || limit_ns > 100000000ull) return GC_ERR_LIMIT;     // at most 0.1 s
    gc::wait_limit_kernel<<<1, 64, 0, static_cast<cudaStream_t>(cuda_stream)>>>(limit_ns, dev_status,
                                                                               waited_ns);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

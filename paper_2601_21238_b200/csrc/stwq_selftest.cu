// Self-tests that run on the device without touching the product kernels' data.
//
// stwq_selftest_wait_expiry: one CTA, no TMA, no tensor memory. It initialises an mbarrier that
// nothing ever arrives at and waits for it with the same bounded wait every GEMM kernel uses
// (stwq_ptx::mbar_wait). The wait must give up after the context's limit, set the CTA's abort
// flag, and the kernel must then report STWQ_DEV_TIMEOUT through the context's status word and
// return normally, exactly the path a product kernel takes when a copy or an MMA never completes.
// The kernel also records how long the wait lasted so that the host can check the limit was
// honoured. Nothing here can hang: the wait is bounded by the global timer.
#include "stwq_internal.cuh"
#include "stwq_ptx.cuh"

using namespace stwq_ptx;

namespace {

__global__ void wait_expiry_kernel(uint32_t* status, unsigned long long limit_ns, unsigned long long* waited_ns)
{
    __shared__ __align__(8) unsigned long long bar_storage;
    __shared__ uint32_t abort_flag;
    const uint32_t bar = smem_u32(&bar_storage);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);              // one arrival expected; nobody arrives
        abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned long long t0 = globaltimer_ns();
        const bool ok = mbar_wait(bar, 0u, &abort_flag, limit_ns);
        const unsigned long long dt = globaltimer_ns() - t0;
        if (waited_ns) *waited_ns = dt;
        if (!ok || abort_flag) atomicOr(status, STWQ_DEV_TIMEOUT);
    }
}

}  // namespace

extern "C" int stwq_selftest_wait_expiry(stwq_ctx* ctx, uint64_t* waited_ns_device, void* stream)
{
    if (!ctx) return STWQ_ERR_NULL;
    int prev = -1;
    const bool switched = cudaGetDevice(&prev) == cudaSuccess && prev != ctx->device;
    if (switched) cudaSetDevice(ctx->device);
    // never longer than a second here, whatever the context's limit says: this is a test of the
    // mechanism, not of patience
    unsigned long long limit_ns = (unsigned long long)ctx->wait_limit_ms * 1000000ull;
    if (limit_ns > 1000000000ull) limit_ns = 1000000000ull;
    wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        ctx->d_status, limit_ns, reinterpret_cast<unsigned long long*>(waited_ns_device));
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (switched) cudaSetDevice(prev);
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

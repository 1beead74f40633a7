// Peak probe for the int8 tensor path: what the tcgen05 kind::i8 pipe delivers on this GPU, at the
// clocks it holds, when nothing but the pipe is working. Used as the measured denominator beside
// the nominal int8 peak when a GEMM's "fraction of peak" is quoted.
//
// Every CTA pair issues the instruction the GEMM kernels issue (tcgen05.mma.cta_group::2.kind::i8,
// M 256, N 256, K 32, int32 accumulators in tensor memory) over operand tiles that stay resident in
// shared memory: no global traffic, no epilogue. The tiles hold pseudo-random bytes (an all-zero
// operand would draw less power and flatter the clock). Two accumulator buffers alternate; the
// issuing thread commits every eight k-blocks and stays at most two commits ahead of the pipe, so
// the queue is never empty and never unbounded. int32 sums wrap, which costs nothing and is never
// read. ops per launch = pairs * kblocks * 4 * (2 * 256 * 256 * 32).
#include "stwq_internal.cuh"
#include "stwq_ptx.cuh"

using namespace stwq_ptx;

namespace {

constexpr int kStageBytes = 128 * 128 + 128 * 128;   // this CTA's 128 rows of A and its half (128 rows) of B
constexpr int kProbeStages = 4;                       // 128 KB: also keeps the kernel at one CTA per SM, so that
                                                      // two CTAs never compete for one SM's tensor memory
constexpr int kProbeSmem = kProbeStages * kStageBytes + 64 + 1024;
constexpr int kGroup = 8;                             // k-blocks per commit

__global__ void __launch_bounds__(128, 1) probe_i8_kernel(int kblocks, uint32_t* status, unsigned long long limit_ns)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t bars = base + kProbeStages * kStageBytes;      // two commit barriers
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kProbeStages * kStageBytes + 32);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + kProbeStages * kStageBytes + 36);
    const uint32_t rank = cluster_ctarank();

    // operand bytes: a cheap integer hash of the address, different in every CTA
    uint32_t* words = reinterpret_cast<uint32_t*>(smem);
    for (int i = threadIdx.x; i < kProbeStages * kStageBytes / 4; i += blockDim.x) {
        uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x * 40503u + 12345u;
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        words[i] = h;
    }
    if (threadIdx.x == 0) {
        mbar_init(bars, 1);
        mbar_init(bars + 8u, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_async_smem();                                  // the tensor core reads shared memory through the async proxy
    if ((threadIdx.x >> 5) == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (threadIdx.x == 0 && rank == 0) {
        constexpr uint32_t idesc = make_idesc_i8(256, 256);
        bool ok = true;
        int group = 0;
        for (int kb = 0; kb < kblocks && ok; ++kb) {
            const int s = kb & (kProbeStages - 1);
            const uint32_t d_tmem = tmem_base + (uint32_t)(((kb / kGroup) & 1) * 256);
            const uint64_t a_desc = make_smem_desc(base + s * kStageBytes);
            const uint64_t b_desc = make_smem_desc(base + s * kStageBytes + 128 * 128);
#pragma unroll
            for (int k = 0; k < 4; ++k) tc_mma_i8_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, kb >= 2 * kGroup ? 1u : (uint32_t)((kb % kGroup) | k));
            if ((kb % kGroup) == kGroup - 1 || kb == kblocks - 1) {
                tc_commit_pair(bars + 8u * (group & 1));
                if (group >= 1) ok = mbar_wait(bars + 8u * ((group - 1) & 1), (uint32_t)((group - 1) >> 1) & 1u, abort_flag, limit_ns);
                ++group;
            }
        }
        if (ok && group >= 1) ok = mbar_wait(bars + 8u * ((group - 1) & 1), (uint32_t)((group - 1) >> 1) & 1u, abort_flag, limit_ns);
        if (!ok) atomicOr(status, STWQ_DEV_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    if ((threadIdx.x >> 5) == 0) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

}  // namespace

extern "C" int stwq_probe_int8_peak(stwq_ctx* ctx, int kblocks, int cta_pairs, int64_t* ops_per_launch, void* stream)
{
    if (!ctx) return STWQ_ERR_NULL;
    if (kblocks < 1 || kblocks > (1 << 22) || cta_pairs < 0) return STWQ_ERR_DIM;
    int prev = -1;
    const bool switched = cudaGetDevice(&prev) == cudaSuccess && prev != ctx->device;
    if (switched) cudaSetDevice(ctx->device);
    int rc = STWQ_OK;
    cudaError_t e = cudaSuccess;
    if (!ctx->probe_configured) {
        e = cudaFuncSetAttribute(probe_i8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem);
        if (e == cudaSuccess) ctx->probe_configured = 1;
    }
    if (e == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.blockDim = dim3(128, 1, 1);
        cfg.dynamicSmemBytes = kProbeSmem;
        cfg.stream = static_cast<cudaStream_t>(stream);
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int pairs = cta_pairs;
        if (pairs == 0) {                                 // as many pairs as can be resident at once
            cfg.gridDim = dim3((unsigned)(ctx->sm_count & ~1), 1, 1);
            int n = 0;
            e = cudaOccupancyMaxActiveClusters(&n, probe_i8_kernel, &cfg);
            pairs = (e == cudaSuccess && n > 0) ? (n < ctx->sm_count / 2 ? n : ctx->sm_count / 2) : 0;
        }
        if (pairs > ctx->sm_count / 2) pairs = ctx->sm_count / 2;
        if (e == cudaSuccess && pairs > 0) {
            cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
            e = cudaLaunchKernelEx(&cfg, probe_i8_kernel, kblocks, ctx->d_status,
                                   (unsigned long long)ctx->wait_limit_ms * 1000000ull);
            ctx->launches += 1;
            if (e == cudaSuccess) e = cudaGetLastError();
            if (ops_per_launch) *ops_per_launch = (int64_t)pairs * kblocks * 4ll * (2ll * 256 * 256 * 32);
        } else if (e == cudaSuccess) {
            e = cudaErrorLaunchOutOfResources;
        }
    }
    if (e != cudaSuccess) rc = stwq_cuda_fail(ctx, e);
    if (switched) cudaSetDevice(prev);
    return rc;
}

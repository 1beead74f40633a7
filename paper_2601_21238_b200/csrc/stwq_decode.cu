// Few-row (decode-step) variant of the quantized linear: M <= 256 rows, typically one raster-order
// decode step in which a whole batch advances one token position (Section 2: "one token at a
// time"). The arithmetic is that of qgemm2 (int8 x int8 -> int32 on the tensor cores, then the
// Appendix A.1 dequantizer with bias and activation); what differs is the decomposition. With so
// few rows the weights dominate the traffic (Wq is read once, 16.8 MB at the decode shapes):
//
//   * one CTA pair (tcgen05 cta_group::2) per work item; the pair's 256 accumulator rows cover
//     all of M, so Wq is staged exactly once on the whole GPU;
//   * a work item is a 128-column slice of N and, when N alone does not give one item per pair,
//     one of `ksplit` ranges of K (split-K);
//   * the two operands have separate 8-stage rings. Each ring has its own producer warp, and the
//     lanes of a producer warp issue the loads of different stages in the same instruction: one
//     thread alone needs about 160 ns per request (wait, expect, issue are a dependent chain),
//     2.6 us for a 16-k-block slab before its last byte is even asked for. The kernel can be
//     launched as a programmatic dependent of the quantize kernel: it then starts while that
//     kernel still runs, streams Wq, and only waits for the codes of X (griddepcontrol.wait)
//     before the first load of Xq, which comes from L2;
//   * two threads (in two warps) issue the MMAs, each into its own accumulator, because one thread
//     cannot issue tcgen05.mma faster than one per ~61 ns whatever the instruction's width, and a
//     256 x 128 x 32 instruction occupies the pipe for only 33 ns; the epilogue adds the accumulators;
//   * split-K partials are exact int32 sums. Every epilogue warp writes its 32 x 64 piece of the
//     pair's partial accumulator to scratch memory (lane-interleaved, so that each instruction
//     moves 512 contiguous bytes) and then bumps a counter that belongs to that piece; the warp
//     that arrives last (for that piece, across the K ranges) adds the pieces up and runs the
//     dequantize epilogue. Nobody waits for anybody: there is no spin on another CTA, the
//     reduction order does not matter for integers, and the last warp puts the counter back to
//     zero for the next call;
//   * the output leaves through shared memory (the Xq ring, idle by then) and TMA stores.
//
// Scratch (owned by the context): partials [item][rank][warp][16][32 lanes][4] int32 and one
// counter per (N slice, rank, warp). Calls that use it must be ordered on the GPU (one stream,
// or events), like every other use of a context's workspace.
#include <cuda.h>

#include "stwq_internal.cuh"
#include "stwq_ptx.cuh"

using namespace stwq_ptx;

namespace {

constexpr int kBM = 128;       // rows per CTA (256 per pair)
constexpr int kBK = 128;       // bytes of K per k-block
constexpr int kBN = 128;       // columns per work item
constexpr int kEpi = 8;        // epilogue warps per CTA: 4 lane quarters x 2 column halves
constexpr int kStagesA = 8;    // Xq ring (128 KB; doubles as output staging)
constexpr int kStagesB = 8;    // Wq ring (64 KB)
constexpr int kIssuers = 2;            // MMA-issuing threads, one accumulator each (4 measured no faster: with 2 the
                                       // loop already runs at what L2 delivers, and every accumulator costs the epilogue a read)
constexpr int kFirstEpiWarp = 2 + kIssuers;   // warps: 0 Wq producer, 1 Xq producer, 2.. MMA issuers, then the epilogue
constexpr int kThreads = 32 * (kFirstEpiWarp + kEpi);
constexpr int kPieceInts = 2 * 32 * 32;   // one warp's piece of a partial: 32 rows x 64 columns

struct DecParams {
    int64_t M;
    int N, K, P;
    const int32_t* pos_ids;
    const float* s_w;
    const float* s_tok;
    const float* bias;
    int ksplit, kb_per_split, num_kb;
    int32_t* partial;
    uint32_t* counters;
    uint32_t* status;
    unsigned long long wait_limit_ns;
};

struct SmemDec {
    static constexpr int kABytes = kBM * kBK;               // 16 KB
    static constexpr int kBBytes = (kBN / 2) * kBK;         // 8 KB: this CTA's half of the Wq slice
    static constexpr int kOffB = kStagesA * kABytes;
    static constexpr int kOffScale = kOffB + kStagesB * kBBytes; // per epilogue warp: s_w and bias of its 64 columns
    static constexpr int kOffBars = kOffScale + kEpi * 2 * 64 * 4;
    static constexpr int kNumBars = 2 * kStagesA + 2 * kStagesB + 1;
    static constexpr int kOffMisc = kOffBars + kNumBars * 8;
    static constexpr int kTotal = kOffMisc + 16;
    static constexpr int kDynamic = kTotal + 1024;
    static_assert(kDynamic <= 227 * 1024, "shared memory budget");
    static_assert(kStagesA * kABytes >= kEpi * 8192, "the Xq ring doubles as output staging");
    static_assert(kIssuers * kBN <= 512 && kStagesA % kIssuers == 0 && kStagesB % kIssuers == 0, "issuers own fixed ring stages");
};

__device__ __forceinline__ uint4 ld_cg_v4(const void* p)
{
    uint4 v;
    asm volatile("ld.global.cg.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
// Let the next kernel in the stream start early / wait for the previous one (programmatic
// dependent launch). Both are no-ops for a kernel that was launched the ordinary way.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <int OUT, int ACT>
__global__ void __launch_bounds__(kThreads, 1)
decode_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
              const __grid_constant__ CUtensorMap tmY, const DecParams p)
{
    using L = SmemDec;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);

    const uint32_t bars = base + L::kOffBars;
    auto bar_full_a = [&](int s) { return bars + 8u * s; };
    auto bar_empty_a = [&](int s) { return bars + 8u * (kStagesA + s); };
    auto bar_full_b = [&](int s) { return bars + 8u * (2 * kStagesA + s); };
    auto bar_empty_b = [&](int s) { return bars + 8u * (2 * kStagesA + kStagesB + s); };
    const uint32_t bar_tfull = bars + 8u * (2 * kStagesA + 2 * kStagesB);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kOffMisc);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::kOffMisc + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may queue up behind this grid
    const uint32_t rank = cluster_ctarank();            // 0 = even CTA = MMA leader
    const int item = blockIdx.x >> 1;
    const int nt = item / p.ksplit;                     // which 128-column slice of N
    const int ks = item % p.ksplit;                     // which range of K
    const int kb0 = ks * p.kb_per_split;
    const int kb1 = min(kb0 + p.kb_per_split, p.num_kb);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStagesA; ++s) {
            mbar_init(bar_full_a(s), 1);                 // leader's producer arrives with expect_tx
            mbar_init(bar_empty_a(s), 1);                // multicast commit
        }
        for (int s = 0; s < kStagesB; ++s) {
            mbar_init(bar_full_b(s), 1);
            mbar_init(bar_empty_b(s), 1);
        }
        mbar_init(bar_tfull, kIssuers);                  // one commit from each MMA issuer
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    __syncthreads();
    // The cluster barrier is split: arrive now, wait just before the first access to the peer
    // (a load that signals the leader's barrier, a commit that arrives in both CTAs). Tensor memory
    // is allocated in between, and the producers do not wait for it at all.
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kIssuers * kBN)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        tc_fence_before();
    }
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");        // barriers of both CTAs are initialised
    const unsigned long long limit = p.wait_limit_ns;
    uint32_t tmem_base = 0;
    if (warp >= 2) {
        // the tensor-memory address, published by warp 2, is needed by warp 2 and the epilogue warps only
        asm volatile("bar.sync 1, %0;" ::"r"(kThreads - 64) : "memory");
        tc_fence_after();
        tmem_base = *tmem_slot;
    }

    if (warp == 0) {
        // ------------------------------------------------------------------ Wq producer
        // Sixteen lanes, one per stage of the Wq ring, issue their loads in the same instruction:
        // a single thread needs about 160 ns per request (wait, expect, issue form a dependent
        // chain), which for the 16 k-blocks of a slab is 2.6 us before the last byte is even asked for.
        if (lane < kStagesB) {
            bool ok = true;
            const uint32_t full0 = mapa_u32(bar_full_b(0), 0);
            const int n0 = nt * kBN + (int)rank * (kBN / 2);
            const int s = lane;
            int it = lane;
            for (; kb0 + it < kb1; it += kStagesB) {
                const uint32_t ph = (uint32_t)(it / kStagesB) & 1u;
                if (!mbar_wait(bar_empty_b(s), ph ^ 1u, abort_flag, limit)) { ok = false; break; }
                if (rank == 0) mbar_expect_tx(bar_full_b(s), 2 * L::kBBytes);
                tma_load_2d_pair(base + L::kOffB + s * L::kBBytes, &tmB, (kb0 + it) * kBK, n0, full0 + 8u * s);
            }
            ok = __all_sync((1u << kStagesB) - 1u, ok);
            if (!ok && rank == 0 && it >= kStagesB) {     // giving up: this lane's last load may still be in flight
                const int j = it - kStagesB;
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(bar_full_b(s), (uint32_t)(j / kStagesB) & 1u))
                    if (globaltimer_ns() - t0 > limit) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ Xq producer
        if (lane < kStagesA) {
            grid_dependency_wait();                      // the codes of X come from the previous kernel
            bool ok = true;
            const uint32_t full0 = mapa_u32(bar_full_a(0), 0);
            const int m0 = (int)rank * kBM;
            const int s = lane;
            int it = lane;
            for (; kb0 + it < kb1; it += kStagesA) {
                const uint32_t ph = (uint32_t)(it / kStagesA) & 1u;
                if (!mbar_wait(bar_empty_a(s), ph ^ 1u, abort_flag, limit)) { ok = false; break; }
                if (rank == 0) mbar_expect_tx(bar_full_a(s), 2 * L::kABytes);
                tma_load_2d_pair(base + s * L::kABytes, &tmA, (kb0 + it) * kBK, m0, full0 + 8u * s);
            }
            ok = __all_sync((1u << kStagesA) - 1u, ok);
            if (!ok && rank == 0 && it >= kStagesA) {
                const int j = it - kStagesA;
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(bar_full_a(s), (uint32_t)(j / kStagesA) & 1u))
                    if (globaltimer_ns() - t0 > limit) break;
            }
        }
    } else if (warp < kFirstEpiWarp) {
        // ------------------------------------------------------------------ MMA issuers (leader)
        // One thread cannot issue tcgen05.mma faster than about one per 61 ns, whatever the
        // instruction's shape, and a 256 x 128 x 32 instruction keeps the pipe busy for only 33 ns.
        // So kIssuers threads issue, each in a warp of its own: issuer i takes the k-blocks i,
        // i + kIssuers, ... into accumulator i (tensor-memory columns 128 i ..); the epilogue adds
        // the accumulators (int32, exact). Each issuer releases the ring stages of its own k-blocks.
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = make_idesc_i8(2 * kBM, kBN);
            const int who = warp - 2;
            const uint32_t d_tmem = tmem_base + (uint32_t)(who * kBN);
            bool ok = true;
            for (int it = who; kb0 + it < kb1; it += kIssuers) {
                const int sa = it % kStagesA, sb = it % kStagesB;
                if (!mbar_wait(bar_full_b(sb), (uint32_t)(it / kStagesB) & 1u, abort_flag, limit)) { ok = false; break; }
                if (!mbar_wait(bar_full_a(sa), (uint32_t)(it / kStagesA) & 1u, abort_flag, limit)) { ok = false; break; }
                tc_fence_after();
                const uint64_t a_desc = make_smem_desc(base + sa * L::kABytes);
                const uint64_t b_desc = make_smem_desc(base + L::kOffB + sb * L::kBBytes);
#pragma unroll
                for (int k = 0; k < kBK / 32; ++k)
                    tc_mma_i8_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (it >= kIssuers || k != 0) ? 1u : 0u);
                tc_commit_pair(bar_empty_a(sa));
                tc_commit_pair(bar_empty_b(sb));
            }
            if (ok) tc_commit_pair(bar_tfull);
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int ew = warp - kFirstEpiWarp;              // 0..7
        const int q = warp & 3;                           // TMEM lane quarter
        const int sub = ew >> 2;                          // column half of the slice
        const int n0 = nt * kBN + sub * 64;               // first column of this warp's piece
        const int row0 = (int)rank * kBM + q * 32;
        const int64_t row = (int64_t)row0 + lane;
        float* my_sw = reinterpret_cast<float*>(smem + L::kOffScale) + ew * 128;
        float* my_bias = my_sw + 64;
        float st = 0.0f;
        if (OUT != STWQ_OUT_INT32) {
            for (int i = lane; i < 64; i += 32) {
                const int col = n0 + i;
                my_sw[i] = col < p.N ? __ldg(p.s_w + col) : 0.0f;
                my_bias[i] = (p.bias != nullptr && col < p.N) ? __ldg(p.bias + col) : 0.0f;
            }
            if (row < p.M) {
                const int pos = p.pos_ids[row];
                if (pos >= 0 && pos < p.P) st = p.s_tok[pos];
                else if (item == 0 && sub == 0) atomicOr(p.status, STWQ_DEV_POS_RANGE);
            }
            __syncwarp();
        }
        bool ok = mbar_wait(bar_tfull, 0u, abort_flag, limit);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(sub * 64);
            // This row's 64 accumulators are handled as two halves of 32 columns, one after the other.
            // 32 columns of this row: the sum of the issuers' accumulators (accumulator i exists only
            // if the item has more than i k-blocks)
            const int n_acc = min(kb1 - kb0, kIssuers);
            auto load_acc = [&](uint32_t addr, uint32_t (&r)[32]) {
                tmem_ld32(addr, r);
                tmem_ld_wait();
                for (int a = 1; a < n_acc; ++a) {
                    uint32_t r2[32];
                    tmem_ld32(addr + (uint32_t)(a * kBN), r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] += r2[j];
                }
            };
            bool finish = true;
            if (p.ksplit > 1) {
                // publish this warp's piece of the partial sum, then see who is last
                int32_t* piece = p.partial + ((((size_t)nt * p.ksplit + ks) * 2 + rank) * kEpi + ew) * kPieceInts;
#pragma unroll 1
                for (int h = 0; h < 2; ++h) {
                    uint32_t r[32];
                    load_acc(taddr + 32u * h, r);
#pragma unroll
                    for (int g = 0; g < 8; ++g) st_global_v4(piece + ((size_t)(h * 8 + g) * 32 + lane) * 4, r + g * 4);
                }
                __threadfence();
                __syncwarp();
                uint32_t* counter = p.counters + ((size_t)nt * 2 + rank) * kEpi + ew;
                uint32_t old = 0;
                if (lane == 0) {
                    old = atomicAdd(counter, 1u);
                    if (old == (uint32_t)p.ksplit - 1u) *counter = 0u;    // everyone has arrived: ready for the next call
                }
                old = __shfl_sync(0xffffffffu, old, 0);
                finish = (old == (uint32_t)p.ksplit - 1u);
                if (finish) __threadfence();
            }
            if (finish) {
                // 32 rows x 64 columns -> this warp's staging tiles (8 KB of the idle Xq ring): one
                // 32 x 128-byte tile for bf16, two for fp32 / int32, 128-byte swizzled as TMA expects
                const uint32_t stage = base + (uint32_t)ew * 8192u;
                const uint64_t st2 = pack_f2(st, st);
#pragma unroll 1
                for (int h = 0; h < 2; ++h) {             // two halves of 32 columns
                    uint32_t r[32];
                    if (p.ksplit > 1) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = 0u;
                        for (int s2 = 0; s2 < p.ksplit; ++s2) {
                            const int32_t* src = p.partial + ((((size_t)nt * p.ksplit + s2) * 2 + rank) * kEpi + ew) * kPieceInts;
#pragma unroll
                            for (int g = 0; g < 8; ++g) {
                                const uint4 a = ld_cg_v4(src + ((size_t)(h * 8 + g) * 32 + lane) * 4);
                                r[g * 4 + 0] += a.x; r[g * 4 + 1] += a.y; r[g * 4 + 2] += a.z; r[g * 4 + 3] += a.w;
                            }
                        }
                    } else {
                        load_acc(taddr + 32u * h, r);
                    }
                    const float* hsw = my_sw + h * 32;
                    const float* hbi = my_bias + h * 32;
                    if (OUT == STWQ_OUT_BF16) {
                        uint32_t w[16];
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            const uint64_t sw = pack_f2(hsw[j], hsw[j + 1]);
                            const uint64_t bi = pack_f2(hbi[j], hbi[j + 1]);
                            uint64_t z = fma_f2(pack_f2((float)(int32_t)r[j], (float)(int32_t)r[j + 1]), mul_f2(st2, sw), bi);
                            z = apply_act_f2<ACT>(z);
                            float v0, v1;
                            unpack_f2(z, v0, v1);
                            w[j / 2] = pack_bf16(v0, v1);
                        }
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const uint32_t piece16 = (uint32_t)((h * 4 + g) ^ (lane & 7));
                            st_shared_v4(stage + (uint32_t)lane * 128u + piece16 * 16u, w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3]);
                        }
                    } else {
                        if (OUT != STWQ_OUT_INT32) {
#pragma unroll
                            for (int j = 0; j < 32; j += 2) {
                                const uint64_t sw = pack_f2(hsw[j], hsw[j + 1]);
                                const uint64_t bi = pack_f2(hbi[j], hbi[j + 1]);
                                const uint64_t z = fma_f2(pack_f2((float)(int32_t)r[j], (float)(int32_t)r[j + 1]), mul_f2(st2, sw), bi);
                                float v0, v1;
                                unpack_f2(z, v0, v1);
                                r[j] = __float_as_uint(apply_act<ACT>(v0));
                                r[j + 1] = __float_as_uint(apply_act<ACT>(v1));
                            }
                        }
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            const uint32_t piece16 = (uint32_t)(g ^ (lane & 7));
                            st_shared_v4(stage + (uint32_t)h * 4096u + (uint32_t)lane * 128u + piece16 * 16u, r[4 * g], r[4 * g + 1],
                                         r[4 * g + 2], r[4 * g + 3]);
                        }
                    }
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0 && row0 < p.M) {
                    if (OUT == STWQ_OUT_BF16) {
                        if (n0 < p.N) tma_store_2d(&tmY, stage, n0, row0);
                    } else {
                        if (n0 < p.N) tma_store_2d(&tmY, stage, n0, row0);
                        if (n0 + 32 < p.N) tma_store_2d(&tmY, stage + 4096u, n0 + 32, row0);
                    }
                    bulk_commit();
                    bulk_wait_read0();                    // the staging tiles have been read before the CTA may exit;
                                                          // the writes themselves complete with the grid
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, STWQ_DEV_TIMEOUT);
    cluster_sync_all();                                  // no remote arrive or multicast still to land
    tc_fence_after();
    if (warp == 2) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kIssuers * kBN) : "memory");
    }
}

template <int OUT, int ACT>
int launch_variant(stwq_ctx* ctx, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmY,
                   const DecParams& p, int items, bool dependent, cudaStream_t st)
{
    auto kern = decode_kernel<OUT, ACT>;
    const uint64_t bit = 1ull << (OUT * 4 + ACT);
    if (!(ctx->configured_decode & bit)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemDec::kDynamic);
        if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
        ctx->configured_decode |= bit;
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // may start while the previous kernel of the stream (the quantize kernel) still runs
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)(2 * items), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = SmemDec::kDynamic;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmY, p);
    ctx->launches += 1;
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

// How a few-row problem is cut into work items.
struct DecPlan {
    int num_kb, tiles_n, ksplit, kb_per_split, items;
};
DecPlan plan_decode(const stwq_ctx* ctx, int K, int N)
{
    DecPlan d;
    d.num_kb = (K + kBK - 1) / kBK;
    d.tiles_n = (N + kBN - 1) / kBN;
    // One work item per CTA pair if N allows; otherwise K may be split so that more pairs have
    // work. The exchange of partial sums costs 2-3 us, so this pays only for long K: measured
    // (M 256, weights from HBM, N 1024-4096) no split is best up to K 2048 (7.7-11.3 us against
    // 10.3-13.0 us with two ranges), and from K 4096 on two to four ranges of at least eight
    // k-blocks each (K 8192, N 1024: 27.2 us whole, 17.2 us in four ranges, 18.3 in eight).
    const int pairs = ctx->sm_count / 2;
    int ksplit = 1;
    if (d.tiles_n * 4 < pairs * 3 && d.num_kb >= 32) {
        ksplit = pairs / d.tiles_n;
        if (ksplit > d.num_kb / 8) ksplit = d.num_kb / 8;
        if (ksplit > 4) ksplit = 4;
        if (ksplit < 1) ksplit = 1;
    }
    if (ctx->force_ksplit > 0) ksplit = ctx->force_ksplit < d.num_kb ? ctx->force_ksplit : d.num_kb;
    if (ctx->force_ksplit < 0) ksplit = 1;
    d.kb_per_split = (d.num_kb + ksplit - 1) / ksplit;
    d.ksplit = (d.num_kb + d.kb_per_split - 1) / d.kb_per_split;      // every range holds at least one k-block
    d.items = d.tiles_n * d.ksplit;
    return d;
}

}  // namespace

// Bytes of split-K scratch the few-row path wants for a [<= 256, K] x [N, K] problem (0: no split).
size_t stwq_decode_split_bytes(const stwq_ctx* ctx, int K, int N)
{
    const DecPlan d = plan_decode(ctx, K, N);
    return d.ksplit > 1 ? (size_t)d.items * 2 * kEpi * kPieceInts * sizeof(int32_t) : 0;
}

// Scratch for split-K (shared by the few-row kernel and the tail of the tiled GEMM): a fixed
// region of kSplitCounters arrival counters, zero between calls because the last arriver resets
// its counter, followed by room for the int32 partial sums.
int stwq_split_ws(stwq_ctx* ctx, size_t partial_bytes, size_t n_counters, uint32_t** counters, int32_t** partial,
                  cudaStream_t st)
{
    constexpr size_t kSplitCounters = 16384;
    constexpr size_t counter_bytes = kSplitCounters * sizeof(uint32_t);
    if (n_counters > kSplitCounters) return STWQ_ERR_DIM;
    int rc = stwq_ensure_ws(ctx, &ctx->ws_dec, &ctx->ws_dec_bytes, partial_bytes + counter_bytes, st, counter_bytes);
    if (rc != STWQ_OK) return rc;
    *counters = reinterpret_cast<uint32_t*>(ctx->ws_dec);
    *partial = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(ctx->ws_dec) + counter_bytes);
    return STWQ_OK;
}

int stwq_launch_decode(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K, int N,
                       const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* bias,
                       int act, int out_dtype, void* Y, bool after_quantize, cudaStream_t st)
{
    const int elem = out_dtype == STWQ_OUT_BF16 ? 2 : 4;
    // the TMA store of Y needs 16-byte row pitches; otherwise the general tiled kernel runs
    if (M > 2 * kBM || ((int64_t)N * elem) % 16 != 0)
        return stwq_launch_qgemm(ctx, Xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype, Y, st);

    DecParams p;
    p.M = M; p.N = N; p.K = K; p.P = P;
    p.pos_ids = pos_ids; p.s_w = s_w; p.s_tok = s_tok; p.bias = bias;
    const DecPlan plan = plan_decode(ctx, K, N);
    p.num_kb = plan.num_kb;
    p.kb_per_split = plan.kb_per_split;
    p.ksplit = plan.ksplit;
    const int tiles_n = plan.tiles_n;
    const int items = plan.items;
    p.partial = nullptr;
    p.counters = nullptr;
    if (p.ksplit > 1) {
        int rc = stwq_split_ws(ctx, (size_t)items * 2 * kEpi * kPieceInts * sizeof(int32_t), (size_t)tiles_n * 2 * kEpi,
                               &p.counters, &p.partial, st);
        if (rc == STWQ_ERR_DIM)                            // more N slices than counters: no split-K path
            return stwq_launch_qgemm(ctx, Xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype, Y, st);
        if (rc != STWQ_OK) return rc;
    }
    p.status = ctx->d_status;
    p.wait_limit_ns = (unsigned long long)ctx->wait_limit_ms * 1000000ull;

    CUtensorMap tmA, tmB, tmY;
    int rc = stwq_encode_2d(ctx, &tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Xq, M, K, kBK, kBM);
    if (rc != STWQ_OK) return rc;
    rc = stwq_encode_2d(ctx, &tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, N, K, kBK, kBN / 2);
    if (rc != STWQ_OK) return rc;
    if (out_dtype == STWQ_OUT_BF16)
        rc = stwq_encode_2d(ctx, &tmY, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, M, N, 64, 32);
    else if (out_dtype == STWQ_OUT_F32)
        rc = stwq_encode_2d(ctx, &tmY, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, Y, M, N, 32, 32);
    else
        rc = stwq_encode_2d(ctx, &tmY, CU_TENSOR_MAP_DATA_TYPE_INT32, 4, Y, M, N, 32, 32);
    if (rc != STWQ_OK) return rc;
    const bool dependent = after_quantize && ctx->debug != 5;   // tuning: 5 = ordinary launch

#define STWQ_CASE(O, A) \
    if (out_dtype == O && act == A) return launch_variant<O, A>(ctx, tmA, tmB, tmY, p, items, dependent, st);
    if (out_dtype == STWQ_OUT_INT32) return launch_variant<STWQ_OUT_INT32, STWQ_ACT_NONE>(ctx, tmA, tmB, tmY, p, items, dependent, st);
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_NONE)
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_GELU_ERF)
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_GELU_TANH)
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_GELU_FAST)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_NONE)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_GELU_ERF)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_GELU_TANH)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_GELU_FAST)
#undef STWQ_CASE
    return STWQ_ERR_BITS;
}

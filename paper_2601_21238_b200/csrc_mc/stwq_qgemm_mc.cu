// qgemm_mc: the int8 GEMM + dequantize epilogue of qgemm2 with the Xq operand shared between two
// CTA pairs of a cluster (single-GPU builds only; this file is left out of multi-GPU runs and the
// library then uses qgemm2 for every problem).
//
//   acc[m,n] = sum_k Xq[m,k] * Wq[n,k]                              (Section 3, Y = X W on codes)
//   Y[m,n]   = act( float(acc) * (s_tok[pos[m]] * s_w[n]) + bias[n] )   (Appendix A.1 dequantizer)
//
// With all 74 pairs running, the main loop of qgemm2 is bound by what L2 can deliver to the SMs
// (32 KB per SM and k-block, about 11 TB/s over the chip). Here a cluster of four CTAs = two
// pairs computes two neighbouring 256 x 256 tiles of the same 256 rows: pair 0 the tile of column
// block 2j, pair 1 that of 2j + 1. Both need the same rows of Xq. CTA (pair p, rank r) fetches
// 64 of rank r's 128 rows and TMA delivers them into the shared memory of both CTAs of rank r
// (cluster multicast), so every byte of Xq leaves L2 once per two pairs: 24 KB per SM and
// k-block instead of 32 KB. Wq is staged as in qgemm2, each CTA its half of its pair's slice.
//
// Barriers per stage s:
//   empty[s]  in every CTA, count 2: the MMA issuers of both pairs commit to it in all four CTAs
//             (a stage may be overwritten only when neither pair reads it any more, because the
//             partner pair's CTA writes into it too)
//   full[s]   leader (rank 0) CTA: count 2 = its producer's arrive.expect_tx (both CTAs' Wq bytes
//             + its own 16 KB of Xq) and the relay arrive of the rank-1 CTA;
//             rank-1 CTA: count 1 = its producer's arrive.expect_tx (its own 16 KB of Xq); a relay
//             thread waits for it and arrives on the leader's full[s]
// Accumulator barriers, epilogue and time-outs are those of qgemm2.
#include <cuda.h>

#include "stwq_internal.cuh"
#include "stwq_ptx.cuh"

using namespace stwq_ptx;

namespace {

constexpr int kBM = 128;      // rows per CTA
constexpr int kBK = 128;      // bytes of K per stage
constexpr int BN = 256;       // columns per pair tile

struct McParams {
    int64_t M;
    int N, K, P;
    const int32_t* pos_ids;
    const float* s_w;
    const float* s_tok;
    const float* bias;
    int super_n;               // pairs of tile columns
    int num_units;             // tiles_m * super_n
    int num_kb;
    uint32_t* status;
    unsigned long long wait_limit_ns;
    void* Y;
    int y_vec32;
};

template <int STAGES, int EPI, int STORE>
struct SmemMc {
    static constexpr int kABytes = kBM * kBK;               // 16 KB: 128 rows of Xq (two halves of 64)
    static constexpr int kBBytes = (BN / 2) * kBK;          // 16 KB: this CTA's half of the Wq slice
    static constexpr int kOffB = STAGES * kABytes;
    static constexpr int kOffStage = STAGES * (kABytes + kBBytes);
    static constexpr int kOffScale = kOffStage + (STORE == 0 ? EPI * 8192 : 0);
    static constexpr int kOffBars = kOffScale + 2 * BN * 4 * 4;   // per epilogue warp: s_w and bias of its columns
    static constexpr int kNumBars = 2 * STAGES + 4;
    static constexpr int kOffMisc = kOffBars + kNumBars * 8;
    static constexpr int kTotal = kOffMisc + 16;
    static constexpr int kDynamic = kTotal + 1024;
    static_assert(kDynamic <= 227 * 1024, "shared memory budget");
};

// TMA tile load delivered to the same shared-memory offset of every CTA named in `mask`; each
// destination's barrier at the offset of `bar` is credited with the bytes it received.
__device__ __forceinline__ void tma_load_2d_mc(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar,
                                               uint16_t mask)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster "
        "[%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar), "h"(mask)
        : "memory");
}
// Arrive (once all MMAs issued so far have completed) on the barrier at this offset in the CTAs of `mask`.
__device__ __forceinline__ void tc_commit_mask(uint32_t bar, uint16_t mask)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"(mask)
        : "memory");
}

template <int STAGES, int EPI, int OUT, int ACT, int STORE>
__global__ void __launch_bounds__(64 + 32 * EPI, 1)
qgemm_mc_kernel(const __grid_constant__ CUtensorMap tmAh, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmY, const McParams p)
{
    using L = SmemMc<STAGES, EPI, STORE>;
    constexpr int kChunkCols = (OUT == STWQ_OUT_BF16) ? 64 : 32;
    constexpr int kChunks = BN / kChunkCols;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);

    const uint32_t bars = base + L::kOffBars;
    auto bar_full = [&](int s) { return bars + 8u * s; };
    auto bar_empty = [&](int s) { return bars + 8u * (STAGES + s); };
    auto bar_tfull = [&](int a) { return bars + 8u * (2 * STAGES + a); };
    auto bar_tempty = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kOffMisc);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::kOffMisc + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const uint32_t crank = cluster_ctarank();            // 0..3
    const uint32_t rank = crank & 1u;                    // within the pair; 0 = MMA leader
    const uint32_t pi = crank >> 1;                      // pair within the cluster
    const uint32_t leader = crank & ~1u;                 // cluster rank of this pair's leader
    const int cluster_id = blockIdx.x >> 2;
    const int num_clusters = gridDim.x >> 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full(s), rank == 0 ? 2 : 1);
            mbar_init(bar_empty(s), 2);                  // one commit from each pair's issuer
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull(a), 1);
            mbar_init(bar_tempty(a), 2 * EPI);           // every epilogue warp of both CTAs of the pair
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(2 * BN)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                  // barriers of all four CTAs are initialised
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const unsigned long long limit = p.wait_limit_ns;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (every CTA)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            const uint32_t full_leader0 = mapa_u32(bar_full(0), leader);
            const uint16_t mask = (uint16_t)((1u << rank) | (1u << (2u + rank)));   // the two CTAs of this rank
            const uint32_t own_bytes = rank == 0 ? (uint32_t)(2 * L::kBBytes + L::kABytes) : (uint32_t)L::kABytes;
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int u = cluster_id; ok && u < p.num_units; u += num_clusters) {
                const int mt = u / p.super_n;
                const int nt = 2 * (u % p.super_n) + (int)pi;
                const int a_row = mt * (2 * kBM) + (int)rank * kBM + (int)pi * 64;   // the 64 rows this CTA fetches
                const int n0 = nt * BN + (int)rank * (BN / 2);                         // may lie beyond N: zero fill
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(bar_empty(s), ph ^ 1u, abort_flag, limit)) { ok = false; break; }
                    mbar_expect_tx(bar_full(s), own_bytes);
                    tma_load_2d_pair(base + L::kOffB + s * L::kBBytes, &tmB, kb * kBK, n0, full_leader0 + 8u * s);
                    tma_load_2d_mc(base + s * L::kABytes + pi * 8192u, &tmAh, kb * kBK, a_row, bar_full(s), mask);
                }
            }
            if (!ok) {
                // loads in flight into this CTA's memory are awaited (bounded) before it may exit
                const uint32_t first = it > (uint32_t)STAGES ? it - STAGES : 0u;
                for (uint32_t j = first; j < it; ++j) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(bar_full(j % STAGES), (j / STAGES) & 1u))
                        if (globaltimer_ns() - t0 > limit) break;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // -------------------------------------------------------------- MMA issuer (pair leader)
            constexpr uint32_t idesc = make_idesc_i8(2 * kBM, BN);
            const uint16_t pair_mask = (uint16_t)(3u << (2u * pi));
            uint32_t it = 0, t = 0;
            bool ok = true;
            for (int u = cluster_id; ok && u < p.num_units; u += num_clusters, ++t) {
                const int acc = t & 1;
                const uint32_t aph = (t >> 1) & 1u;
                if (!mbar_wait(bar_tempty(acc), aph ^ 1u, abort_flag, limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(bar_full(s), ph, abort_flag, limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_smem_desc(base + s * L::kABytes);
                    const uint64_t b_desc = make_smem_desc(base + L::kOffB + s * L::kBBytes);
#pragma unroll
                    for (int k = 0; k < kBK / 32; ++k)
                        tc_mma_i8_pair(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb != 0 || k != 0) ? 1u : 0u);
                    tc_commit_mask(bar_empty(s), (uint16_t)0xF);      // stage free: tell all four CTAs
                }
                if (ok) tc_commit_mask(bar_tfull(acc), pair_mask);
            }
        } else if (lane == 0) {
            // -------------------------------------------------------------- relay (rank-1 CTA)
            // this CTA's rows of Xq have landed: tell the leader, whose issuer reads them
            const uint32_t full_leader0 = mapa_u32(bar_full(0), leader);
            uint32_t it = 0;
            bool ok = true;
            for (int u = cluster_id; ok && u < p.num_units; u += num_clusters) {
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(bar_full(s), ph, abort_flag, limit)) { ok = false; break; }
                    mbar_arrive_cluster(full_leader0 + 8u * s);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int ew = warp - 2;                          // 0..EPI-1
        const int q = warp & 3;                           // TMEM lane quarter
        const int sub = ew >> 2;                          // which of the EPI/4 warps of this quarter
        constexpr int kSubs = EPI / 4;
        constexpr int kMyChunks = kChunks / kSubs;        // column chunks this warp owns per tile
        constexpr int kMyCols = kMyChunks * kChunkCols;
        static_assert(kChunks % kSubs == 0, "chunks must divide among the warps of a quarter");
        const uint32_t stage0 = base + L::kOffStage + (uint32_t)ew * 8192u;   // two staging tiles (STORE == 0)
        float* my_sw = reinterpret_cast<float*>(smem + L::kOffScale) + ew * 2 * kMyCols;
        float* my_bias = my_sw + kMyCols;
        const uint32_t tempty0 = mapa_u32(bar_tempty(0), leader);
        constexpr int kElem = (OUT == STWQ_OUT_BF16) ? 2 : 4;
        uint32_t t = 0, nstore = 0;
        bool ok = true;
        for (int u = cluster_id; u < p.num_units; u += num_clusters, ++t) {
            const int acc = t & 1;
            const uint32_t aph = (t >> 1) & 1u;
            const int m0 = (u / p.super_n) * (2 * kBM) + (int)rank * kBM;
            const int n0 = (2 * (u % p.super_n) + (int)pi) * BN;
            const int64_t row = (int64_t)m0 + q * 32 + lane;
            float st = 0.0f;
            if (OUT != STWQ_OUT_INT32) {
                // column scales and biases of this warp's chunks -> its private shared copy, and
                // the row scale, all fetched before the accumulator is waited for
                __syncwarp();
                for (int i = lane * 4; i < kMyCols; i += 128) {
                    const int k = i / kChunkCols;
                    const int col = n0 + (sub + k * kSubs) * kChunkCols + (i % kChunkCols);
                    float4 sw = make_float4(0.f, 0.f, 0.f, 0.f), bi = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (col < p.N) {                      // N is a multiple of 4: the float4 is in range
                        sw = __ldg(reinterpret_cast<const float4*>(p.s_w + col));
                        if (p.bias != nullptr) bi = __ldg(reinterpret_cast<const float4*>(p.bias + col));
                    }
                    *reinterpret_cast<float4*>(my_sw + i) = sw;
                    *reinterpret_cast<float4*>(my_bias + i) = bi;
                }
                if (row < p.M && n0 < p.N) {
                    const int pos = p.pos_ids[row];
                    if (pos >= 0 && pos < p.P) st = p.s_tok[pos];
                    else atomicOr(p.status, STWQ_DEV_POS_RANGE);
                }
                __syncwarp();
            }
            if (ok) ok = mbar_wait(bar_tfull(acc), aph, abort_flag, limit);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN);
            // all of this warp's accumulator columns at once, the buffer handed back as soon as they
            // have landed; conversion and stores follow from registers
            constexpr int kLoadsPerChunk = (OUT == STWQ_OUT_BF16) ? 2 : 1;
            constexpr int kLoads = kMyChunks * kLoadsPerChunk;
            uint32_t racc[kLoads][32];
#pragma unroll
            for (int k = 0; k < kMyChunks; ++k) {
                const int c = sub + k * kSubs;
#pragma unroll
                for (int h = 0; h < kLoadsPerChunk; ++h)
                    tmem_ld32(taddr + (uint32_t)(c * kChunkCols + h * 32), racc[k * kLoadsPerChunk + h]);
            }
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tempty0 + 8u * acc);
#pragma unroll
            for (int k = 0; k < kMyChunks; ++k, ++nstore) {
                const int c = sub + k * kSubs;
                const int col0 = n0 + c * kChunkCols;
                const float* csw = my_sw + k * kChunkCols;
                const float* cbi = my_bias + k * kChunkCols;
                const uint32_t* r0 = racc[k * kLoadsPerChunk];
                const uint32_t* r1 = racc[k * kLoadsPerChunk + kLoadsPerChunk - 1];
                uint32_t w[32];                           // this row's 128 bytes of output
                const uint64_t st2 = pack_f2(st, st);
                if (OUT == STWQ_OUT_BF16) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const uint32_t* r = h == 0 ? r0 : r1;
                            const float4 sw = *reinterpret_cast<const float4*>(csw + h * 32 + j);
                            const float4 bi = *reinterpret_cast<const float4*>(cbi + h * 32 + j);
                            uint64_t z01 = fma_f2(pack_f2((float)(int32_t)r[j + 0], (float)(int32_t)r[j + 1]),
                                                  mul_f2(st2, pack_f2(sw.x, sw.y)), pack_f2(bi.x, bi.y));
                            uint64_t z23 = fma_f2(pack_f2((float)(int32_t)r[j + 2], (float)(int32_t)r[j + 3]),
                                                  mul_f2(st2, pack_f2(sw.z, sw.w)), pack_f2(bi.z, bi.w));
                            if (ACT != STWQ_ACT_NONE) {
                                z01 = gelu_fast_f2(z01);
                                z23 = gelu_fast_f2(z23);
                            }
                            float v0, v1, v2, v3;
                            unpack_f2(z01, v0, v1);
                            unpack_f2(z23, v2, v3);
                            w[h * 16 + j / 2] = pack_bf16(v0, v1);
                            w[h * 16 + j / 2 + 1] = pack_bf16(v2, v3);
                        }
                    }
                } else if (OUT == STWQ_OUT_F32) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const float4 sw = *reinterpret_cast<const float4*>(csw + j);
                        const float4 bi = *reinterpret_cast<const float4*>(cbi + j);
                        const uint64_t z01 = fma_f2(pack_f2((float)(int32_t)r0[j + 0], (float)(int32_t)r0[j + 1]),
                                                    mul_f2(st2, pack_f2(sw.x, sw.y)), pack_f2(bi.x, bi.y));
                        const uint64_t z23 = fma_f2(pack_f2((float)(int32_t)r0[j + 2], (float)(int32_t)r0[j + 3]),
                                                    mul_f2(st2, pack_f2(sw.z, sw.w)), pack_f2(bi.z, bi.w));
                        float v0, v1, v2, v3;
                        unpack_f2(z01, v0, v1);
                        unpack_f2(z23, v2, v3);
                        w[j + 0] = __float_as_uint(apply_act<ACT, false>(v0));
                        w[j + 1] = __float_as_uint(apply_act<ACT, false>(v1));
                        w[j + 2] = __float_as_uint(apply_act<ACT, false>(v2));
                        w[j + 3] = __float_as_uint(apply_act<ACT, false>(v3));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) w[j] = r0[j];
                }
                if (STORE == 1) {
                    // straight from registers: this thread's 128 contiguous bytes of row `row`
                    if (row < p.M && col0 < p.N) {
                        uint8_t* y = reinterpret_cast<uint8_t*>(p.Y) + ((size_t)row * (size_t)p.N + (size_t)col0) * kElem;
                        if (p.y_vec32 && col0 + kChunkCols <= p.N) {
#pragma unroll
                            for (int g = 0; g < 4; ++g) st_global_v8(y + g * 32, w + g * 8);
                        } else {
                            const int valid = (p.N - col0) * kElem;        // a multiple of 16 bytes
#pragma unroll
                            for (int g = 0; g < 8; ++g)
                                if (g * 16 < valid) st_global_v4(y + g * 16, w + g * 4);
                        }
                    }
                } else {
                    const uint32_t stage_tile = stage0 + (nstore & 1u) * 4096u;
                    const uint32_t my_row_addr = stage_tile + (uint32_t)lane * 128u;
                    // the store that last used this staging tile (two stores ago) must have been read
                    if (lane == 0) bulk_wait_read1();
                    __syncwarp();
#pragma unroll
                    for (int g = 0; g < 8; ++g) {         // eight 16-byte pieces, swizzled by row
                        const uint32_t piece = (uint32_t)(g ^ (lane & 7));
                        st_shared_v4(my_row_addr + piece * 16u, w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3]);
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        if (col0 < p.N && (int64_t)m0 + q * 32 < p.M) tma_store_2d(&tmY, stage_tile, col0, m0 + q * 32);
                        bulk_commit();    // one group per chunk, even an empty one: wait_group.read 1 counts groups
                    }
                }
            }
        }
        if (STORE == 0 && lane == 0) bulk_wait0();         // stores complete before the CTA may exit
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, STWQ_DEV_TIMEOUT);
    cluster_sync_all();                                  // no remote arrive or multicast still to land
    tc_fence_after();
    if (warp == 2) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * BN) : "memory");
    }
}

// ---------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

int fail(stwq_ctx* ctx, cudaError_t e)
{
    ctx->last_cuda_error = (int)e;
    (void)cudaGetLastError();
    return STWQ_ERR_CUDA;
}

int encode_2d(stwq_ctx* ctx, CUtensorMap* map, CUtensorMapDataType dt, int elem_bytes, const void* ptr, int64_t rows,
              int64_t cols, int box_cols, int box_rows)
{
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)cols * (cuuint64_t)elem_bytes};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, dt, 2, const_cast<void*>(ptr), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        ctx->last_cuda_error = (int)r;
        return STWQ_ERR_CUDA;
    }
    return STWQ_OK;
}

// Per-device launch state of this library (the context of the main library knows nothing of it).
struct McState {
    int max_clusters[2] = {0, 0};          // by STORE
    uint32_t configured[2] = {0, 0};
};
McState g_state[64];

template <int STAGES, int EPI, int OUT, int ACT, int STORE>
int launch_variant(stwq_ctx* ctx, const CUtensorMap& tmAh, const CUtensorMap& tmB, const CUtensorMap& tmY,
                   const McParams& p, bool dependent, cudaStream_t st)
{
    using L = SmemMc<STAGES, EPI, STORE>;
    auto kern = qgemm_mc_kernel<STAGES, EPI, OUT, ACT, STORE>;
    if (ctx->device < 0 || ctx->device >= 64) return STWQ_ERR_DIM;
    McState& S = g_state[ctx->device];
    const uint32_t bit = 1u << (OUT * 4 + ACT);
    if (!(S.configured[STORE] & bit)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamic);
        if (e != cudaSuccess) return fail(ctx, e);
        S.configured[STORE] |= bit;
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 4;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(64 + 32 * EPI, 1, 1);
    cfg.dynamicSmemBytes = L::kDynamic;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // persistent: exactly as many clusters as can be resident at once (a cluster sits in one GPC)
    if (S.max_clusters[STORE] <= 0) {
        cfg.gridDim = dim3((unsigned)(ctx->sm_count & ~3), 1, 1);
        int n = 0;
        cudaError_t e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess || n <= 0) return fail(ctx, e == cudaSuccess ? cudaErrorLaunchOutOfResources : e);
        S.max_clusters[STORE] = n < ctx->sm_count / 4 ? n : ctx->sm_count / 4;
    }
    int clusters = S.max_clusters[STORE];
    if (p.num_units < clusters) clusters = p.num_units;
    cfg.gridDim = dim3((unsigned)(4 * clusters), 1, 1);
    cfg.numAttrs = dependent ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmAh, tmB, tmY, p);
    ctx->launches += 1;
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : fail(ctx, e);
}

template <int STAGES, int STORE>
int launch_store(stwq_ctx* ctx, const CUtensorMap& tmAh, const CUtensorMap& tmB, const CUtensorMap& tmY,
                 const McParams& p, int act, int out_dtype, bool dependent, cudaStream_t st)
{
#define STWQ_CASE(O, A) \
    if (out_dtype == O && act == A) return launch_variant<STAGES, 8, O, A, STORE>(ctx, tmAh, tmB, tmY, p, dependent, st);
    if (out_dtype == STWQ_OUT_INT32)
        return launch_variant<STAGES, 8, STWQ_OUT_INT32, STWQ_ACT_NONE, STORE>(ctx, tmAh, tmB, tmY, p, dependent, st);
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_NONE)
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_GELU_ERF)
    STWQ_CASE(STWQ_OUT_F32, STWQ_ACT_GELU_TANH)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_NONE)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_GELU_ERF)
    STWQ_CASE(STWQ_OUT_BF16, STWQ_ACT_GELU_TANH)
#undef STWQ_CASE
    return STWQ_ERR_BITS;
}

}  // namespace

// The one symbol the main library looks up. Same contract as its own tiled GEMM launcher: all
// pointers are device pointers, the launch is asynchronous on `stream`, nothing is allocated.
// Returns STWQ_ERR_DIM for problems it does not take (fewer than two tile columns; output types
// other than fp32 / bf16 / int32), which the caller then runs with its own kernel.
extern "C" __attribute__((visibility("default"))) int stwq_mc_launch(
    stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K, int N, const int8_t* Wq,
    const float* s_w, const float* s_tok, int P, const float* bias, int act, int out_dtype, void* Y,
    int after_quantize, void* stream)
{
    if (N <= BN) return STWQ_ERR_DIM;
    if (out_dtype != STWQ_OUT_F32 && out_dtype != STWQ_OUT_BF16 && out_dtype != STWQ_OUT_INT32) return STWQ_ERR_DIM;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int tiles_m = (int)((M + 2 * kBM - 1) / (2 * kBM));
    const int tiles_n = (N + BN - 1) / BN;
    McParams p;
    p.M = M; p.N = N; p.K = K; p.P = P;
    p.pos_ids = pos_ids; p.s_w = s_w; p.s_tok = s_tok; p.bias = bias;
    p.super_n = (tiles_n + 1) / 2;
    p.num_units = tiles_m * p.super_n;
    p.num_kb = (K + kBK - 1) / kBK;
    p.status = ctx->d_status;
    p.wait_limit_ns = (unsigned long long)ctx->wait_limit_ms * 1000000ull;
    p.Y = Y;
    const int elem = out_dtype == STWQ_OUT_BF16 ? 2 : 4;
    p.y_vec32 = ((reinterpret_cast<uintptr_t>(Y) & 31u) == 0 && ((int64_t)N * elem) % 32 == 0) ? 1 : 0;

    CUtensorMap tmAh, tmB, tmY;
    int rc = encode_2d(ctx, &tmAh, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Xq, M, K, kBK, 64);
    if (rc != STWQ_OK) return rc;
    rc = encode_2d(ctx, &tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, N, K, kBK, BN / 2);
    if (rc != STWQ_OK) return rc;
    if (out_dtype == STWQ_OUT_BF16)
        rc = encode_2d(ctx, &tmY, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, M, N, 64, 32);
    else if (out_dtype == STWQ_OUT_F32)
        rc = encode_2d(ctx, &tmY, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, Y, M, N, 32, 32);
    else
        rc = encode_2d(ctx, &tmY, CU_TENSOR_MAP_DATA_TYPE_INT32, 4, Y, M, N, 32, 32);
    if (rc != STWQ_OK) return rc;
    const bool direct = K >= 1536 && act == STWQ_ACT_NONE;
    if (direct) return launch_store<6, 1>(ctx, tmAh, tmB, tmY, p, act, out_dtype, after_quantize != 0, st);
    return launch_store<4, 0>(ctx, tmAh, tmB, tmY, p, act, out_dtype, after_quantize != 0, st);
}

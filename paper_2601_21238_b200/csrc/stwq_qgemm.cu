// qgemm: int8 x int8 -> int32 GEMM with the dequantize / bias / GELU epilogue of the quantized
// linear layer (Section 3: Y = X W on the integer codes; Appendix A.1: x_hat = delta * code).
//
//   acc[m,n] = sum_k Xq[m,k] * Wq[n,k]
//   Y[m,n]   = act( float(acc) * (s_tok[pos[m]] * s_w[n]) + bias[n] )
//
// Blackwell design. Persistent CTAs, one per SM, 192 threads in three roles:
//   warp 0      producer: TMA (cp.async.bulk.tensor, 128-byte swizzle) loads a 128 x 128-byte
//               slice of Xq and a BN x 128-byte slice of Wq per k-block into a ring of stages
//   warp 1      one thread issues tcgen05.mma.kind::i8 (M=128, N=BN, K=32; four per k-block);
//               accumulators live in tensor memory, two buffers of BN columns so that the next
//               tile's main loop overlaps this tile's epilogue
//   warps 2-5   epilogue: tcgen05.ld 32 columns at a time (one row per thread), int32 -> fp32,
//               scale, bias, activation, convert, store
// Synchronisation is by mbarriers only (full/empty per stage, full/empty per accumulator);
// tcgen05.commit signals MMA completion. Every wait is bounded: on expiry the CTA records
// STWQ_DEV_TIMEOUT, all roles leave their loops, outstanding copies are awaited (bounded), tensor
// memory is freed and the kernel returns.
// Out-of-range rows and columns of edge tiles, and the K tail, are zero-filled by TMA and
// masked at the store.
#include <cuda.h>
#include <cuda_bf16.h>

#include "stwq_internal.cuh"
#include "stwq_ptx.cuh"

namespace {

constexpr int kBM = 128;           // rows per tile = TMEM lanes
constexpr int kBK = 128;           // int8 elements (= bytes) per k-block = one swizzle row
constexpr int kThreads = 192;

struct GemmParams {
    int64_t M;
    int N, K, P;
    const int32_t* pos_ids;
    const float* s_w;
    const float* s_tok;
    const float* bias;
    void* Y;
    int tiles_n, num_tiles, num_kb;
    uint32_t* status;
    unsigned long long wait_limit_ns;
};

using namespace stwq_ptx;

template <int BN, int STAGES>
struct SmemLayout {
    static constexpr int kABytes = kBM * kBK;
    static constexpr int kBBytes = BN * kBK;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kOffB = STAGES * kABytes;
    static constexpr int kOffScale = STAGES * kStageBytes;        // float [4 warps][BN]
    static constexpr int kOffBias = kOffScale + 4 * BN * 4;       // float [4 warps][BN]
    static constexpr int kOffBars = kOffBias + 4 * BN * 4;        // u64 [2*STAGES + 4]
    static constexpr int kNumBars = 2 * STAGES + 4;
    static constexpr int kOffMisc = kOffBars + kNumBars * 8;      // u32 tmem slot, u32 abort
    static constexpr int kTotal = kOffMisc + 16;
    static constexpr int kDynamic = kTotal + 1024;                // slack for 1024-byte alignment
};

// ---------------------------------------------------------------------------- kernel
template <int BN, int STAGES, int OUT, int ACT>
__global__ void __launch_bounds__(kThreads, 1)
qgemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
             const GemmParams p)
{
    using L = SmemLayout<BN, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);

    float* sm_scale = reinterpret_cast<float*>(smem + L::kOffScale);
    float* sm_bias = reinterpret_cast<float*>(smem + L::kOffBias);
    const uint32_t bars = base + L::kOffBars;
    auto bar_full = [&](int s) { return bars + 8u * s; };
    auto bar_empty = [&](int s) { return bars + 8u * (STAGES + s); };
    auto bar_tfull = [&](int a) { return bars + 8u * (2 * STAGES + a); };
    auto bar_tempty = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kOffMisc);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + L::kOffMisc + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full(s), 1);
            mbar_init(bar_empty(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull(a), 1);
            mbar_init(bar_tempty(a), 4);
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(tmem_slot)),
                     "r"(2 * BN)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const unsigned long long limit = p.wait_limit_ns;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;                      // k-blocks issued so far
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x) {
                const int m0 = (tile / p.tiles_n) * kBM;
                const int n0 = (tile % p.tiles_n) * BN;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(bar_empty(s), ph ^ 1u, abort_flag, limit)) { ok = false; break; }
                    mbar_expect_tx(bar_full(s), L::kStageBytes);
                    tma_load_2d(base + s * L::kABytes, &tmA, kb * kBK, m0, bar_full(s));
                    tma_load_2d(base + L::kOffB + s * L::kBBytes, &tmB, kb * kBK, n0, bar_full(s));
                }
            }
            if (!ok) {
                // wait (bounded) for the copies still in flight before the CTA may exit
                const uint32_t first = it > (uint32_t)STAGES ? it - STAGES : 0u;
                for (uint32_t j = first; j < it; ++j) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(bar_full(j % STAGES), (j / STAGES) & 1u))
                        if (globaltimer_ns() - t0 > limit) break;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_i8(kBM, BN);
            uint32_t it = 0, t = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x, ++t) {
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
                        tc_mma_i8(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    tc_commit(bar_empty(s));       // stage reusable once these MMAs have read it
                }
                if (ok) tc_commit(bar_tfull(acc)); // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;                    // TMEM lane quarter this warp may read
        // each epilogue warp keeps its own copy of the tile's column scales and biases, so the
        // four warps never have to meet at a barrier
        float* scale_t = sm_scale + (warp - 2) * BN;
        float* bias_t = sm_bias + (warp - 2) * BN;
        uint32_t t = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x, ++t) {
            const int acc = t & 1;
            const uint32_t aph = (t >> 1) & 1u;
            const int m0 = (tile / p.tiles_n) * kBM;
            const int n0 = (tile % p.tiles_n) * BN;
            if (OUT != STWQ_OUT_INT32) {
                __syncwarp();
                for (int j = lane; j < BN; j += 32) {
                    const int col = n0 + j;
                    scale_t[j] = col < p.N ? p.s_w[col] : 0.0f;
                    bias_t[j] = (p.bias != nullptr && col < p.N) ? p.bias[col] : 0.0f;
                }
                __syncwarp();
            }
            const int64_t row = (int64_t)m0 + q * 32 + lane;
            const bool row_ok = row < p.M;
            float st = 0.0f;
            if (OUT != STWQ_OUT_INT32 && row_ok) {
                const int pos = p.pos_ids[row];
                if (pos >= 0 && pos < p.P) st = p.s_tok[pos];
                else atomicOr(p.status, STWQ_DEV_POS_RANGE);
            }
            if (ok) ok = mbar_wait(bar_tfull(acc), aph, abort_flag, limit);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(taddr + (uint32_t)(c * 32), r);
                tmem_ld_wait();
                const int col0 = n0 + c * 32;
                if (!row_ok || col0 >= p.N) continue;
                if (OUT == STWQ_OUT_INT32) {
                    int32_t* y = reinterpret_cast<int32_t*>(p.Y) + row * p.N + col0;
                    if ((p.N & 3) == 0 && col0 + 32 <= p.N) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<uint4*>(y + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
                    } else {
                        for (int j = 0; j < 32 && col0 + j < p.N; ++j) y[j] = (int32_t)r[j];
                    }
                } else {
                    float v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float sc = __fmul_rn(st, scale_t[c * 32 + j]);
                        v[j] = apply_act<ACT>(__fmaf_rn((float)(int32_t)r[j], sc, bias_t[c * 32 + j]));
                    }
                    if (OUT == STWQ_OUT_F32) {
                        float* y = reinterpret_cast<float*>(p.Y) + row * p.N + col0;
                        if ((p.N & 3) == 0 && col0 + 32 <= p.N) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<float4*>(y + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                        } else {
                            for (int j = 0; j < 32 && col0 + j < p.N; ++j) y[j] = v[j];
                        }
                    } else {
                        __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(p.Y) + row * p.N + col0;
                        if ((p.N & 7) == 0 && col0 + 32 <= p.N) {
#pragma unroll
                            for (int j = 0; j < 32; j += 8) {
                                __nv_bfloat162 b0 = __floats2bfloat162_rn(v[j], v[j + 1]);
                                __nv_bfloat162 b1 = __floats2bfloat162_rn(v[j + 2], v[j + 3]);
                                __nv_bfloat162 b2 = __floats2bfloat162_rn(v[j + 4], v[j + 5]);
                                __nv_bfloat162 b3 = __floats2bfloat162_rn(v[j + 6], v[j + 7]);
                                uint4 u;
                                u.x = *reinterpret_cast<uint32_t*>(&b0);
                                u.y = *reinterpret_cast<uint32_t*>(&b1);
                                u.z = *reinterpret_cast<uint32_t*>(&b2);
                                u.w = *reinterpret_cast<uint32_t*>(&b3);
                                *reinterpret_cast<uint4*>(y + j) = u;
                            }
                        } else {
                            for (int j = 0; j < 32 && col0 + j < p.N; ++j) y[j] = __float2bfloat16_rn(v[j]);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty(acc));
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, STWQ_DEV_TIMEOUT);
    if (warp == 2) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * BN)
                     : "memory");
    }
}

// ---------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// 2-D map over a row-major [rows, K] int8 matrix; box = 128 bytes of K x box_rows rows.
int make_map(stwq_ctx* ctx, CUtensorMap* map, const void* ptr, int64_t rows, int K, int box_rows)
{
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t gstride[1] = {(cuuint64_t)K};
    cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        ctx->last_cuda_error = (int)r;
        return STWQ_ERR_CUDA;
    }
    return STWQ_OK;
}

template <int BN, int STAGES, int OUT, int ACT>
int launch_variant(stwq_ctx* ctx, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmParams& p,
                   cudaStream_t st)
{
    using L = SmemLayout<BN, STAGES>;
    auto kern = qgemm_kernel<BN, STAGES, OUT, ACT>;
    const uint64_t bit = 1ull << ((BN == 256 ? 0 : 16) + OUT * 4 + ACT);
    if (!(ctx->configured_mask & bit)) {  // opt in to large dynamic shared memory once per device
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamic);
        if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
        ctx->configured_mask |= bit;
    }
    const int grid = p.num_tiles < ctx->sm_count ? p.num_tiles : ctx->sm_count;
    kern<<<grid, kThreads, L::kDynamic, st>>>(tmA, tmB, p);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

template <int BN, int STAGES>
int launch_bn(stwq_ctx* ctx, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmParams& p, int act,
              int out_dtype, cudaStream_t st)
{
#define STWQ_CASE(O, A) \
    if (out_dtype == O && act == A) return launch_variant<BN, STAGES, O, A>(ctx, tmA, tmB, p, st);
    if (out_dtype == STWQ_OUT_INT32) return launch_variant<BN, STAGES, STWQ_OUT_INT32, STWQ_ACT_NONE>(ctx, tmA, tmB, p, st);
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

}  // namespace

int stwq_launch_qgemm(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K, int N,
                      const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* bias,
                      int act, int out_dtype, void* Y, cudaStream_t st)
{
    // Tile width: 256 columns unless that leaves the last wave of CTAs mostly idle.
    const int tiles_m = (int)((M + kBM - 1) / kBM);
    auto waves_eff = [&](int bn) {
        const int64_t tiles = (int64_t)tiles_m * ((N + bn - 1) / bn);
        const int64_t waves = (tiles + ctx->sm_count - 1) / ctx->sm_count;
        return (double)tiles / (double)(waves * ctx->sm_count) * ((double)N / (double)(((N + bn - 1) / bn) * bn));
    };
    const int bn = (waves_eff(256) + 0.02 >= waves_eff(128)) ? 256 : 128;

    GemmParams p;
    p.M = M; p.N = N; p.K = K; p.P = P;
    p.pos_ids = pos_ids; p.s_w = s_w; p.s_tok = s_tok; p.bias = bias; p.Y = Y;
    p.tiles_n = (N + bn - 1) / bn;
    p.num_tiles = tiles_m * p.tiles_n;
    p.num_kb = (K + kBK - 1) / kBK;
    p.status = ctx->d_status;
    p.wait_limit_ns = (unsigned long long)ctx->wait_limit_ms * 1000000ull;

    CUtensorMap tmA, tmB;
    int rc = make_map(ctx, &tmA, Xq, M, K, kBM);
    if (rc != STWQ_OK) return rc;
    rc = make_map(ctx, &tmB, Wq, N, K, bn);
    if (rc != STWQ_OK) return rc;
    if (bn == 256) return launch_bn<256, 4>(ctx, tmA, tmB, p, act, out_dtype, st);
    return launch_bn<128, 6>(ctx, tmA, tmB, p, act, out_dtype, st);
}

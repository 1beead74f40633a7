// One-kernel quantized attention head (Section 5: the matrix multiplications of attention run in
// 6 or 8 bits, Appendix C: over a quantized KV cache). Same arithmetic as the three separate stages
// (integer Q K^T, fp32 softmax, Eq. 1 quantizer of the probabilities on [0, 1], integer P V, the
// dequantizers of Appendix A.1), but the scores and the probability codes never leave the SM:
//
//   * a CTA owns 128 queries of one head and walks over the visible keys in chunks of 128;
//   * S = Qq Kq^T of a chunk: tcgen05.mma kind::i8 (M 128, N 128) into tensor memory, operands staged
//     by TMA from the code caches (the head dimension is padded to 128 bytes with zeros by TMA);
//   * the probabilities of a row must be divided by the sum over ALL its keys before they can be
//     quantized, so the keys are walked twice: the first walk only keeps the running maximum and
//     the running sum of every row (one thread per row: a thread reads its row of the accumulator,
//     nothing is exchanged between threads), the second walk recomputes S, turns it into codes
//     round(p * (2^b - 1)), and writes them into shared memory in the 128-byte-swizzled K-major
//     layout a tensor-core operand needs;
//   * O += Pcodes (unsigned) x Vq (signed): a second tcgen05.mma, accumulated over the chunks in
//     tensor memory, dequantized with delta_p * s_v[c] at the end.
//
// Everything a thread does per score is ordinary-pipe work except one ex2 per walk: the
// int32 -> fp32 conversions are done with the 1.5 * 2^23 trick (|acc| <= 256 * 128 * 128 = 2^22 fits),
// and so is the rounding of the codes. Per CTA everything is sequential (MMA, then the threads,
// then the next MMA); two CTAs per SM overlap one another.
//
// HBM traffic: Q codes, the K and V code caches (once per 128 queries, from L2 after the first
// time), and O; against fp32 scores written and read back plus the codes of P in the staged form.
#include <cuda.h>

#include "stwq_internal.cuh"
#include "stwq_ptx.cuh"

using namespace stwq_ptx;

namespace {

constexpr int kQT = 128;          // queries per CTA
constexpr int kKT = 128;          // keys per chunk
constexpr int kKStages = 2;       // ring of key chunks
constexpr int kVStages = 2;       // ring of value chunks
constexpr int kSoftWarps = 4;     // one per tensor-memory lane quarter
constexpr int kThreads = 32 * (2 + kSoftWarps);   // warp 0: TMA, warp 1: MMA + tensor memory, then the row threads
constexpr int kTile = 128 * 128;  // bytes of one 128 x 128-byte operand tile
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kMagic = 12582912.0f;             // 1.5 * 2^23: adding it rounds to an integer in the mantissa
constexpr uint32_t kMagicBits = 0x4B400000u;

struct FaParams {
    int Tq, Tk, d, causal, P, n_qt, dkb, out_bf16;
    const int32_t* pos_q;
    const float* s_q;
    const float* s_kcol;          // padded to a multiple of 128 entries
    const float* s_v;
    float levels;
    void* O;
    uint32_t* status;
    unsigned long long wait_limit_ns;
};

struct FaSmem {
    int offK, offV, offP, offBars, vbytes, total;
    __host__ __device__ FaSmem(int d, int dkb)
    {
        vbytes = d * 128;                                 // d rows of 128 keys
        offK = dkb * kTile;                               // after the query tile(s)
        offV = offK + kKStages * dkb * kTile;
        offP = offV + kVStages * vbytes;
        offBars = offP + kTile;
        total = offBars + 128;
    }
};
constexpr int kNumBars = 1 + 2 * kKStages + 2 * kVStages + 5;   // q, k full/empty, v full/empty, sfull sfree pfull pfree ofull

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}
__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// int32 accumulator (|v| <= 2^22) -> fp32, exact, without the conversion unit
__device__ __forceinline__ float acc_to_float(uint32_t v) { return __uint_as_float(v + kMagicBits) - kMagic; }

__global__ void __launch_bounds__(kThreads, 2)
qattn_fused_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const FaParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const FaSmem L(p.d, p.dkb);

    const uint32_t bars = base + (uint32_t)L.offBars;
    const uint32_t bar_q = bars;
    auto bar_kfull = [&](int s) { return bars + 8u * (1 + s); };
    auto bar_kempty = [&](int s) { return bars + 8u * (1 + kKStages + s); };
    auto bar_vfull = [&](int s) { return bars + 8u * (1 + 2 * kKStages + s); };
    auto bar_vempty = [&](int s) { return bars + 8u * (1 + 2 * kKStages + kVStages + s); };
    const uint32_t bar_sfull = bars + 8u * (1 + 2 * kKStages + 2 * kVStages);
    const uint32_t bar_sfree = bar_sfull + 8u;
    const uint32_t bar_pfull = bar_sfull + 16u;
    const uint32_t bar_pfree = bar_sfull + 24u;
    const uint32_t bar_ofull = bar_sfull + 32u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L.offBars + 8 * kNumBars);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // long (late) query tiles first: under a causal mask they walk over the most keys
    const int qt = p.n_qt - 1 - (int)blockIdx.y;
    const int g = blockIdx.x;
    const int q0 = qt * kQT;
    const int kmax = p.causal ? min(p.Tk - 1, min(q0 + kQT - 1, p.Tq - 1) + p.Tk - p.Tq) : p.Tk - 1;   // last key any row sees
    const int nch = kmax / kKT + 1;
    const int tmem_cols = p.d <= 128 ? 256 : 512;        // S: columns 0..127, O: columns 128..128 + d - 1

    if (threadIdx.x == 0) {
        mbar_init(bar_q, 1);
        for (int s = 0; s < kKStages; ++s) { mbar_init(bar_kfull(s), 1); mbar_init(bar_kempty(s), 1); }
        for (int s = 0; s < kVStages; ++s) { mbar_init(bar_vfull(s), 1); mbar_init(bar_vempty(s), 1); }
        mbar_init(bar_sfull, 1);
        mbar_init(bar_sfree, kSoftWarps);
        mbar_init(bar_pfull, kSoftWarps);
        mbar_init(bar_pfree, 1);
        mbar_init(bar_ofull, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        tc_fence_before();
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const unsigned long long limit = p.wait_limit_ns;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            bool ok = true;
            mbar_expect_tx(bar_q, (uint32_t)(p.dkb * kTile));
            for (int kb = 0; kb < p.dkb; ++kb) tma_load_3d(base + kb * kTile, &tmQ, kb * 128, q0, g, bar_q);
            int it = 0;
            for (; it < 2 * nch; ++it) {
                const int j = it < nch ? it : it - nch;
                const int s = it % kKStages;
                if (!mbar_wait(bar_kempty(s), ((uint32_t)(it / kKStages) & 1u) ^ 1u, abort_flag, limit)) { ok = false; break; }
                mbar_expect_tx(bar_kfull(s), (uint32_t)(p.dkb * kTile));
                for (int kb = 0; kb < p.dkb; ++kb)
                    tma_load_3d(base + L.offK + (s * p.dkb + kb) * kTile, &tmK, kb * 128, j * kKT, g, bar_kfull(s));
                if (it >= nch) {
                    const int sv = j % kVStages;
                    if (!mbar_wait(bar_vempty(sv), ((uint32_t)(j / kVStages) & 1u) ^ 1u, abort_flag, limit)) { ok = false; break; }
                    mbar_expect_tx(bar_vfull(sv), (uint32_t)L.vbytes);
                    tma_load_3d(base + L.offV + sv * L.vbytes, &tmV, j * kKT, 0, g, bar_vfull(sv));
                }
            }
            if (!ok) {
                // giving up: loads already issued may still be landing in this CTA's shared memory
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try_wait(bar_q, 0u))
                    if (globaltimer_ns() - t0 > limit) break;
                for (int b = 1; b <= kKStages && it - b >= 0; ++b) {
                    const int jt = it - b;
                    while (!mbar_try_wait(bar_kfull(jt % kKStages), (uint32_t)(jt / kKStages) & 1u))
                        if (globaltimer_ns() - t0 > limit) break;
                }
                for (int b = 1; b <= kVStages && it - nch - b >= 0; ++b) {
                    const int jv = it - nch - b;
                    while (!mbar_try_wait(bar_vfull(jv % kVStages), (uint32_t)(jv / kVStages) & 1u))
                        if (globaltimer_ns() - t0 > limit) break;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc_s = make_idesc_i8(kQT, kKT);
            const uint32_t idesc_pv = make_idesc_i8(kQT, p.d) & ~(1u << 7);      // A = unsigned codes
            const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 128u;
            bool ok = mbar_wait(bar_q, 0u, abort_flag, limit);
            for (int it = 0; ok && it < 2 * nch; ++it) {
                const int j = it < nch ? it : it - nch;
                const int s = it % kKStages;
                if (!mbar_wait(bar_kfull(s), (uint32_t)(it / kKStages) & 1u, abort_flag, limit)) { ok = false; break; }
                if (it > 0 && !mbar_wait(bar_sfree, (uint32_t)(it - 1) & 1u, abort_flag, limit)) { ok = false; break; }
                tc_fence_after();
                for (int kb = 0; kb < p.dkb; ++kb) {
                    const uint64_t a_desc = make_smem_desc(base + kb * kTile);
                    const uint64_t b_desc = make_smem_desc(base + L.offK + (s * p.dkb + kb) * kTile);
                    const int nk = min(4, (p.d - kb * 128 + 31) / 32);           // the rest of the 128 bytes is TMA's zero fill
                    for (int k = 0; k < nk; ++k)
                        tc_mma_i8(tmem_s, a_desc + 2u * k, b_desc + 2u * k, idesc_s, (kb | k) != 0 ? 1u : 0u);
                }
                tc_commit(bar_sfull);
                tc_commit(bar_kempty(s));
                if (it >= nch) {
                    const int sv = j % kVStages;
                    if (!mbar_wait(bar_vfull(sv), (uint32_t)(j / kVStages) & 1u, abort_flag, limit)) { ok = false; break; }
                    if (!mbar_wait(bar_pfull, (uint32_t)j & 1u, abort_flag, limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_smem_desc(base + L.offP);
                    const uint64_t b_desc = make_smem_desc(base + L.offV + sv * L.vbytes);
#pragma unroll
                    for (int k = 0; k < kKT / 32; ++k)
                        tc_mma_i8(tmem_o, a_desc + 2u * k, b_desc + 2u * k, idesc_pv, (j | k) != 0 ? 1u : 0u);
                    tc_commit(bar_pfree);
                    tc_commit(bar_vempty(sv));
                }
            }
            if (ok) tc_commit(bar_ofull);
        }
    } else {
        // ------------------------------------------------------------------ one thread per query row
        const int q = warp & 3;                           // the lane quarter of tensor memory this warp may read
        const int r = q * 32 + lane;                      // row of the tile
        const int i = q0 + r;                             // query index within the head
        const bool valid = i < p.Tq;
        float a = 0.0f;
        if (valid) {
            const int pos = p.pos_q[i];
            if (pos >= 0 && pos < p.P) a = p.s_q[pos];
            else if (g == 0) atomicOr(p.status, STWQ_DEV_POS_RANGE);
        }
        // rows beyond Tq hold zero codes; they run through the same arithmetic and are not stored
        const int last = (p.causal && valid) ? min(p.Tk - 1, i + p.Tk - p.Tq) : p.Tk - 1;   // last visible key of the row
        const int wlast = __reduce_max_sync(0xffffffffu, last);
        const int wfirst = __reduce_min_sync(0xffffffffu, last);
        const uint64_t a2 = dup_f2(a * kLog2e);           // scores are kept in units of log2 e
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t prow = base + (uint32_t)L.offP + (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u;
        float m = -INFINITY, l = 0.0f, inv = 0.0f;
        bool ok = true;
        for (int it = 0; it < 2 * nch; ++it) {
            const bool second = it >= nch;
            const int j = second ? it - nch : it;
            if (it == nch) inv = __fdiv_rn(p.levels, l);
            ok = mbar_wait(bar_sfull, (uint32_t)it & 1u, abort_flag, limit);
            if (ok && second && j > 0) ok = mbar_wait(bar_pfree, (uint32_t)(j - 1) & 1u, abort_flag, limit);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int cb = 0; cb < 4; ++cb) {
                const int col0 = j * kKT + cb * 32;
                const uint32_t pc0 = prow + (uint32_t)(((2 * cb) ^ (r & 7)) * 16);
                const uint32_t pc1 = prow + (uint32_t)(((2 * cb + 1) ^ (r & 7)) * 16);
                if (col0 > wlast) {                       // nobody in this warp sees these keys
                    if (second) {
                        st_shared_v4(pc0, 0u, 0u, 0u, 0u);
                        st_shared_v4(pc1, 0u, 0u, 0u, 0u);
                    }
                    continue;
                }
                uint32_t v[32];
                tmem_ld32(taddr + (uint32_t)(cb * 32), v);
                tmem_ld_wait();
                // z = acc * (s_q * log2 e * s_kcol): the score in units of log2 e
                const float4* kc = reinterpret_cast<const float4*>(p.s_kcol + col0);
                float z[32];
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    const float4 s4 = __ldg(kc + (c >> 2));
                    const uint64_t z01 = mul_f2(pack_f2(acc_to_float(v[c]), acc_to_float(v[c + 1])), mul_f2(a2, pack_f2(s4.x, s4.y)));
                    const uint64_t z23 = mul_f2(pack_f2(acc_to_float(v[c + 2]), acc_to_float(v[c + 3])), mul_f2(a2, pack_f2(s4.z, s4.w)));
                    unpack_f2(z01, z[c], z[c + 1]);
                    unpack_f2(z23, z[c + 2], z[c + 3]);
                }
                if (col0 + 31 > wfirst) {                 // the mask cuts through this block for some row
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (col0 + c > last) z[c] = -INFINITY;
                }
                if (!second) {
                    float bm = z[0];
#pragma unroll
                    for (int c = 1; c < 32; ++c) bm = fmaxf(bm, z[c]);
                    const float mn = fmaxf(m, bm);        // finite: key 0 is visible to every row
                    float sum0 = 0.0f, sum1 = 0.0f;
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        sum0 += ex2f(z[c] - mn);
                        sum1 += ex2f(z[c + 1] - mn);
                    }
                    l = l * ex2f(m - mn) + (sum0 + sum1);
                    m = mn;
                } else {
                    uint32_t w[8];
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        // u = p * levels; adding 1.5 * 2^23 leaves round-to-nearest-even(u) in the low mantissa bits
                        const uint32_t b0 = __float_as_uint(fmaf(ex2f(z[c] - m), inv, kMagic));
                        const uint32_t b1 = __float_as_uint(fmaf(ex2f(z[c + 1] - m), inv, kMagic));
                        const uint32_t b2 = __float_as_uint(fmaf(ex2f(z[c + 2] - m), inv, kMagic));
                        const uint32_t b3 = __float_as_uint(fmaf(ex2f(z[c + 3] - m), inv, kMagic));
                        w[c >> 2] = prmt(prmt(b0, b1, 0x0040u), prmt(b2, b3, 0x0040u), 0x5410u);
                    }
                    st_shared_v4(pc0, w[0], w[1], w[2], w[3]);
                    st_shared_v4(pc1, w[4], w[5], w[6], w[7]);
                }
            }
            tc_fence_before();
            if (second) fence_async_smem();               // the codes become visible to the tensor core's reads
            __syncwarp();
            if (lane == 0) {
                if (second) mbar_arrive(bar_pfull);
                mbar_arrive(bar_sfree);
            }
        }
        // ------------------------------------------------------------------ O = acc * (delta_p * s_v[c])
        if (ok) ok = mbar_wait(bar_ofull, 0u, abort_flag, limit);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after();
            const float delta_p = __fdiv_rn(1.0f, p.levels);
            const int64_t row_off = ((int64_t)g * p.Tq + i) * p.d;
#pragma unroll 1
            for (int cb = 0; cb * 32 < p.d; ++cb) {
                uint32_t v[32];
                tmem_ld32(taddr + 128u + (uint32_t)(cb * 32), v);
                tmem_ld_wait();
                const int ncol = min(32, p.d - cb * 32);  // 32 or 16
                const float4* sv4 = reinterpret_cast<const float4*>(p.s_v + cb * 32);
                float o[32];
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (c < ncol) s4 = __ldg(sv4 + (c >> 2));
                    o[c] = __fmul_rn((float)(int32_t)v[c], __fmul_rn(delta_p, s4.x));
                    o[c + 1] = __fmul_rn((float)(int32_t)v[c + 1], __fmul_rn(delta_p, s4.y));
                    o[c + 2] = __fmul_rn((float)(int32_t)v[c + 2], __fmul_rn(delta_p, s4.z));
                    o[c + 3] = __fmul_rn((float)(int32_t)v[c + 3], __fmul_rn(delta_p, s4.w));
                }
                if (valid) {
                    if (p.out_bf16) {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.O) + row_off + cb * 32);
#pragma unroll
                        for (int c = 0; c < 32; c += 8)
                            if (c < ncol)
                                dst[c >> 3] = make_uint4(pack_bf16(o[c], o[c + 1]), pack_bf16(o[c + 2], o[c + 3]),
                                                         pack_bf16(o[c + 4], o[c + 5]), pack_bf16(o[c + 6], o[c + 7]));
                    } else {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.O) + row_off + cb * 32);
#pragma unroll
                        for (int c = 0; c < 32; c += 4)
                            if (c < ncol) dst[c >> 2] = make_float4(o[c], o[c + 1], o[c + 2], o[c + 3]);
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, STWQ_DEV_TIMEOUT);
    tc_fence_after();
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

}  // namespace

// Qq [G, Tq, d] codes of the queries; Kc [G, Tmax, d], Vt [G, d, Tmax] the code caches; s_kcol_pad
// holds at least round_up(Tk, 128) entries. O [G, Tq, d] fp32 or bf16.
int stwq_launch_qattn_fused(stwq_ctx* ctx, const int8_t* Qq, const int32_t* pos_q, int G, int Tq, int Tk, int d, int Tmax,
                            const int8_t* Kc, const int8_t* Vt, const float* s_q, const float* s_kcol_pad, const float* s_v,
                            int P, int bits, int causal, int out_dtype, void* O, cudaStream_t st)
{
    FaParams p;
    p.Tq = Tq; p.Tk = Tk; p.d = d; p.causal = causal ? 1 : 0; p.P = P;
    p.n_qt = (Tq + kQT - 1) / kQT;
    p.dkb = (d + 127) / 128;
    p.out_bf16 = out_dtype == STWQ_OUT_BF16 ? 1 : 0;
    p.pos_q = pos_q; p.s_q = s_q; p.s_kcol = s_kcol_pad; p.s_v = s_v;
    p.levels = (float)((1 << bits) - 1);
    p.O = O;
    p.status = ctx->d_status;
    p.wait_limit_ns = (unsigned long long)ctx->wait_limit_ms * 1000000ull;
    CUtensorMap tmQ, tmK, tmV;
    int rc = stwq_encode_3d(ctx, &tmQ, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Qq, Tq, d, G, d, (int64_t)Tq * d, 128, kQT);
    if (rc != STWQ_OK) return rc;
    rc = stwq_encode_3d(ctx, &tmK, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Kc, Tmax, d, G, d, (int64_t)Tmax * d, 128, kKT);
    if (rc != STWQ_OK) return rc;
    rc = stwq_encode_3d(ctx, &tmV, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Vt, d, Tmax, G, Tmax, (int64_t)d * Tmax, kKT, d);
    if (rc != STWQ_OK) return rc;
    if (p.n_qt > 65535) return STWQ_ERR_DIM;
    const FaSmem L(d, p.dkb);
    // at most two CTAs per SM (each holds 256 columns of tensor memory when d <= 128, all 512 beyond)
    int dyn = L.total + 1024;
    if (dyn < 78 * 1024) dyn = 78 * 1024;
    if (!ctx->attn_configured) {
        cudaError_t e = cudaFuncSetAttribute(qattn_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
        ctx->attn_configured = 1;
    }
    qattn_fused_kernel<<<dim3((unsigned)G, (unsigned)p.n_qt), kThreads, (size_t)dyn, st>>>(tmQ, tmK, tmV, p);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

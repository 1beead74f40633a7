// Inline-PTX wrappers for the Blackwell (sm_100a) features the GEMM kernels use: mbarriers with
// bounded waits, TMA tensor copies, tcgen05 MMA / commit / tensor-memory loads, and the operand
// descriptors of tcgen05.mma. Included by the GEMM translation units only.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "stwq_internal.cuh"

namespace stwq_ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait. Returns false if the CTA is aborting or the limit expired (then sets abort).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          unsigned long long limit_ns)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    uint32_t polls = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++polls & 31u) == 0u) {
            if (*abort_flag) return false;
            if (globaltimer_ns() - t0 > limit_ns) {
                *abort_flag = 1u;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
          "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
          "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
          "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand tile stored as rows of 128 bytes with the
// 128-byte swizzle (what TMA writes): 8-row groups are 1024 bytes apart (stride byte offset),
// the leading byte offset is unused for swizzled K-major layouts (set to 1), descriptor version 1.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// Instruction descriptor: D = s32, A = B = s8, both K-major, dense, no saturation.
__host__ __device__ constexpr uint32_t make_idesc_i8(int m, int n)
{
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ---- CTA pairs (cta_group::2), stores
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
// TMA load whose completion bytes are credited to a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                                 uint32_t bar_cluster_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar_cluster_addr)
        : "memory");
}
// The same with a third coordinate (batched operands: one matrix per head).
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2,
                                                 uint32_t bar_cluster_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar_cluster_addr)
        : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2)
                 : "memory");
}
__device__ __forceinline__ void tc_mma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive (once all MMAs issued so far have completed) on the barrier at this offset in both CTAs.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)
{
    const uint16_t mask = 3;
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"(mask)
        : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1)
                 : "memory");
}
// Ask for a tile to be brought into L2 (no shared-memory destination, nothing to wait for).
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap* map, int c0, int c1)
{
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global [%0, {%1, %2}];" ::"l"(map), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t* w)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                 "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}
__device__ __forceinline__ void st_global_v4(void* p, const uint32_t* w)
{
    asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&b);
}


// GELU in the epilogue.
//
// STWQ_ACT_GELU_ERF is z Phi(z) with Phi(-|z|) = erfc(|z| / sqrt2) / 2 evaluated as one exp2 of a
// polynomial (see gelu_erf_f2; absolute error on Phi below 1.5e-7) and Phi(|z|) = 1 - Phi(-|z|).
// STWQ_ACT_GELU_TANH is z * sigmoid(2u), u = sqrt(2/pi) (z + 0.044715 z^3), with the hardware's
// exp2 and reciprocal (relative error about 2^-22 each).
// STWQ_ACT_GELU_FAST is z/2 (1 + tanh(u)) with the hardware tanh (tanh.approx.f32, relative error
// about 2^-11): six instructions per element. Its error on y stays below 6e-4 |z|, a quarter of
// the bf16 rounding unit. The epilogue of a K = 1024 tile has only a few thousand issue slots,
// which is why the short form exists; the caller asks for it by name.
// Each form comes as a scalar function (fp32 output) and as a packed one on two values (bf16
// output and chained codes), the packed one sharing its multiplies between the two halves.
__device__ __forceinline__ float tanh_approx(float x)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Packed fp32 arithmetic (two IEEE round-to-nearest operations per instruction on sm_100): the
// epilogue is bound by instruction issue, and this halves its multiply / fma count. Each half
// rounds exactly like the scalar instruction.
__device__ __forceinline__ uint64_t pack_f2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f2(uint64_t v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t mul_f2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma_f2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t dup_f2(float v) { return pack_f2(v, v); }
// The short GELU on a pair: z/2 (1 + tanh(z (c1 + c3 z^2))).
__device__ __forceinline__ uint64_t gelu_fast_f2(uint64_t z)
{
    const uint64_t u = mul_f2(z, fma_f2(dup_f2(0.035677408136300125f), mul_f2(z, z), dup_f2(0.79788456080286536f)));
    float u0, u1;
    unpack_f2(u, u0, u1);
    const uint64_t t = pack_f2(tanh_approx(u0), tanh_approx(u1));
    const uint64_t h = mul_f2(dup_f2(0.5f), z);
    return fma_f2(h, t, h);
}
// The tanh form to fp32 accuracy on a pair: z / (1 + exp(-2u)).
__device__ __forceinline__ uint64_t gelu_tanh_f2(uint64_t z)
{
    // -2 log2(e) sqrt(2/pi) (1 + 0.044715 z^2) z
    const uint64_t a = mul_f2(z, fma_f2(dup_f2(-0.1029432395800235f), mul_f2(z, z), dup_f2(-2.302208198144325f)));
    float a0, a1;
    unpack_f2(a, a0, a1);
    const uint64_t den = fma_f2(dup_f2(1.0f), pack_f2(ex2_approx(a0), ex2_approx(a1)), dup_f2(1.0f));
    float d0, d1;
    unpack_f2(den, d0, d1);
    return mul_f2(z, pack_f2(rcp_approx(d0), rcp_approx(d1)));
}
// The erf form on a pair. For m = |z|: Phi(-m) = erfc(m / sqrt2) / 2 = 2^(-m^2 log2(e) / 2 + q(m)),
// q(m) = log2(erfcx(m / sqrt2)) - 1, a smooth, slowly varying function that a degree-7 polynomial
// (STWQ_ERF_Q0..7, a weighted least-maximum fit on [0, 5.94]) follows closely enough for an absolute error
// on Phi below 4e-8; evaluated in fp32 with the hardware exp2 the error stays below 1.5e-7. Beyond
// m = 5.94 the argument is clamped (Phi < 1.5e-9 there). One special-function instruction per
// element, where the textbook rational forms of erfc need a reciprocal and an exponential.
#define STWQ_ERF_Q0 -0.9999998807907104f
#define STWQ_ERF_Q1 -1.1511108875274658f
#define STWQ_ERF_Q2 0.26219436526298523f
#define STWQ_ERF_Q3 -0.05269109085202217f
#define STWQ_ERF_Q4 0.007389252074062824f
#define STWQ_ERF_Q5 -0.0004212251224089414f
#define STWQ_ERF_Q6 -5.390652222558856e-05f
#define STWQ_ERF_Q7 8.4704415712622e-06f
#define STWQ_ERF_MMAX 5.94f
#define STWQ_ERF_HALF_LOG2E -0.72134752044448170368f
__device__ __forceinline__ uint64_t gelu_erf_f2(uint64_t z)
{
    float z0, z1;
    unpack_f2(z, z0, z1);
    const uint64_t m = pack_f2(fminf(fabsf(z0), STWQ_ERF_MMAX), fminf(fabsf(z1), STWQ_ERF_MMAX));
    uint64_t q = fma_f2(dup_f2(STWQ_ERF_Q7), m, dup_f2(STWQ_ERF_Q6));
    q = fma_f2(q, m, dup_f2(STWQ_ERF_Q5));
    q = fma_f2(q, m, dup_f2(STWQ_ERF_Q4));
    q = fma_f2(q, m, dup_f2(STWQ_ERF_Q3));
    q = fma_f2(q, m, dup_f2(STWQ_ERF_Q2));
    q = fma_f2(q, m, dup_f2(STWQ_ERF_Q1));
    q = fma_f2(q, m, dup_f2(STWQ_ERF_Q0));
    const uint64_t a = fma_f2(mul_f2(m, m), dup_f2(STWQ_ERF_HALF_LOG2E), q);
    float a0, a1;
    unpack_f2(a, a0, a1);
    float h0, h1;
    unpack_f2(mul_f2(z, pack_f2(ex2_approx(a0), ex2_approx(a1))), h0, h1);    // z Phi(-|z|)
    return pack_f2(z0 < 0.0f ? h0 : z0 - h0, z1 < 0.0f ? h1 : z1 - h1);
}
__device__ __forceinline__ float gelu_erf(float z)
{
    const float m = fminf(fabsf(z), STWQ_ERF_MMAX);
    float q = fmaf(STWQ_ERF_Q7, m, STWQ_ERF_Q6);
    q = fmaf(q, m, STWQ_ERF_Q5);
    q = fmaf(q, m, STWQ_ERF_Q4);
    q = fmaf(q, m, STWQ_ERF_Q3);
    q = fmaf(q, m, STWQ_ERF_Q2);
    q = fmaf(q, m, STWQ_ERF_Q1);
    q = fmaf(q, m, STWQ_ERF_Q0);
    const float h = z * ex2_approx(fmaf(m * m, STWQ_ERF_HALF_LOG2E, q));
    return z < 0.0f ? h : z - h;
}
template <int ACT>
__device__ __forceinline__ uint64_t apply_act_f2(uint64_t z)
{
    if (ACT == STWQ_ACT_GELU_ERF) return gelu_erf_f2(z);
    if (ACT == STWQ_ACT_GELU_TANH) return gelu_tanh_f2(z);
    if (ACT == STWQ_ACT_GELU_FAST) return gelu_fast_f2(z);
    return z;
}
template <int ACT>
__device__ __forceinline__ float apply_act(float z)
{
    if (ACT == STWQ_ACT_GELU_FAST) {
        const float u = z * fmaf(0.035677408136300125f, z * z, 0.79788456080286536f);
        const float h = 0.5f * z;
        return fmaf(h, tanh_approx(u), h);
    }
    if (ACT == STWQ_ACT_GELU_ERF) return gelu_erf(z);
    if (ACT == STWQ_ACT_GELU_TANH) {
        const float u = 0.79788456080286536f * fmaf(0.044715f * z * z, z, z);
        return __fdividef(z, 1.0f + __expf(-2.0f * u));
    }
    return z;
}

}  // namespace stwq_ptx

// 2-D tensor map over a dense row-major [rows, cols] matrix with 128-byte swizzle (host side).
int stwq_encode_2d(stwq_ctx* ctx, CUtensorMap* map, CUtensorMapDataType dt, int elem_bytes, const void* ptr,
                   int64_t rows, int64_t cols, int box_cols, int box_rows);
// 3-D tensor map over `batch` row-major [rows, cols] matrices, rows row_pitch bytes apart, matrices
// batch_pitch bytes apart; the box is one matrix deep.
int stwq_encode_3d(stwq_ctx* ctx, CUtensorMap* map, CUtensorMapDataType dt, int elem_bytes, const void* ptr,
                   int64_t rows, int64_t cols, int64_t batch, int64_t row_pitch, int64_t batch_pitch, int box_cols,
                   int box_rows);

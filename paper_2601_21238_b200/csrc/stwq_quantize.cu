// Activation quantization with static per-token-position scales (Eq. 1 applied to the left
// factor of Eq. 2; Section 4.2):  Xq[m,k] = clamp(round((X[m,k] * rc[k]) * rt[pos[m]])).
//
// HBM-bound streaming kernel: 4 bytes in, 1 byte out per element. A warp owns a span of 512
// consecutive columns; lane l handles the four float4 at columns 4*(32*j + l), j = 0..3, so
// every warp-wide load is one contiguous 512-byte request and every warp-wide store one
// contiguous 128-byte request. The span of a warp never changes, so the 16 reciprocal channel
// scales a lane needs stay in registers for the whole kernel; the per-row reciprocal token scale
// is one IEEE division per row and warp.
//
// Large inputs take a second kernel with the same arithmetic (quantize_ring_kernel below): one
// persistent CTA per SM whose producer thread streams 16 KB runs of the flat array X into a
// ten-stage shared-memory ring with TMA (160 KB in flight per SM, which no register-based scheme
// reaches), while sixteen consumer warps convert them; the reciprocal channel and position scales
// live in shared-memory tables computed once per CTA behind the first loads.
#include <cuda.h>

#include "stwq_internal.cuh"
#include "stwq_ptx.cuh"

namespace {

constexpr int kSpan = 512;          // columns per warp and row
constexpr int kThreads = 256;

__device__ __forceinline__ float4 ld_stream(const float* p)
{
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p));
    return v;
}

// Four values -> four packed codes. u = (x * rc) * rt in two IEEE multiplies, round to nearest
// even (cvt.rni: NaN -> 0, +-Inf and huge values -> INT_MIN / INT_MAX), then clamp and pack. With
// 8 bits the clamp is the saturation of cvt.pack (two instructions for four codes); with fewer
// bits the integers are clamped first. A row with a bad position gets rt = 0, which makes every
// finite u zero and every other u NaN, i.e. code 0 throughout.
template <bool B8>
__device__ __forceinline__ uint32_t quantize4(const float4 v, const float4 rc, float rt, int qmin, int qmax)
{
    int q0 = __float2int_rn(__fmul_rn(__fmul_rn(v.x, rc.x), rt));
    int q1 = __float2int_rn(__fmul_rn(__fmul_rn(v.y, rc.y), rt));
    int q2 = __float2int_rn(__fmul_rn(__fmul_rn(v.z, rc.z), rt));
    int q3 = __float2int_rn(__fmul_rn(__fmul_rn(v.w, rc.w), rt));
    if (!B8) {
        q0 = max(min(q0, qmax), qmin);
        q1 = max(min(q1, qmax), qmin);
        q2 = max(min(q2, qmax), qmin);
        q3 = max(min(q3, qmax), qmin);
    }
    uint32_t hi, packed;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(packed) : "r"(q1), "r"(q0), "r"(hi));
    return packed;
}

__device__ __forceinline__ void load_row(const float* xrow, int col0, int K, float4 (&v)[4])
{
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int c = col0 + j * 128;
        if (c < K) v[j] = ld_stream(xrow + c);
    }
}

// Reciprocal token scale of row m (0 and `ok` false if its position is out of range).
__device__ __forceinline__ float row_scale(const int32_t* pos_ids, const float* s_tok, int P, int64_t m, bool& ok)
{
    const int p = pos_ids[m];
    ok = (p >= 0) && (p < P);
    return ok ? __frcp_rn(s_tok[p]) : 0.0f;
}

// The loop is software-pipelined: the loads of the next row (and its position scale) are in
// flight while the current row is converted, and the first row's loads are issued before the
// reciprocal channel scales are computed, so that a warp that only sees a few rows (M of a few
// thousand) does not serialise two memory round trips and sixteen divisions in front of them.
// VPL = float4 per lane and row: a warp's span is 128 VPL columns (512, or 256 where that leaves fewer
// lanes without columns, e.g. K = 1280 = 5 x 256).
template <bool B8, int VPL>
__global__ void __launch_bounds__(kThreads)
quantize_kernel(const float* __restrict__ X, const int32_t* __restrict__ pos_ids, int64_t M, int K,
                const float* __restrict__ s_ch, const float* __restrict__ s_tok, int P, int qmin,
                int qmax, int8_t* __restrict__ Xq, int spans, int64_t row_stride,
                uint32_t* __restrict__ status)
{
    // Programmatic dependent launch, both directions. If this grid was launched as a dependent of
    // the previous kernel of the stream, its blocks may already be resident while that kernel
    // drains; nothing is read or written before that kernel has completed (wait). And a kernel
    // launched as a dependent of this one (the GEMM, which has a prologue, and in the few-row case
    // weights to stream, that do not depend on Xq) may start now; it waits for this grid to
    // finish before it touches Xq. Launched the ordinary way, both instructions do nothing.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int span = (int)(warp % spans);
    int64_t m = warp / spans;
    const int col0 = span * (128 * VPL) + lane * 4;
    if (m >= M) return;

    float4 v[VPL], vn[VPL];
    auto load = [&](int64_t r, float4 (&d)[VPL]) {
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int c = col0 + j * 128;
            if (c < K) d[j] = ld_stream(X + r * K + c);
        }
    };
    load(m, v);
    bool ok;
    float rt = row_scale(pos_ids, s_tok, P, m, ok);

    // reciprocal channel scales of this lane's 4 VPL columns (1 where there is no scaling)
    float rc[4 * VPL];
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
        const int c = col0 + j * 128;
#pragma unroll
        for (int e = 0; e < 4; ++e)
            rc[j * 4 + e] = (s_ch != nullptr && c + e < K) ? __frcp_rn(s_ch[c + e]) : 1.0f;
    }

    while (true) {
        const int64_t mn = m + row_stride;
        const bool more = mn < M;
        bool okn = false;
        float rtn = 0.0f;
        if (more) {
            load(mn, vn);
            rtn = row_scale(pos_ids, s_tok, P, mn, okn);
        }
        if (!ok && lane == 0 && span == 0) atomicOr(status, STWQ_DEV_POS_RANGE);
        int8_t* qrow = Xq + m * K;
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int c = col0 + j * 128;
            if (c < K)
                *reinterpret_cast<uint32_t*>(qrow + c) =
                    quantize4<B8>(v[j], make_float4(rc[j * 4 + 0], rc[j * 4 + 1], rc[j * 4 + 2], rc[j * 4 + 3]), rt, qmin, qmax);
        }
        if (!more) break;
#pragma unroll
        for (int j = 0; j < VPL; ++j) v[j] = vn[j];
        m = mn;
        rt = rtn;
        ok = okn;
    }
}

// ---------------------------------------------------------------------------- bf16 input
// The same quantizer for activations held in bf16 (a bf16 value is an fp32 value, so the
// arithmetic and the result are those of quantize_kernel on the widened input). A warp owns a
// 512-column span; a lane owns two runs of 8 consecutive columns (one 16-byte load each) and
// stores 8 codes per run.
__device__ __forceinline__ uint4 ld_stream_u4(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <bool B8>
__global__ void __launch_bounds__(kThreads)
quantize_bf16_kernel(const uint16_t* __restrict__ X, const int32_t* __restrict__ pos_ids, int64_t M, int K,
                     const float* __restrict__ s_ch, const float* __restrict__ s_tok, int P, int qmin, int qmax,
                     int8_t* __restrict__ Xq, int spans, int64_t row_stride, uint32_t* __restrict__ status)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");               // see quantize_kernel
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int span = (int)(warp % spans);
    int64_t m = warp / spans;
    const int col0 = span * kSpan + lane * 8;
    if (m >= M) return;
    uint4 v[2], vn[2];
    auto load = [&](int64_t r, uint4 (&d)[2]) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int c = col0 + j * 256;
            if (c < K) d[j] = ld_stream_u4(X + r * K + c);
        }
    };
    load(m, v);
    bool ok;
    float rt = row_scale(pos_ids, s_tok, P, m, ok);
    float rc[16];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int c = col0 + j * 256 + e;
            rc[j * 8 + e] = (s_ch != nullptr && c < K) ? __frcp_rn(s_ch[c]) : 1.0f;
        }
    while (true) {
        const int64_t mn = m + row_stride;
        const bool more = mn < M;
        bool okn = false;
        float rtn = 0.0f;
        if (more) {
            load(mn, vn);
            rtn = row_scale(pos_ids, s_tok, P, mn, okn);
        }
        if (!ok && lane == 0 && span == 0) atomicOr(status, STWQ_DEV_POS_RANGE);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int c = col0 + j * 256;
            if (c < K) {
                const float4 a = make_float4(bf16_lo(v[j].x), bf16_hi(v[j].x), bf16_lo(v[j].y), bf16_hi(v[j].y));
                const float4 b = make_float4(bf16_lo(v[j].z), bf16_hi(v[j].z), bf16_lo(v[j].w), bf16_hi(v[j].w));
                uint2 o;
                o.x = quantize4<B8>(a, make_float4(rc[j * 8 + 0], rc[j * 8 + 1], rc[j * 8 + 2], rc[j * 8 + 3]), rt, qmin, qmax);
                o.y = quantize4<B8>(b, make_float4(rc[j * 8 + 4], rc[j * 8 + 5], rc[j * 8 + 6], rc[j * 8 + 7]), rt, qmin, qmax);
                *reinterpret_cast<uint2*>(Xq + m * K + c) = o;
            }
        }
        if (!more) break;
        v[0] = vn[0];
        v[1] = vn[1];
        m = mn;
        rt = rtn;
        ok = okn;
    }
}

// ---------------------------------------------------------------------------- asymmetric codes
// Eq. 1 as printed with a static zero point per position: cs = clamp(round(u) + zs[pos], -h, h-1).
// Besides the codes the kernel accumulates rowcorr[m] = sum_k cs[m,k] - K zs[pos[m]] (zeroed by the
// launcher; one atomic per warp and row), which the GEMM epilogue multiplies by the weights'
// zero points. A warp owns a 512-column span of a row and the loop is pipelined as in
// quantize_kernel: the next row's loads, scale and zero point are in flight while this row is
// converted.
__global__ void __launch_bounds__(kThreads)
quantize_asym_kernel(const float* __restrict__ X, const int32_t* __restrict__ pos_ids, int64_t M, int K,
                     const float* __restrict__ s_ch, const float* __restrict__ s_tok, const int32_t* __restrict__ z_tok,
                     int P, int qmin, int qmax, int8_t* __restrict__ Xq, int32_t* __restrict__ rowcorr, int spans,
                     int64_t row_stride, uint32_t* __restrict__ status)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the GEMM's prologue may start (see quantize_kernel)
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int span = (int)(warp % spans);
    int64_t m = warp / spans;
    const int col0 = span * kSpan + lane * 4;
    if (m >= M) return;

    float4 v[4], vn[4];
    load_row(X + m * K, col0, K, v);
    bool ok;
    float rt = row_scale(pos_ids, s_tok, P, m, ok);
    int zs = ok ? z_tok[pos_ids[m]] : 0;

    float rc[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int c = col0 + j * 128;
#pragma unroll
        for (int e = 0; e < 4; ++e)
            rc[j * 4 + e] = (s_ch != nullptr && c + e < K) ? __frcp_rn(s_ch[c + e]) : 1.0f;
    }

    while (true) {
        const int64_t mn = m + row_stride;
        const bool more = mn < M;
        bool okn = false;
        float rtn = 0.0f;
        int zsn = 0;
        if (more) {
            load_row(X + mn * K, col0, K, vn);
            rtn = row_scale(pos_ids, s_tok, P, mn, okn);
            zsn = okn ? z_tok[pos_ids[mn]] : 0;
        }
        if (!ok && lane == 0 && span == 0) atomicOr(status, STWQ_DEV_POS_RANGE);
        int sum = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = col0 + j * 128;
            if (c < K) {
                const int q0 = stwq_code_asym(__fmul_rn(__fmul_rn(v[j].x, rc[j * 4 + 0]), rt), zs, qmin, qmax);
                const int q1 = stwq_code_asym(__fmul_rn(__fmul_rn(v[j].y, rc[j * 4 + 1]), rt), zs, qmin, qmax);
                const int q2 = stwq_code_asym(__fmul_rn(__fmul_rn(v[j].z, rc[j * 4 + 2]), rt), zs, qmin, qmax);
                const int q3 = stwq_code_asym(__fmul_rn(__fmul_rn(v[j].w, rc[j * 4 + 3]), rt), zs, qmin, qmax);
                sum += q0 + q1 + q2 + q3;
                uint32_t hi, packed;
                asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0));
                asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(packed) : "r"(q1), "r"(q0), "r"(hi));
                *reinterpret_cast<uint32_t*>(Xq + m * K + c) = packed;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) atomicAdd(rowcorr + m, sum - (span == 0 ? K * zs : 0));
        if (!more) break;
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = vn[j];
        m = mn;
        rt = rtn;
        zs = zsn;
        ok = okn;
    }
}

// ---------------------------------------------------------------------------- TMA ring variant
// X is dense, so a tile is simply 4096 consecutive floats of the flat array (16 KB of contiguous
// DRAM, which streams a quarter faster than sixteen 1 KB pieces of sixteen rows: 6.0-6.4 against
// 4.7-4.8 TB/s of reads with nobody consuming). The tensor map views X as [M K / 256, 256] and a
// box is 16 of those rows. Every consumer thread owns two float4 slots of the tile and tracks the
// (row, column) its slots fall on as the tile index advances, without divisions.
constexpr int kTileFloats = 4096;
constexpr int kTileBytes = kTileFloats * 4;  // 16 KB
constexpr int kRingStages = 10;
constexpr int kConsumerWarps = 16;           // 256 floats of a tile each
constexpr int kRingThreads = 32 * (1 + kConsumerWarps);
constexpr int kRingMaxK = 8192;              // table of reciprocal channel scales: 32 KB
constexpr int kRingMaxP = 2048;              // table of reciprocal position scales: 8 KB
constexpr int kRingOffRc = kRingStages * kTileBytes;
constexpr int kRingOffRt = kRingOffRc + kRingMaxK * 4;
constexpr int kRingOffBars = kRingOffRt + kRingMaxP * 4;
constexpr int kRingSmem = kRingOffBars + 2 * kRingStages * 8 + 16 + 128;

template <bool B8>
__global__ void __launch_bounds__(kRingThreads, 1)
quantize_ring_kernel(const __grid_constant__ CUtensorMap tmX, const int32_t* __restrict__ pos_ids, int64_t total, int K,
                     const float* __restrict__ s_ch, const float* __restrict__ s_tok, int P, int qmin, int qmax,
                     int8_t* __restrict__ Xq, int num_tiles, int step_row, int step_col,
                     uint32_t* __restrict__ status, unsigned long long limit)
{
    using namespace stwq_ptx;
    asm volatile("griddepcontrol.wait;" ::: "memory");               // see quantize_kernel
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 127u) & ~127u;
    uint8_t* smem = smem_raw + (base - raw);
    float* rc_s = reinterpret_cast<float*>(smem + kRingOffRc);
    float* rt_s = reinterpret_cast<float*>(smem + kRingOffRt);
    const uint32_t bars = base + kRingOffBars;
    auto bar_full = [&](int s) { return bars + 8u * s; };
    auto bar_empty = [&](int s) { return bars + 8u * (kRingStages + s); };
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + kRingOffBars + 2 * kRingStages * 8);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kRingStages; ++s) {
            mbar_init(bar_full(s), 1);
            mbar_init(bar_empty(s), kConsumerWarps);
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++it) {
                const int s = it % kRingStages;
                const uint32_t ph = (it / kRingStages) & 1u;
                if (!mbar_wait(bar_empty(s), ph ^ 1u, abort_flag, limit)) { ok = false; break; }
                mbar_expect_tx(bar_full(s), kTileBytes);
                tma_load_2d(base + s * kTileBytes, &tmX, 0, t * 16, bar_full(s));   // rows past the end are zero-filled
            }
            if (!ok) {
                const uint32_t first = it > (uint32_t)kRingStages ? it - kRingStages : 0u;
                for (uint32_t j = first; j < it; ++j) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(bar_full(j % kRingStages), (j / kRingStages) & 1u))
                        if (globaltimer_ns() - t0 > limit) break;
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int cw = warp - 1;
        const int ct = threadIdx.x - 32;
        for (int i = ct; i < K; i += 32 * kConsumerWarps) rc_s[i] = s_ch != nullptr ? __frcp_rn(s_ch[i]) : 1.0f;
        for (int i = ct; i < P; i += 32 * kConsumerWarps) rt_s[i] = __frcp_rn(s_tok[i]);
        asm volatile("bar.sync 1, %0;" ::"n"(32 * kConsumerWarps) : "memory");
        // slot j of this thread: floats [256 cw + 128 j + 4 lane, +4) of every tile; K is a
        // multiple of 4, so a slot never straddles two rows
        // f, col: where the slot falls in the current tile. fa, rowa, cola: the same three tiles
        // ahead, which is how early the row's position id is fetched (a dependent global load per
        // tile must not sit on the consumer's critical path); pq holds the ids in flight.
        constexpr int kAhead = 3;
        int64_t f[2], fa[2], rowa[2];
        int col[2], cola[2], pq[2][kAhead];
        const int64_t stride = (int64_t)gridDim.x * kTileFloats;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const uint32_t f0 = (uint32_t)blockIdx.x * kTileFloats + 256u * cw + 128u * j + 4u * lane;
            f[j] = fa[j] = f0;
            rowa[j] = f0 / (uint32_t)K;
            col[j] = cola[j] = (int)(f0 % (uint32_t)K);
#pragma unroll
            for (int a = 0; a < kAhead; ++a) {
                pq[j][a] = fa[j] < total ? pos_ids[rowa[j]] : 0;
                fa[j] += stride;
                rowa[j] += step_row;
                cola[j] += step_col;
                if (cola[j] >= K) { cola[j] -= K; ++rowa[j]; }
            }
        }
        uint32_t it = 0;
        for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++it) {
            const int s = it % kRingStages;
            const uint32_t ph = (it / kRingStages) & 1u;
            int64_t fc[2];
            int cc[2], pc[2];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                fc[j] = f[j]; cc[j] = col[j]; pc[j] = pq[j][0];
                f[j] += stride;
                col[j] += step_col;
                if (col[j] >= K) col[j] -= K;
#pragma unroll
                for (int a = 0; a + 1 < kAhead; ++a) pq[j][a] = pq[j][a + 1];
                pq[j][kAhead - 1] = fa[j] < total ? pos_ids[rowa[j]] : 0;
                fa[j] += stride;
                rowa[j] += step_row;
                cola[j] += step_col;
                if (cola[j] >= K) { cola[j] -= K; ++rowa[j]; }
            }
            bool ok = mbar_wait(bar_full(s), ph, abort_flag, limit);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint8_t* tile = smem + s * kTileBytes;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                if (fc[j] < total) {
                    const int p = pc[j];
                    const bool pok = (p >= 0) && (p < P);
                    const float rt = pok ? rt_s[p] : 0.0f;
                    if (!pok && cc[j] == 0) atomicOr(status, STWQ_DEV_POS_RANGE);
                    const float4 v = *reinterpret_cast<const float4*>(tile + (256 * cw + 128 * j + 4 * lane) * 4);
                    const float4 rc = *reinterpret_cast<const float4*>(rc_s + cc[j]);
                    *reinterpret_cast<uint32_t*>(Xq + fc[j]) = quantize4<B8>(v, rc, rt, qmin, qmax);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(s));
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(status, STWQ_DEV_TIMEOUT);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// Requires M * K to be a multiple of 256 (the flat view has whole rows of 256 floats).
int launch_ring(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, const float* s_ch,
                const float* s_tok, int P, int qmin, int qmax, int8_t* Xq, bool dependent, cudaStream_t st)
{
    const int64_t total = M * (int64_t)K;
    CUtensorMap tmX;
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    cuuint64_t gdim[2] = {256, (cuuint64_t)(total / 256)};
    cuuint64_t gstride[1] = {1024};
    cuuint32_t box[2] = {256, 16};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(&tmX, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(X), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        ctx->last_cuda_error = (int)r;
        return STWQ_ERR_CUDA;
    }
    const bool b8 = (qmin == -128);
    auto kern = b8 ? quantize_ring_kernel<true> : quantize_ring_kernel<false>;
    if (!(ctx->quant_ring_configured & (b8 ? 1 : 2))) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingSmem);
        if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
        ctx->quant_ring_configured |= (b8 ? 1 : 2);
    }
    const int num_tiles = (int)((total + kTileFloats - 1) / kTileFloats);       // the caller has checked that this fits
    const int grid = num_tiles < ctx->sm_count ? num_tiles : ctx->sm_count;
    const int64_t step = (int64_t)grid * kTileFloats;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(kRingThreads, 1, 1);
    cfg.dynamicSmemBytes = kRingSmem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    const unsigned long long limit = (unsigned long long)ctx->wait_limit_ms * 1000000ull;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmX, pos_ids, total, K, s_ch, s_tok, P, qmin, qmax, Xq, num_tiles,
                                       (int)(step / K), (int)(step % K), ctx->d_status, limit);
    ctx->launches += 1;
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

}  // namespace

// Rows handled concurrently by the register-streaming kernels: a warp owns one 512-column span of
// a row and strides over the rows. Chosen so that (a) the grid fits the resident blocks (one
// block beyond them would run alone after all the others: a second wave for a single block),
// (b) every warp sees the same number of rows, (c) the warp count is a multiple of a block's.
static int64_t rows_in_flight_for(int64_t max_blocks, int warps_per_block, int spans, int64_t M)
{
    int64_t rows = max_blocks * warps_per_block / spans;
    if (rows < 1) rows = 1;
    if (rows > M) rows = M;
    for (int64_t passes = (M + rows - 1) / rows;; ++passes) {
        int64_t r = (M + passes - 1) / passes;
        while ((r * spans) % warps_per_block != 0) ++r;
        if (r * spans / warps_per_block <= max_blocks || r <= 1 || passes >= M) return r;
    }
}

int stwq_launch_quantize_asym(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, const float* s_ch,
                              const float* s_tok, const int32_t* z_tok, int P, int bits, int8_t* Xq, int32_t* rowcorr,
                              cudaStream_t st)
{
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    const int spans = (K + kSpan - 1) / kSpan;
    const int warps_per_block = kThreads / 32;
    static int per_sm_asym = 0;                             // resident blocks per SM (the same on every B200)
    if (per_sm_asym <= 0) {
        int n = 0;
        cudaError_t eo = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, quantize_asym_kernel, kThreads, 0);
        if (eo != cudaSuccess) return stwq_cuda_fail(ctx, eo);
        per_sm_asym = n > 0 ? n : 1;
    }
    const int64_t rows_in_flight = rows_in_flight_for((int64_t)ctx->sm_count * per_sm_asym, warps_per_block, spans, M);
    const unsigned blocks = (unsigned)(rows_in_flight * spans / warps_per_block);
    cudaError_t e = cudaMemsetAsync(rowcorr, 0, (size_t)M * sizeof(int32_t), st);
    if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
    quantize_asym_kernel<<<blocks, kThreads, 0, st>>>(X, pos_ids, M, K, s_ch, s_tok, z_tok, P, qmin, qmax, Xq, rowcorr,
                                                      spans, rows_in_flight, ctx->d_status);
    ctx->launches += 1;
    e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

int stwq_launch_quantize_bf16(stwq_ctx* ctx, const void* X, const int32_t* pos_ids, int64_t M, int K,
                              const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq, cudaStream_t st)
{
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    const int spans = (K + kSpan - 1) / kSpan;
    const int warps_per_block = kThreads / 32;
    static int per_sm_bf16 = 0;                             // resident blocks per SM (the same on every B200)
    if (per_sm_bf16 <= 0) {
        int n = 0;
        cudaError_t eo = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, quantize_bf16_kernel<true>, kThreads, 0);
        if (eo != cudaSuccess) return stwq_cuda_fail(ctx, eo);
        per_sm_bf16 = n > 0 ? n : 1;
    }
    const int64_t rows_in_flight = rows_in_flight_for((int64_t)ctx->sm_count * per_sm_bf16, warps_per_block, spans, M);
    const unsigned blocks = (unsigned)(rows_in_flight * spans / warps_per_block);
    const uint16_t* x = static_cast<const uint16_t*>(X);
    if (bits == 8)
        quantize_bf16_kernel<true><<<blocks, kThreads, 0, st>>>(x, pos_ids, M, K, s_ch, s_tok, P, qmin, qmax, Xq, spans,
                                                                rows_in_flight, ctx->d_status);
    else
        quantize_bf16_kernel<false><<<blocks, kThreads, 0, st>>>(x, pos_ids, M, K, s_ch, s_tok, P, qmin, qmax, Xq, spans,
                                                                 rows_in_flight, ctx->d_status);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

int stwq_launch_quantize(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K,
                         const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq,
                         bool dependent, cudaStream_t st)
{
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    // The TMA-ring kernel is kept as a variant (STWQ_OPT_VARIANT = 8; its tables bound K and P): with
    // the grid sized as below the register-streaming kernel is the faster one at every size
    // measured (6.3-6.4 TB/s of algorithmic bytes on 0.7-1.3 GB inputs against 5.4-5.6).
    const bool ring_ok = K <= kRingMaxK && P <= kRingMaxP && ctx->encode_tiled != nullptr && M < ((int64_t)1 << 29) &&
                         (M * (int64_t)K) % 256 == 0;
    const bool ring = ring_ok && ctx->debug == 8;
    if (ring) return launch_ring(ctx, X, pos_ids, M, K, s_ch, s_tok, P, qmin, qmax, Xq, dependent, st);
    // 512-column spans, or 256-column ones where the last 512-column span would be at most half
    // full (K = 768, 1280, ...: fewer lanes without columns) and on inputs of up to 2^24 elements,
    // where more, lighter warps start and finish the short kernel sooner (45 MB: 11.1 -> 10.6 us;
    // from 170 MB on the wider spans are 5 % faster)
    const int rem = K % kSpan;
    const int vpl = ((rem != 0 && rem <= kSpan / 2) || M * (int64_t)K <= ((int64_t)1 << 24)) ? 2 : 4;
    const int span_cols = 128 * vpl;
    const int spans = (K + span_cols - 1) / span_cols;
    const int warps_per_block = kThreads / 32;
    // As many warps as can be resident, then the row stride is shrunk so that every warp sees the
    // same number of rows (no ragged last pass).
    int& per_sm = vpl == 4 ? ctx->quant_blocks_per_sm : ctx->quant_blocks_per_sm2;
    if (per_sm <= 0) {
        int n = 0;
        cudaError_t e = vpl == 4 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, quantize_kernel<true, 4>, kThreads, 0)
                                 : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, quantize_kernel<true, 2>, kThreads, 0);
        if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
        per_sm = n > 0 ? n : 1;
    }
    const int64_t rows_in_flight = rows_in_flight_for((int64_t)ctx->sm_count * per_sm, warps_per_block, spans, M);
    const int64_t blocks = rows_in_flight * spans / warps_per_block;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3((unsigned)blocks, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    auto kern = vpl == 4 ? (bits == 8 ? quantize_kernel<true, 4> : quantize_kernel<false, 4>)
                         : (bits == 8 ? quantize_kernel<true, 2> : quantize_kernel<false, 2>);
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, X, pos_ids, M, K, s_ch, s_tok, P, qmin, qmax, Xq, spans, rows_in_flight,
                                       ctx->d_status);
    ctx->launches += 1;
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

// Activation quantization with static per-token-position scales (Eq. 1 applied to the left
// factor of Eq. 2; Section 4.2):  Xq[m,k] = clamp(round((X[m,k] * rc[k]) * rt[pos[m]])).
//
// HBM-bound streaming kernel: 4 bytes in, 1 byte out per element. A warp owns a span of 512
// consecutive columns; lane l handles the four float4 at columns 4*(32*j + l), j = 0..3, so
// every warp-wide load is one contiguous 512-byte request and every warp-wide store one
// contiguous 128-byte request. The span of a warp never changes, so the 16 reciprocal channel
// scales a lane needs stay in registers for the whole kernel; the per-row reciprocal token scale
// is one IEEE division per row and warp.
#include "stwq_internal.cuh"

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
    return ok ? __fdiv_rn(1.0f, s_tok[p]) : 0.0f;
}

// The loop is software-pipelined: the loads of the next row (and its position scale) are in
// flight while the current row is converted, and the first row's loads are issued before the
// reciprocal channel scales are computed, so that a warp that only sees a few rows (M of a few
// thousand) does not serialise two memory round trips and sixteen divisions in front of them.
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
    const int col0 = span * kSpan + lane * 4;
    if (m >= M) return;

    float4 v[4], vn[4];
    load_row(X + m * K, col0, K, v);
    bool ok;
    float rt = row_scale(pos_ids, s_tok, P, m, ok);

    // reciprocal channel scales of this lane's 16 columns (1 where there is no scaling)
    float rc[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int c = col0 + j * 128;
#pragma unroll
        for (int e = 0; e < 4; ++e)
            rc[j * 4 + e] = (s_ch != nullptr && c + e < K) ? __fdiv_rn(1.0f, s_ch[c + e]) : 1.0f;
    }

    while (true) {
        const int64_t mn = m + row_stride;
        const bool more = mn < M;
        bool okn = false;
        float rtn = 0.0f;
        if (more) {
            load_row(X + mn * K, col0, K, vn);
            rtn = row_scale(pos_ids, s_tok, P, mn, okn);
        }
        if (!ok && lane == 0 && span == 0) atomicOr(status, STWQ_DEV_POS_RANGE);
        int8_t* qrow = Xq + m * K;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = col0 + j * 128;
            if (c < K) {
                int q0 = stwq_code(__fmul_rn(__fmul_rn(v[j].x, rc[j * 4 + 0]), rt), qmin, qmax);
                int q1 = stwq_code(__fmul_rn(__fmul_rn(v[j].y, rc[j * 4 + 1]), rt), qmin, qmax);
                int q2 = stwq_code(__fmul_rn(__fmul_rn(v[j].z, rc[j * 4 + 2]), rt), qmin, qmax);
                int q3 = stwq_code(__fmul_rn(__fmul_rn(v[j].w, rc[j * 4 + 3]), rt), qmin, qmax);
                if (!ok) q0 = q1 = q2 = q3 = 0;
                const uint32_t packed = (uint32_t)(q0 & 0xff) | ((uint32_t)(q1 & 0xff) << 8) |
                                        ((uint32_t)(q2 & 0xff) << 16) | ((uint32_t)(q3 & 0xff) << 24);
                *reinterpret_cast<uint32_t*>(qrow + c) = packed;
            }
        }
        if (!more) break;
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = vn[j];
        m = mn;
        rt = rtn;
        ok = okn;
    }
}

}  // namespace

int stwq_launch_quantize(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K,
                         const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq,
                         bool dependent, cudaStream_t st)
{
    const int spans = (K + kSpan - 1) / kSpan;
    const int warps_per_block = kThreads / 32;
    // As many warps as can be resident, then the row stride is shrunk so that every warp sees the
    // same number of rows (no ragged last pass).
    if (ctx->quant_blocks_per_sm <= 0) {
        int n = 0;
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, quantize_kernel, kThreads, 0);
        if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
        ctx->quant_blocks_per_sm = n > 0 ? n : 1;
    }
    const int64_t max_warps = (int64_t)ctx->sm_count * ctx->quant_blocks_per_sm * warps_per_block;
    int64_t rows_in_flight = max_warps / spans;
    if (rows_in_flight < 1) rows_in_flight = 1;
    if (rows_in_flight > M) rows_in_flight = M;
    const int64_t passes = (M + rows_in_flight - 1) / rows_in_flight;
    rows_in_flight = (M + passes - 1) / passes;
    // total warps must be rows_in_flight * spans and a multiple of warps_per_block
    while ((rows_in_flight * spans) % warps_per_block != 0) ++rows_in_flight;
    const int64_t blocks = rows_in_flight * spans / warps_per_block;
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
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
    cudaError_t e = cudaLaunchKernelEx(&cfg, quantize_kernel, X, pos_ids, M, K, s_ch, s_tok, P, qmin, qmax, Xq, spans,
                                       rows_in_flight, ctx->d_status);
    ctx->launches += 1;
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

// Dynamic token-wise quantization (DTWQ): the baseline that static token-wise quantization
// replaces (Section 1, Section 4.2, Table 5). The range of every row is found at run time:
//     v[k] = X[m,k] * rc[k],  a_m = max_k |v[k]|,  s_m = 2 a_m / (2^b - 1),
//     Xq[m,k] = clamp(round(v[k] * (1 / s_m)))
// and s_m is handed to the dequantizer in place of the static s_tok[pos[m]]. It exists here to
// be timed beside the static kernel: it has to finish a reduction over the row (warp shuffles,
// then one exchange through shared memory) before it can emit the first code of that row.
//
// K > 1024: one block per row at a time (grid-stride), 256 threads; a thread keeps its 4 NV values of
// the row in registers between the two phases, so X is read once; the reciprocal channel scales
// of its columns stay in registers across rows. K <= 8192. K <= 1024: a warp per row (below).
#include "stwq_internal.cuh"

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float4 ld_stream(const float* p)
{
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p));
    return v;
}

template <int NV>
__global__ void __launch_bounds__(kThreads)
dtwq_kernel(const float* __restrict__ X, int64_t M, int K, const float* __restrict__ s_ch, int bits,
            int8_t* __restrict__ Xq, float* __restrict__ s_row, int32_t* __restrict__ row_ids)
{
    __shared__ float warp_max[2][kThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    float rc[NV][4];
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        const int c = 4 * threadIdx.x + j * 4 * kThreads;
#pragma unroll
        for (int e = 0; e < 4; ++e) rc[j][e] = (s_ch != nullptr && c + e < K) ? __frcp_rn(s_ch[c + e]) : 1.0f;
    }
    int it = 0;
    for (int64_t m = blockIdx.x; m < M; m += gridDim.x, ++it) {
        const float* xrow = X + m * K;
        float v[NV][4];
        float a = 0.0f;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int c = 4 * threadIdx.x + j * 4 * kThreads;
            if (c < K) {
                const float4 x = ld_stream(xrow + c);
                v[j][0] = __fmul_rn(x.x, rc[j][0]);
                v[j][1] = __fmul_rn(x.y, rc[j][1]);
                v[j][2] = __fmul_rn(x.z, rc[j][2]);
                v[j][3] = __fmul_rn(x.w, rc[j][3]);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float av = fabsf(v[j][e]);
                    if (av > a) a = av;                   // false for NaN: it does not take part
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
        float* wm = warp_max[it & 1];                     // two buffers: one barrier per row is enough
        if (lane == 0) wm[warp] = a;
        __syncthreads();
        float t = wm[0];
#pragma unroll
        for (int i = 1; i < kThreads / 32; ++i) t = fmaxf(t, wm[i]);
        const float s = stwq_delta(t, bits);
        const float rt = __frcp_rn(s);
        if (threadIdx.x == 0) {
            s_row[m] = s;
            if (row_ids != nullptr) row_ids[m] = (int32_t)m;
        }
        int8_t* qrow = Xq + m * K;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int c = 4 * threadIdx.x + j * 4 * kThreads;
            if (c < K) {
                const int q0 = stwq_code(__fmul_rn(v[j][0], rt), qmin, qmax);
                const int q1 = stwq_code(__fmul_rn(v[j][1], rt), qmin, qmax);
                const int q2 = stwq_code(__fmul_rn(v[j][2], rt), qmin, qmax);
                const int q3 = stwq_code(__fmul_rn(v[j][3], rt), qmin, qmax);
                uint32_t hi, packed;
                asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0));
                asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(packed) : "r"(q1), "r"(q0), "r"(hi));
                *reinterpret_cast<uint32_t*>(qrow + c) = packed;
            }
        }
    }
}

// K <= 1024: a warp per row (no block barrier: the row maximum is a warp-shuffle reduction), a lane
// keeps up to eight float4 of the row, and the next row's loads are in flight while this row is
// reduced and converted, as in the static kernel.
template <int NV>
__global__ void __launch_bounds__(kThreads)
dtwq_warp_kernel(const float* __restrict__ X, int64_t M, int K, const float* __restrict__ s_ch, int bits,
                 int8_t* __restrict__ Xq, float* __restrict__ s_row, int32_t* __restrict__ row_ids, int64_t row_stride)
{
    // the reciprocal channel scales are the same for every warp: the block computes them once
    __shared__ __align__(16) float rc_sh[128 * NV];
    for (int c = threadIdx.x; c < 128 * NV; c += kThreads)
        rc_sh[c] = (s_ch != nullptr && c < K) ? __frcp_rn(s_ch[c]) : 1.0f;
    __syncthreads();
    const int lane = threadIdx.x & 31;
    int64_t m = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    if (m >= M) return;
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    float4 x[NV], xn[NV];
    auto load = [&](int64_t r, float4 (&d)[NV]) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int c = 4 * lane + 128 * j;
            if (c < K) d[j] = ld_stream(X + r * K + c);
        }
    };
    load(m, x);
    float rc[NV][4];
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        const float4 r4 = *reinterpret_cast<const float4*>(rc_sh + 4 * lane + 128 * j);
        rc[j][0] = r4.x; rc[j][1] = r4.y; rc[j][2] = r4.z; rc[j][3] = r4.w;
    }
    while (true) {
        const int64_t mn = m + row_stride;
        const bool more = mn < M;
        if (more) load(mn, xn);
        // the products x * rc are formed twice (for the maximum, then for the codes) rather than
        // kept: two multiplies per element are cheaper than 32 more registers per thread
        float a = 0.0f;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int c = 4 * lane + 128 * j;
            if (c < K) {
                const float av0 = fabsf(__fmul_rn(x[j].x, rc[j][0])), av1 = fabsf(__fmul_rn(x[j].y, rc[j][1]));
                const float av2 = fabsf(__fmul_rn(x[j].z, rc[j][2])), av3 = fabsf(__fmul_rn(x[j].w, rc[j][3]));
                if (av0 > a) a = av0;                     // false for NaN: it does not take part
                if (av1 > a) a = av1;
                if (av2 > a) a = av2;
                if (av3 > a) a = av3;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
        const float s = stwq_delta(a, bits);
        const float rt = __frcp_rn(s);
        if (lane == 0) {
            s_row[m] = s;
            if (row_ids != nullptr) row_ids[m] = (int32_t)m;
        }
        int8_t* qrow = Xq + m * K;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int c = 4 * lane + 128 * j;
            if (c < K) {
                const int q0 = stwq_code(__fmul_rn(__fmul_rn(x[j].x, rc[j][0]), rt), qmin, qmax);
                const int q1 = stwq_code(__fmul_rn(__fmul_rn(x[j].y, rc[j][1]), rt), qmin, qmax);
                const int q2 = stwq_code(__fmul_rn(__fmul_rn(x[j].z, rc[j][2]), rt), qmin, qmax);
                const int q3 = stwq_code(__fmul_rn(__fmul_rn(x[j].w, rc[j][3]), rt), qmin, qmax);
                uint32_t hi, packed;
                asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0));
                asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(packed) : "r"(q1), "r"(q0), "r"(hi));
                *reinterpret_cast<uint32_t*>(qrow + c) = packed;
            }
        }
        if (!more) break;
#pragma unroll
        for (int j = 0; j < NV; ++j) x[j] = xn[j];
        m = mn;
    }
}

template <int NV>
int launch_warp_rows(stwq_ctx* ctx, const float* X, int64_t M, int K, const float* s_ch, int bits, int8_t* Xq,
                     float* s_row, int32_t* row_ids, cudaStream_t st)
{
    static int per_sm = 0;                                  // resident blocks per SM (the same on every B200)
    if (per_sm <= 0) {
        int n = 0;
        cudaError_t eo = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, dtwq_warp_kernel<NV>, kThreads, 0);
        if (eo != cudaSuccess) return stwq_cuda_fail(ctx, eo);
        per_sm = n > 0 ? n : 1;
    }
    // as many warps as are resident, every warp the same number of rows, whole blocks
    const int wpb = kThreads / 32;
    const int64_t max_warps = (int64_t)ctx->sm_count * per_sm * wpb;
    int64_t rows = max_warps < M ? max_warps : M;
    for (int64_t passes = (M + rows - 1) / rows;; ++passes) {
        rows = (M + passes - 1) / passes;
        rows = (rows + wpb - 1) / wpb * wpb;
        if (rows <= max_warps || passes >= M) break;
    }
    dtwq_warp_kernel<NV><<<(unsigned)(rows / wpb), kThreads, 0, st>>>(X, M, K, s_ch, bits, Xq, s_row, row_ids, rows);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

}  // namespace

int stwq_launch_dtwq(stwq_ctx* ctx, const float* X, int64_t M, int K, const float* s_ch, int bits, int8_t* Xq,
                     float* s_row, int32_t* row_ids, cudaStream_t st)
{
    if (K <= 512) return launch_warp_rows<4>(ctx, X, M, K, s_ch, bits, Xq, s_row, row_ids, st);
    if (K <= 1024) return launch_warp_rows<8>(ctx, X, M, K, s_ch, bits, Xq, s_row, row_ids, st);
    const int nv = (K + 4 * kThreads - 1) / (4 * kThreads);
    if (nv > 8) return STWQ_ERR_DIM;
    // grid-stride over the rows with exactly the resident blocks (more would start as a second wave)
    static int per_sm[4] = {0, 0, 0, 0};
    const int v = nv <= 1 ? 0 : (nv <= 2 ? 1 : (nv <= 4 ? 2 : 3));
    if (per_sm[v] <= 0) {
        int n = 0;
        cudaError_t eo = v == 0   ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, dtwq_kernel<1>, kThreads, 0)
                         : v == 1 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, dtwq_kernel<2>, kThreads, 0)
                         : v == 2 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, dtwq_kernel<4>, kThreads, 0)
                                  : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, dtwq_kernel<8>, kThreads, 0);
        if (eo != cudaSuccess) return stwq_cuda_fail(ctx, eo);
        per_sm[v] = n > 0 ? n : 1;
    }
    const int64_t max_blocks = (int64_t)ctx->sm_count * per_sm[v];
    const unsigned grid = (unsigned)(M < max_blocks ? M : max_blocks);
    if (v == 0) dtwq_kernel<1><<<grid, kThreads, 0, st>>>(X, M, K, s_ch, bits, Xq, s_row, row_ids);
    else if (v == 1) dtwq_kernel<2><<<grid, kThreads, 0, st>>>(X, M, K, s_ch, bits, Xq, s_row, row_ids);
    else if (v == 2) dtwq_kernel<4><<<grid, kThreads, 0, st>>>(X, M, K, s_ch, bits, Xq, s_row, row_ids);
    else dtwq_kernel<8><<<grid, kThreads, 0, st>>>(X, M, K, s_ch, bits, Xq, s_row, row_ids);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

// Dynamic token-wise quantization (DTWQ): the baseline that static token-wise quantization
// replaces (Section 1, Section 4.2, Table 5). The range of every row is found at run time:
//     v[k] = X[m,k] * rc[k],  a_m = max_k |v[k]|,  s_m = 2 a_m / (2^b - 1),
//     Xq[m,k] = clamp(round(v[k] * (1 / s_m)))
// and s_m is handed to the dequantizer in place of the static s_tok[pos[m]]. It exists here to
// be timed beside the static kernel: it has to finish a reduction over the row (warp shuffles,
// then one exchange through shared memory) before it can emit the first code of that row.
//
// One block per row at a time (grid-stride), 256 threads; a thread keeps its 4 NV values of the
// row in registers between the two phases, so X is read once; the reciprocal channel scales of
// its columns stay in registers across rows. K <= 8192.
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
        for (int e = 0; e < 4; ++e) rc[j][e] = (s_ch != nullptr && c + e < K) ? __fdiv_rn(1.0f, s_ch[c + e]) : 1.0f;
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
        const float rt = __fdiv_rn(1.0f, s);
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

}  // namespace

int stwq_launch_dtwq(stwq_ctx* ctx, const float* X, int64_t M, int K, const float* s_ch, int bits, int8_t* Xq,
                     float* s_row, int32_t* row_ids, cudaStream_t st)
{
    const int64_t max_blocks = (int64_t)ctx->sm_count * 8;
    const unsigned grid = (unsigned)(M < max_blocks ? M : max_blocks);
    const int nv = (K + 4 * kThreads - 1) / (4 * kThreads);
    if (nv <= 1) dtwq_kernel<1><<<grid, kThreads, 0, st>>>(X, M, K, s_ch, bits, Xq, s_row, row_ids);
    else if (nv <= 2) dtwq_kernel<2><<<grid, kThreads, 0, st>>>(X, M, K, s_ch, bits, Xq, s_row, row_ids);
    else if (nv <= 4) dtwq_kernel<4><<<grid, kThreads, 0, st>>>(X, M, K, s_ch, bits, Xq, s_row, row_ids);
    else if (nv <= 8) dtwq_kernel<8><<<grid, kThreads, 0, st>>>(X, M, K, s_ch, bits, Xq, s_row, row_ids);
    else return STWQ_ERR_DIM;
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

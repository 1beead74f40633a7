// gps_fold: weight side of the equivalent scaling (Eq. 2, W' = s * W) followed by
// per-output-channel min-max quantization (Appendix B: channel-wise weights) in the symmetric
// form of Eq. 1. Offline, once per layer: one block per output channel, two passes over its
// row (the second one served by L1/L2): abs-max by warp shuffles, then divide-round-clamp.
#include "stwq_internal.cuh"

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
fold_kernel(const float* __restrict__ W, int N, int K, const float* __restrict__ s_ch, int bits,
            int8_t* __restrict__ Wq, float* __restrict__ s_w)
{
    __shared__ float warp_max[kThreads / 32];
    __shared__ float delta_sh;
    const int n = blockIdx.x;
    const float* w = W + (int64_t)n * K;
    float a = 0.0f;
    for (int k = threadIdx.x; k < K; k += kThreads) {
        const float v = s_ch ? __fmul_rn(w[k], s_ch[k]) : w[k];
        a = fmaxf(a, fabsf(v));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = a;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = warp_max[0];
        for (int i = 1; i < kThreads / 32; ++i) t = fmaxf(t, warp_max[i]);
        const float d = stwq_delta(t, bits);
        delta_sh = d;
        s_w[n] = d;
    }
    __syncthreads();
    const float d = delta_sh;
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    for (int k = threadIdx.x; k < K; k += kThreads) {
        const float v = s_ch ? __fmul_rn(w[k], s_ch[k]) : w[k];
        Wq[(int64_t)n * K + k] = (int8_t)stwq_code(__fdiv_rn(v, d), qmin, qmax);
    }
}

// Asymmetric variant (Eq. 1 as printed; Appendix B: channel-wise asymmetric weights): the range of
// the scaled row is [min, max] widened to contain 0; the kernel also returns the signed zero point
// and the sum of the row's codes, which the zero-point correction of the integer product needs.
__global__ void __launch_bounds__(kThreads)
fold_asym_kernel(const float* __restrict__ W, int N, int K, const float* __restrict__ s_ch, int bits,
                 int8_t* __restrict__ Wq, float* __restrict__ s_w, int32_t* __restrict__ z_w, int32_t* __restrict__ colsum)
{
    __shared__ float warp_lo[kThreads / 32], warp_hi[kThreads / 32];
    __shared__ int warp_sum[kThreads / 32];
    __shared__ float delta_sh;
    __shared__ int zs_sh;
    const int n = blockIdx.x;
    const float* w = W + (int64_t)n * K;
    float lo = 0.0f, hi = 0.0f;
    for (int k = threadIdx.x; k < K; k += kThreads) {
        const float v = s_ch ? __fmul_rn(w[k], s_ch[k]) : w[k];
        if (v < lo) lo = v;
        if (v > hi) hi = v;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if ((threadIdx.x & 31) == 0) { warp_lo[threadIdx.x >> 5] = lo; warp_hi[threadIdx.x >> 5] = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float a = warp_lo[0], b = warp_hi[0];
        for (int i = 1; i < kThreads / 32; ++i) { a = fminf(a, warp_lo[i]); b = fmaxf(b, warp_hi[i]); }
        float d;
        int zs;
        stwq_asym_params(a, b, bits, d, zs);
        delta_sh = d;
        zs_sh = zs;
        s_w[n] = d;
        z_w[n] = zs;
    }
    __syncthreads();
    const float d = delta_sh;
    const int zs = zs_sh;
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    int sum = 0;
    for (int k = threadIdx.x; k < K; k += kThreads) {
        const float v = s_ch ? __fmul_rn(w[k], s_ch[k]) : w[k];
        const int c = stwq_code_asym(__fdiv_rn(v, d), zs, qmin, qmax);
        Wq[(int64_t)n * K + k] = (int8_t)c;
        sum += c;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int i = 0; i < kThreads / 32; ++i) t += warp_sum[i];
        colsum[n] = t;
    }
}

}  // namespace

int stwq_launch_fold_asym(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, int bits, int8_t* Wq,
                          float* s_w, int32_t* z_w, int32_t* colsum, cudaStream_t st)
{
    fold_asym_kernel<<<N, kThreads, 0, st>>>(W, N, K, s_ch, bits, Wq, s_w, z_w, colsum);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

int stwq_launch_fold(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, int bits,
                     int8_t* Wq, float* s_w, cudaStream_t st)
{
    fold_kernel<<<N, kThreads, 0, st>>>(W, N, K, s_ch, bits, Wq, s_w);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

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

// 4-bit weight codes stored two per byte (W4A8 of Appendix J / Table 11): the symmetric fold above
// with b = 4, codes in [-8, 7], the code of the even input channel in the low nibble and that of
// the following odd channel in the high nibble (two's complement nibbles). K is even.
__global__ void __launch_bounds__(kThreads)
fold_packed4_kernel(const float* __restrict__ W, int N, int K, const float* __restrict__ s_ch,
                    uint8_t* __restrict__ Wp, float* __restrict__ s_w)
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
        const float d = stwq_delta(t, 4);
        delta_sh = d;
        s_w[n] = d;
    }
    __syncthreads();
    const float d = delta_sh;
    for (int j = threadIdx.x; j < K / 2; j += kThreads) {
        const float v0 = s_ch ? __fmul_rn(w[2 * j], s_ch[2 * j]) : w[2 * j];
        const float v1 = s_ch ? __fmul_rn(w[2 * j + 1], s_ch[2 * j + 1]) : w[2 * j + 1];
        const int c0 = stwq_code(__fdiv_rn(v0, d), -8, 7);
        const int c1 = stwq_code(__fdiv_rn(v1, d), -8, 7);
        Wp[(int64_t)n * (K / 2) + j] = (uint8_t)((c0 & 0xF) | ((c1 & 0xF) << 4));
    }
}

// Packed 4-bit codes -> int8 containers: every byte gives two sign-extended codes. One thread per
// 16 packed bytes (32 codes): a 16-byte load, two 16-byte stores.
__global__ void __launch_bounds__(kThreads)
unpack4_kernel(const uint4* __restrict__ Wp, int64_t n_vec, uint4* __restrict__ Wq)
{
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * kThreads) {
        const uint4 p = Wp[i];
        const uint32_t in[4] = {p.x, p.y, p.z, p.w};
        uint32_t out[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // (v ^ 8) - 8 sign-extends a nibble; bit 7 of each byte is set during the subtraction so
            // that no borrow crosses a byte, and cleared again afterwards
            const uint32_t lo = ((((in[j] & 0x0F0F0F0Fu) ^ 0x08080808u) | 0x80808080u) - 0x08080808u) ^ 0x80808080u;
            const uint32_t hi = (((((in[j] >> 4) & 0x0F0F0F0Fu) ^ 0x08080808u) | 0x80808080u) - 0x08080808u) ^ 0x80808080u;
            out[2 * j] = __byte_perm(lo, hi, 0x5140);         // lo0 hi0 lo1 hi1
            out[2 * j + 1] = __byte_perm(lo, hi, 0x7362);     // lo2 hi2 lo3 hi3
        }
        Wq[2 * i] = make_uint4(out[0], out[1], out[2], out[3]);
        Wq[2 * i + 1] = make_uint4(out[4], out[5], out[6], out[7]);
    }
}

}  // namespace

int stwq_launch_fold_packed4(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, uint8_t* Wp, float* s_w,
                             cudaStream_t st)
{
    fold_packed4_kernel<<<N, kThreads, 0, st>>>(W, N, K, s_ch, Wp, s_w);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

int stwq_launch_unpack4(stwq_ctx* ctx, const uint8_t* Wp, int64_t packed_bytes, int8_t* Wq, cudaStream_t st)
{
    const int64_t n_vec = packed_bytes / 16;
    int64_t blocks = (n_vec + kThreads - 1) / kThreads;
    if (blocks > 148 * 8) blocks = 148 * 8;
    unpack4_kernel<<<(unsigned)blocks, kThreads, 0, st>>>(reinterpret_cast<const uint4*>(Wp), n_vec,
                                                          reinterpret_cast<uint4*>(Wq));
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

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

// Gain-Projected Scaling (Section 4.1, Eq. 13-16; Algorithm 1 of Appendix F) on the GPU: the
// per-input-channel scaling vector s of Eq. 2 from calibration activations X [T,K] and the
// layer's weights W [N,K]. Offline work; a handful of column reductions.
//
//   1. Q(X) per tensor (range by the nearest-rank percentile of |X|), Q(W) per output channel
//      (min-max), symmetric quantizer; dX = X - Q(X), dW = W - Q(W).
//   2. R_x[k] = max_t X[t,k] - min_t X[t,k]; k* = argmax (lowest index on ties).
//   3. s_k* = sqrt(R_x[k*] / R_w[k*]), R_w[k*] = the range of column k* of W.
//   4. s_i = s_k* sqrt(sum_t sum_n |dW[n,i] X[t,i]|) / sqrt(sum_t sum_n |W[n,i] dX[t,i]|)   (Eq. 16)
//      or, variant 1, the stationary point of the gain of Eq. 15:
//      s_i = s_k* (sum dW^2 X^2 / sum W^2 dX^2)^(1/4).
// The double sums of step 4 factor, sum_t sum_n |dW[n,i] X[t,i]| = (sum_n |dW[n,i]|)(sum_t |X[t,i]|)
// and likewise for the squares, so one pass over X and one over W, each reducing along its rows
// per channel, give everything. Sums are kept in fp64 and added in a fixed order (per-chunk
// partials, then chunk by chunk), so the result does not change from run to run.
// Guards as in the fold: zero numerator, denominator or weight range gives s_i = 1; s is clamped
// to [1e-4, 1e4].
#include "stwq_internal.cuh"

namespace {

constexpr int kCols = 128;          // channels per block (one per thread)
constexpr int kMaxChunks = 128;     // row chunks per matrix

// Per-chunk, per-channel partial results of one matrix: four fp64 sums and the extremes.
struct Partials {
    double* sabs;     // sum |v|
    double* sdabs;    // sum |v - Q(v)|
    double* ssq;      // sum v^2
    double* sdsq;     // sum (v - Q(v))^2
    float* vmax;
    float* vmin;
};

__host__ __device__ inline size_t partial_bytes(int K) { return (size_t)kMaxChunks * K * (4 * sizeof(double) + 2 * sizeof(float)); }

__host__ __device__ inline Partials carve(void* base, int K)
{
    Partials p;
    const size_t n = (size_t)kMaxChunks * K;
    p.sabs = reinterpret_cast<double*>(base);
    p.sdabs = p.sabs + n;
    p.ssq = p.sdabs + n;
    p.sdsq = p.ssq + n;
    p.vmax = reinterpret_cast<float*>(p.sdsq + n);
    p.vmin = p.vmax + n;
    return p;
}

// delta of each weight row: 2 max|W[n,:]| / (2^b - 1)
__global__ void __launch_bounds__(256) gps_row_delta_kernel(const float* __restrict__ W, int N, int K, int bits,
                                                            float* __restrict__ wdelta)
{
    __shared__ float red[8];
    for (int n = blockIdx.x; n < N; n += gridDim.x) {
        const float* w = W + (size_t)n * K;
        float a = 0.0f;
        for (int k = threadIdx.x; k < K; k += 256) a = fmaxf(a, fabsf(w[k]));
        for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
        __syncthreads();
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
        __syncthreads();
        if (threadIdx.x == 0) {
            float m = red[0];
            for (int i = 1; i < 8; ++i) m = fmaxf(m, red[i]);
            wdelta[n] = stwq_delta(m, bits);
        }
    }
}

// Column statistics of V [rows, K] over the rows of chunk blockIdx.y. The quantizer's delta is
// per row (row_delta, the weights) or one for the whole tensor (*one_delta, the activations).
__global__ void __launch_bounds__(kCols) gps_colstats_kernel(const float* __restrict__ V, int64_t rows, int K,
                                                             const float* __restrict__ row_delta,
                                                             const float* __restrict__ one_delta, int bits,
                                                             int64_t rows_per_chunk, Partials out)
{
    const int k = blockIdx.x * kCols + threadIdx.x;
    if (k >= K) return;
    const int qmax = (1 << (bits - 1)) - 1, qmin = -qmax - 1;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_chunk;
    const int64_t r1 = r0 + rows_per_chunk < rows ? r0 + rows_per_chunk : rows;
    double sabs = 0.0, sdabs = 0.0, ssq = 0.0, sdsq = 0.0;
    float vmax = -INFINITY, vmin = INFINITY;
    const float d1 = one_delta ? *one_delta : 1.0f;
    for (int64_t r = r0; r < r1; ++r) {
        const float v = V[r * K + k];
        const float d = row_delta ? row_delta[r] : d1;
        const float vhat = __fmul_rn(d, (float)stwq_code(__fdiv_rn(v, d), qmin, qmax));
        const double e = (double)v - (double)vhat;
        sabs += fabs((double)v);
        sdabs += fabs(e);
        ssq += (double)v * (double)v;
        sdsq += e * e;
        vmax = fmaxf(vmax, v);
        vmin = fminf(vmin, v);
    }
    const size_t o = (size_t)blockIdx.y * K + k;
    out.sabs[o] = sabs;
    out.sdabs[o] = sdabs;
    out.ssq[o] = ssq;
    out.sdsq[o] = sdsq;
    out.vmax[o] = vmax;
    out.vmin[o] = vmin;
}

// Adds the chunks up in order; per channel: the activation range R_x and the two factors of the
// numerator and of the denominator of step 4; also the range of each weight column.
struct Channel {
    double* rx;       // R_x[k]
    double* rw;       // range of column k of W
    double* num;      // variant 0: (sum |dW|)(sum |X|); variant 1: (sum dW^2)(sum X^2)
    double* den;      // variant 0: (sum |W|)(sum |dX|); variant 1: (sum W^2)(sum dX^2)
};

__global__ void __launch_bounds__(kCols) gps_combine_kernel(Partials x, int xchunks, Partials w, int wchunks, int K,
                                                            int variant, Channel c)
{
    const int k = blockIdx.x * kCols + threadIdx.x;
    if (k >= K) return;
    double xa = 0.0, xda = 0.0, xs = 0.0, xds = 0.0, wa = 0.0, wda = 0.0, ws = 0.0, wds = 0.0;
    float xmax = -INFINITY, xmin = INFINITY, wmax = -INFINITY, wmin = INFINITY;
    for (int i = 0; i < xchunks; ++i) {
        const size_t o = (size_t)i * K + k;
        xa += x.sabs[o]; xda += x.sdabs[o]; xs += x.ssq[o]; xds += x.sdsq[o];
        xmax = fmaxf(xmax, x.vmax[o]); xmin = fminf(xmin, x.vmin[o]);
    }
    for (int i = 0; i < wchunks; ++i) {
        const size_t o = (size_t)i * K + k;
        wa += w.sabs[o]; wda += w.sdabs[o]; ws += w.ssq[o]; wds += w.sdsq[o];
        wmax = fmaxf(wmax, w.vmax[o]); wmin = fminf(wmin, w.vmin[o]);
    }
    c.rx[k] = (double)xmax - (double)xmin;
    c.rw[k] = (double)wmax - (double)wmin;
    c.num[k] = variant == 0 ? wda * xa : wds * xs;
    c.den[k] = variant == 0 ? wa * xda : ws * xds;
}

// One block: k* (largest R_x, lowest index on ties), s_k*, then every s_i.
__global__ void __launch_bounds__(1024) gps_finish_kernel(Channel c, int K, int variant, float* __restrict__ s,
                                                          int32_t* __restrict__ k_star_out)
{
    __shared__ double best_r[32];
    __shared__ int best_k[32];
    __shared__ double sk_sh;
    double r = -1.0;
    int kk = 0x7fffffff;
    for (int k = threadIdx.x; k < K; k += 1024) {
        const double v = c.rx[k];
        if (v > r) { r = v; kk = k; }            // ascending k within a thread: the first maximum stays
    }
    for (int o = 16; o > 0; o >>= 1) {
        const double r2 = __shfl_xor_sync(0xffffffffu, r, o);
        const int k2 = __shfl_xor_sync(0xffffffffu, kk, o);
        if (r2 > r || (r2 == r && k2 < kk)) { r = r2; kk = k2; }
    }
    if ((threadIdx.x & 31) == 0) { best_r[threadIdx.x >> 5] = r; best_k[threadIdx.x >> 5] = kk; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 32; ++i)
            if (best_r[i] > r || (best_r[i] == r && best_k[i] < kk)) { r = best_r[i]; kk = best_k[i]; }
        if (kk < 0 || kk >= K) kk = 0;            // no channel had a range above -1 (all NaN)
        best_k[0] = kk;
        const double rw = c.rw[kk];
        sk_sh = (rw > 0.0 && r > 0.0) ? sqrt(r / rw) : 1.0;
        if (k_star_out) *k_star_out = kk;
    }
    __syncthreads();
    const int kstar = best_k[0];
    const double sk = sk_sh;
    for (int i = threadIdx.x; i < K; i += 1024) {
        double si;
        if (i == kstar) {
            si = sk;
        } else {
            const double num = c.num[i], den = c.den[i];
            if (!(num > 0.0) || !(den > 0.0)) si = 1.0;
            else if (variant == 0) si = sk * sqrt(num) / sqrt(den);
            else si = sk * sqrt(sqrt(num / den));
        }
        if (si < 1e-4) si = 1e-4;
        if (si > 1e4) si = 1e4;
        s[i] = (float)si;
    }
}

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

// Bytes of scratch stwq_launch_gps needs (beyond the calibration workspace for one position).
size_t stwq_gps_ws_bytes(int K, int N)
{
    return align256(sizeof(float) * ((size_t)N + 64)) + 2 * align256(partial_bytes(K)) + align256((size_t)K * 4 * sizeof(double));
}

int stwq_launch_gps(stwq_ctx* ctx, void* ws_cal, void* ws, const float* X, int64_t T, int K, const float* W, int N,
                    int bits, uint32_t pct_ppm, int variant, float* s, int32_t* k_star_out, cudaStream_t st)
{
    uint8_t* base = reinterpret_cast<uint8_t*>(ws);
    float* dx_scale = reinterpret_cast<float*>(base);            // [1] (padded to 64 floats)
    float* wdelta = dx_scale + 64;                                // [N]
    base += align256(sizeof(float) * ((size_t)N + 64));
    Partials px = carve(base, K);
    base += align256(partial_bytes(K));
    Partials pw = carve(base, K);
    base += align256(partial_bytes(K));
    Channel c;
    c.rx = reinterpret_cast<double*>(base);
    c.rw = c.rx + K;
    c.num = c.rw + K;
    c.den = c.num + K;

    // 1a. per-tensor activation delta: the static calibration with a single position
    int rc = stwq_launch_calibrate(ctx, ws_cal, X, nullptr, T, K, 1, nullptr, bits, pct_ppm, dx_scale, st);
    if (rc != STWQ_OK) return rc;
    // 1b. per-row weight deltas
    const int row_blocks = N < ctx->sm_count * 8 ? N : ctx->sm_count * 8;
    gps_row_delta_kernel<<<row_blocks, 256, 0, st>>>(W, N, K, bits, wdelta);
    // 2-4. column statistics of both matrices, combined per channel, then the scales
    auto chunks_for = [](int64_t rows) {
        int64_t c = (rows + 31) / 32;
        return (int)(c < 1 ? 1 : (c > kMaxChunks ? kMaxChunks : c));
    };
    const int xc = chunks_for(T), wc = chunks_for(N);
    const int64_t xr = (T + xc - 1) / xc, wr = ((int64_t)N + wc - 1) / wc;
    const unsigned colblocks = (unsigned)((K + kCols - 1) / kCols);
    gps_colstats_kernel<<<dim3(colblocks, (unsigned)xc), kCols, 0, st>>>(X, T, K, nullptr, dx_scale, bits, xr, px);
    gps_colstats_kernel<<<dim3(colblocks, (unsigned)wc), kCols, 0, st>>>(W, N, K, wdelta, nullptr, bits, wr, pw);
    gps_combine_kernel<<<colblocks, kCols, 0, st>>>(px, xc, pw, wc, K, variant, c);
    gps_finish_kernel<<<1, 1024, 0, st>>>(c, K, variant, s, k_star_out);
    ctx->launches += 5;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

// stwq_calibrate: static token-wise calibration (Section 4.2). For every token position the
// range half-width is an exact order statistic (nearest-rank percentile) of |X * rc| over all
// calibration rows at that position. Found by radix selection on the IEEE bit pattern of the
// non-negative values (monotone in the value): four passes, each histogramming one byte of the
// values that still match the prefix chosen so far, then picking the bin that holds the rank.
// Integer counting only, so the result does not depend on row or thread order.
//
// Workspace per call (caller-provided, 8-byte aligned), for P positions:
//   hist   [P][256] u64   bin counts of the current pass (zero on entry of every pass)
//   rank   [P]      u64   rank still to be located inside the current prefix (0 = empty position)
//   prefix [P]      u32   bits of the answer fixed so far
#include "stwq_internal.cuh"

namespace {

constexpr int kThreads = 256;

struct CalWs {
    unsigned long long* hist;
    unsigned long long* rank;
    uint32_t* prefix;
};

__host__ __device__ inline CalWs cal_ws(void* base, int P)
{
    CalWs w;
    w.hist = reinterpret_cast<unsigned long long*>(base);
    w.rank = w.hist + (size_t)P * 256;
    w.prefix = reinterpret_cast<uint32_t*>(w.rank + P);
    return w;
}

__global__ void cal_clear_kernel(void* base, int P)
{
    CalWs w = cal_ws(base, P);
    const size_t n = (size_t)P * 256;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
         i += (size_t)gridDim.x * blockDim.x)
        w.hist[i] = 0ull;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)P;
         i += (size_t)gridDim.x * blockDim.x) {
        w.rank[i] = 0ull;
        w.prefix[i] = 0u;
    }
}

// One block per row (grid-stride). pass 0..3 histograms byte (3 - pass) of the bit pattern.
__global__ void __launch_bounds__(kThreads)
cal_hist_kernel(const float* __restrict__ X, const int32_t* __restrict__ pos_ids, int64_t rows,
                int K, int P, const float* __restrict__ s_ch, void* base, int pass, int signed_keys,
                uint32_t* __restrict__ status)
{
    __shared__ uint32_t bins[256];
    CalWs w = cal_ws(base, P);
    const int shift = 24 - 8 * pass;
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        const int p = pos_ids ? pos_ids[r] : 0;               // no ids: one population (per-tensor range)
        if (p < 0 || p >= P) {
            if (threadIdx.x == 0 && pass == 0) atomicOr(status, STWQ_DEV_POS_RANGE);
            continue;
        }
        if (pass > 0 && w.rank[p] == 0ull) continue;          // empty position
        bins[threadIdx.x] = 0u;
        __syncthreads();
        const uint32_t prefix = w.prefix[p];
        const float* x = X + r * K;
        bool bad = false;
        for (int k = threadIdx.x; k < K; k += kThreads) {
            const float t = s_ch ? __fmul_rn(x[k], __fdiv_rn(1.0f, s_ch[k])) : x[k];
            const uint32_t raw = __float_as_uint(t);
            if ((raw & 0x7fffffffu) >= 0x7f800000u) bad = true;
            // key that sorts like the value: |t| for the symmetric range, or the usual
            // order-preserving map of a signed float for the two-sided one
            const uint32_t b = signed_keys ? (raw ^ ((raw >> 31) ? 0xffffffffu : 0x80000000u)) : (raw & 0x7fffffffu);
            const bool match = (pass == 0) || ((b >> (shift + 8)) == (prefix >> (shift + 8)));
            if (match) atomicAdd(&bins[(b >> shift) & 255u], 1u);
        }
        if (bad && pass == 0) atomicOr(status, STWQ_DEV_NONFINITE);
        __syncthreads();
        const uint32_t c = bins[threadIdx.x];
        if (c) atomicAdd(&w.hist[(size_t)p * 256 + threadIdx.x], (unsigned long long)c);
        __syncthreads();
    }
}

// One thread per position: locate the bin that holds the rank, extend the prefix, clear bins.
// raw_out == nullptr: s_tok[p] = delta of the selected |value|. Otherwise the selected signed value
// itself goes to raw_out[p] (0 for a position without rows), and with `mirror` the rank counts from
// the top (rank n + 1 - r), which selects the lower end of a two-sided range.
__global__ void cal_select_kernel(void* base, int P, int pass, uint32_t pct_ppm, int bits,
                                  float* __restrict__ s_tok, float* __restrict__ raw_out, int mirror)
{
    CalWs w = cal_ws(base, P);
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= P) return;
    unsigned long long* h = w.hist + (size_t)p * 256;
    unsigned long long rank = w.rank[p];
    if (pass == 0) {
        unsigned long long n = 0ull;
        for (int i = 0; i < 256; ++i) n += h[i];
        if (n == 0ull) {
            w.rank[p] = 0ull;
            if (raw_out) raw_out[p] = 0.0f;
            else s_tok[p] = 1.0f;
            return;
        }
        rank = ((unsigned long long)pct_ppm * n + 999999ull) / 1000000ull;
        if (rank < 1ull) rank = 1ull;
        if (rank > n) rank = n;
        if (mirror) rank = n + 1ull - rank;
    } else if (rank == 0ull) {
        return;
    }
    const int shift = 24 - 8 * pass;
    unsigned long long cum = 0ull;
    int bin = 255;
    for (int i = 0; i < 256; ++i) {
        const unsigned long long c = h[i];
        if (cum + c >= rank) { bin = i; break; }
        cum += c;
    }
    for (int i = 0; i < 256; ++i) h[i] = 0ull;
    const uint32_t prefix = w.prefix[p] | ((uint32_t)bin << shift);
    w.prefix[p] = prefix;
    w.rank[p] = rank - cum;
    if (pass == 3) {
        if (raw_out) raw_out[p] = __uint_as_float((prefix & 0x80000000u) ? (prefix ^ 0x80000000u) : ~prefix);
        else s_tok[p] = stwq_delta(__uint_as_float(prefix), bits);
    }
}

__global__ void cal_asym_finalize_kernel(const float* __restrict__ up, const float* __restrict__ down, int P, int bits,
                                         float* __restrict__ s_tok, int32_t* __restrict__ z_tok)
{
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= P) return;
    float d;
    int zs;
    stwq_asym_params(down[p], up[p], bits, d, zs);
    s_tok[p] = d;
    z_tok[p] = zs;
}

}  // namespace

size_t stwq_calibrate_ws_bytes(int P)
{
    // histograms, ranks, prefixes, then two float vectors for the two-sided (asymmetric) range
    return (size_t)P * 256 * 8 + (size_t)P * 8 + (size_t)P * 4 + 16 + (size_t)P * 8;
}

int stwq_launch_calibrate(stwq_ctx* ctx, void* ws, const float* Xcal, const int32_t* pos_ids,
                          int64_t rows, int K, int P, const float* s_ch, int bits, uint32_t pct_ppm,
                          float* s_tok, cudaStream_t st)
{
    const int clear_blocks = (int)(((size_t)P * 256 + 255) / 256 < 1024 ? ((size_t)P * 256 + 255) / 256
                                                                          : 1024);
    cal_clear_kernel<<<clear_blocks, 256, 0, st>>>(ws, P);
    ctx->launches += 1;
    int64_t hist_blocks = rows < (int64_t)ctx->sm_count * 16 ? rows : (int64_t)ctx->sm_count * 16;
    for (int pass = 0; pass < 4; ++pass) {
        cal_hist_kernel<<<(unsigned)hist_blocks, kThreads, 0, st>>>(Xcal, pos_ids, rows, K, P, s_ch,
                                                                    ws, pass, 0, ctx->d_status);
        cal_select_kernel<<<(P + 127) / 128, 128, 0, st>>>(ws, P, pass, pct_ppm, bits, s_tok, nullptr, 0);
        ctx->launches += 2;
    }
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

// Two-sided calibration (asymmetric quantizer): the same radix selection on order-preserving keys
// of the signed values, once for the upper end (rank r) and once for the lower (rank n + 1 - r).
int stwq_launch_calibrate_asym(stwq_ctx* ctx, void* ws, const float* Xcal, const int32_t* pos_ids, int64_t rows, int K,
                               int P, const float* s_ch, int bits, uint32_t pct_ppm, float* s_tok, int32_t* z_tok,
                               cudaStream_t st)
{
    float* up = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(ws) + (((size_t)P * 256 * 8 + (size_t)P * 8 + (size_t)P * 4 + 15) & ~(size_t)15));
    float* down = up + P;
    const int clear_blocks = (int)(((size_t)P * 256 + 255) / 256 < 1024 ? ((size_t)P * 256 + 255) / 256 : 1024);
    const int64_t hist_blocks = rows < (int64_t)ctx->sm_count * 16 ? rows : (int64_t)ctx->sm_count * 16;
    for (int side = 0; side < 2; ++side) {
        cal_clear_kernel<<<clear_blocks, 256, 0, st>>>(ws, P);
        ctx->launches += 1;
        for (int pass = 0; pass < 4; ++pass) {
            cal_hist_kernel<<<(unsigned)hist_blocks, kThreads, 0, st>>>(Xcal, pos_ids, rows, K, P, s_ch, ws, pass, 1,
                                                                        ctx->d_status);
            cal_select_kernel<<<(P + 127) / 128, 128, 0, st>>>(ws, P, pass, pct_ppm, bits, nullptr, side == 0 ? up : down,
                                                               side);
            ctx->launches += 2;
        }
    }
    cal_asym_finalize_kernel<<<(P + 127) / 128, 128, 0, st>>>(up, down, P, bits, s_tok, z_tok);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

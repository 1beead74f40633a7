// Quantized attention matmuls and the quantized KV cache (Section 5: all linear layers and matrix
// multiplications run in 6 or 8 bits; Appendix C: so does the KV cache). The two matmuls of a head,
// S = Q K^T and O = P V, run on the tensor cores as batched integer GEMMs (qgemm2 with one matrix
// per head); this file holds what surrounds them:
//
//   rowq_rows_kernel,         rows of Q, K or V -> int8 codes with static scales (the quantizer of
//   rowq_transpose_kernel     Eq. 1 as the linear layers use it: (x * rc[c]) * rt[pos], round to nearest
//                             even, clamp), written densely (Q), at their position in the key cache, or
//                             transposed into the value cache;
//   softmax_quantize_kernel   row softmax of the dequantized scores and the quantizer of the
//                             probabilities: Eq. 1 on the fixed range [0, 1], delta = 1 / (2^b - 1), zero
//                             point 0, unsigned codes.
//
// Readings (the paper names the operands but not their quantizers): queries and keys carry one
// static scale per token position, which factors out of the sum over channels; values carry one
// static scale per channel, because a scale that varied along the keys could not leave the sum over
// keys; the caches hold codes: K as [G, Tmax, d] and V transposed as [G, d, Tmax], so that both
// matmuls read K-major operands.
#include <cuda_bf16.h>

#include "stwq_internal.cuh"

namespace {

constexpr int kRowThreads = 256;

__device__ __forceinline__ uint32_t pack_codes(int q0, int q1, int q2, int q3)
{
    return (uint32_t)(q0 & 0xFF) | ((uint32_t)(q1 & 0xFF) << 8) | ((uint32_t)(q2 & 0xFF) << 16) | ((uint32_t)(q3 & 0xFF) << 24);
}

// Row-major output (Q codes, key cache): a thread per 16 consecutive channels (four 16-byte loads in
// flight, one 16-byte store), consecutive threads along the row and on into the next one.
// out index = g * out_gstride + out_row * d + c, out_row = the row's position (key cache) or its
// index within the matrix (dense output).
__global__ void __launch_bounds__(kRowThreads)
rowq_rows_kernel(const float4* __restrict__ X, int64_t n_vec, int d16, const int32_t* __restrict__ pos_ids, int rows_per_g,
                 int pos0, const float* __restrict__ s_tok, int P, int qmin, int qmax, int8_t* __restrict__ out,
                 int64_t out_gstride, int out_row_from_pos, uint32_t* __restrict__ status)
{
    const int64_t i = (int64_t)blockIdx.x * kRowThreads + threadIdx.x;
    if (i >= n_vec) return;
    const int64_t r = i / d16;
    const int c16 = (int)(i - r * d16);
    const int g = (int)(r / rows_per_g);
    const int t = (int)(r - (int64_t)g * rows_per_g);
    const int pos = pos_ids != nullptr ? pos_ids[t] : pos0 + t;
    const bool ok = pos >= 0 && pos < P;
    if (!ok && c16 == 0) atomicOr(status, STWQ_DEV_POS_RANGE);
    if (out_row_from_pos && !ok) return;                  // no slot in the cache for a position outside [0, P)
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (ok) {
        const float4 v0 = X[4 * i], v1 = X[4 * i + 1], v2 = X[4 * i + 2], v3 = X[4 * i + 3];
        const float rt = __frcp_rn(s_tok[pos]);
        // (x * 1) * rt: no channel scale on queries and keys
        w[0] = pack_codes(stwq_code(__fmul_rn(v0.x, rt), qmin, qmax), stwq_code(__fmul_rn(v0.y, rt), qmin, qmax),
                          stwq_code(__fmul_rn(v0.z, rt), qmin, qmax), stwq_code(__fmul_rn(v0.w, rt), qmin, qmax));
        w[1] = pack_codes(stwq_code(__fmul_rn(v1.x, rt), qmin, qmax), stwq_code(__fmul_rn(v1.y, rt), qmin, qmax),
                          stwq_code(__fmul_rn(v1.z, rt), qmin, qmax), stwq_code(__fmul_rn(v1.w, rt), qmin, qmax));
        w[2] = pack_codes(stwq_code(__fmul_rn(v2.x, rt), qmin, qmax), stwq_code(__fmul_rn(v2.y, rt), qmin, qmax),
                          stwq_code(__fmul_rn(v2.z, rt), qmin, qmax), stwq_code(__fmul_rn(v2.w, rt), qmin, qmax));
        w[3] = pack_codes(stwq_code(__fmul_rn(v3.x, rt), qmin, qmax), stwq_code(__fmul_rn(v3.y, rt), qmin, qmax),
                          stwq_code(__fmul_rn(v3.z, rt), qmin, qmax), stwq_code(__fmul_rn(v3.w, rt), qmin, qmax));
    }
    uint4* o = reinterpret_cast<uint4*>(out + (int64_t)g * out_gstride + (int64_t)(out_row_from_pos ? pos : t) * (d16 * 16));
    o[c16] = make_uint4(w[0], w[1], w[2], w[3]);
}

// Value cache, transposed: a thread takes eight consecutive new positions and four consecutive
// channels (eight 16-byte loads in flight), turns the 8 x 4 block of codes in registers, and writes
// each channel's eight positions as one 8-byte piece of the cache row Vt[g, c, pos0 + t ...]
// (single bytes at a ragged end or when the run does not start on an 8-byte boundary). Four
// consecutive threads cover 32 positions of the same channels, so a warp writes full 32-byte
// sectors. Per-channel scales, no position scale: (x * rc[c]) * 1.
__global__ void __launch_bounds__(kRowThreads)
rowq_transpose_kernel(const float4* __restrict__ V, int G, int d4, int t_new, int pos0, const float4* __restrict__ s_v,
                      int qmin, int qmax, int8_t* __restrict__ Vt, int Tmax)
{
    const int tiles = (t_new + 31) >> 5;
    const int64_t i = (int64_t)blockIdx.x * kRowThreads + threadIdx.x;
    if (i >= (int64_t)G * tiles * d4 * 4) return;
    const int tq = (int)(i & 3);
    int64_t rest = i >> 2;
    const int c4 = (int)(rest % d4);
    rest /= d4;
    const int tile = (int)(rest % tiles);
    const int g = (int)(rest / tiles);
    const int t = tile * 32 + tq * 8;                     // first of this thread's eight positions
    if (t >= t_new) return;
    const int nt = min(8, t_new - t);
    const float4 sv = s_v[c4];
    const float rc[4] = {__frcp_rn(sv.x), __frcp_rn(sv.y), __frcp_rn(sv.z), __frcp_rn(sv.w)};
    float4 v[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        v[r] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < nt) v[r] = V[((int64_t)g * t_new + t + r) * d4 + c4];
    }
    int q[8][4];                                          // [position][channel]
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        q[r][0] = stwq_code(__fmul_rn(v[r].x, rc[0]), qmin, qmax);
        q[r][1] = stwq_code(__fmul_rn(v[r].y, rc[1]), qmin, qmax);
        q[r][2] = stwq_code(__fmul_rn(v[r].z, rc[2]), qmin, qmax);
        q[r][3] = stwq_code(__fmul_rn(v[r].w, rc[3]), qmin, qmax);
    }
    int8_t* o = Vt + ((int64_t)g * d4 * 4 + c4 * 4) * Tmax + pos0 + t;
    const bool wide = nt == 8 && ((pos0 + t) & 7) == 0;   // Tmax is a multiple of 16, the base 16-byte aligned
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        if (wide) {
            *reinterpret_cast<uint2*>(o + (int64_t)c * Tmax) =
                make_uint2(pack_codes(q[0][c], q[1][c], q[2][c], q[3][c]), pack_codes(q[4][c], q[5][c], q[6][c], q[7][c]));
        } else {
#pragma unroll
            for (int r = 0; r < 8; ++r)
                if (r < nt) o[(int64_t)c * Tmax + r] = (int8_t)q[r][c];
        }
    }
}

// Column scales of the keys, followed by zeros up to the padded length.
__global__ void pad_scales_kernel(const float* __restrict__ src, int n, int n_pad, float* __restrict__ dst)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_pad) dst[i] = i < n ? src[i] : 0.0f;
}

// One warp per row of S [rows, ld] (ld >= Tk, padding columns are written as code 0). Causal: query
// i of a matrix (i = row % Tq) sees the keys j <= i + (Tk - Tq).
__global__ void __launch_bounds__(256)
softmax_quantize_kernel(const float* __restrict__ S, int64_t rows, int Tq, int Tk, int ld, int causal, float levels,
                        uint8_t* __restrict__ Pq, float* __restrict__ delta_out)
{
    if (blockIdx.x == 0 && threadIdx.x == 0 && delta_out != nullptr) *delta_out = __fdiv_rn(1.0f, levels);
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int i = (int)(row % Tq);
    const int last = causal ? min(Tk - 1, i + (Tk - Tq)) : Tk - 1;       // last visible key
    const float* s = S + row * ld;
    uint8_t* p = Pq + row * ld;
    float m = -INFINITY;
    for (int j = lane; j <= last; j += 32) m = fmaxf(m, s[j]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float sum = 0.0f;
    for (int j = lane; j <= last; j += 32) sum += exp2f((s[j] - m) * 1.4426950408889634f);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float scale = sum > 0.0f ? __fdiv_rn(levels, sum) : 0.0f;
    for (int j = lane; j < ld; j += 32) {
        float u = 0.0f;
        if (j <= last) u = exp2f((s[j] - m) * 1.4426950408889634f) * scale;
        p[j] = (uint8_t)min(max(__float2int_rn(u), 0), (int)levels);
    }
}

// Few queries against a long cache (a decode step: one new token per head; Section 2). One CTA per
// head and group of up to four queries: the work is reading the head's key and value codes once, so no tensor core is
// involved: integer dot products by dp4a, the score row and its codes in shared memory.
//   1. the query row -> codes (the quantizer of rowq_rows_kernel);
//   2. a thread per key: acc = sum_c Qq[c] Kq[j, c] (the key row is contiguous), S[j] = acc * (s_q * s_kcol[j]);
//   3. row softmax and the quantizer of the probabilities, as in softmax_quantize_kernel;
//   4. a thread per channel and part of the keys: acc = sum_j Pcode[j] Vq[j, c] along the transposed
//      value cache (unsigned x signed dp4a), parts added through shared memory;
//   5. O[c] = acc * (delta_p * s_v[c]).
constexpr int kFewThreads = 256;
__device__ __forceinline__ int dp4a_ss(uint32_t a, uint32_t b, int c)
{
    int r;
    asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
__device__ __forceinline__ int dp4a_us(uint32_t a, uint32_t b, int c)
{
    int r;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
__device__ __forceinline__ float block_reduce(float v, float* scratch, bool is_max)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float w = __shfl_xor_sync(0xffffffffu, v, o);
        v = is_max ? fmaxf(v, w) : v + w;
    }
    __syncthreads();                                      // scratch may still be read from the previous reduction
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float r = scratch[0];
    for (int w = 1; w < kFewThreads / 32; ++w) r = is_max ? fmaxf(r, scratch[w]) : r + scratch[w];
    return r;
}

template <bool BF16, int NQ>
__global__ void __launch_bounds__(kFewThreads)
qattn_few_kernel(const float* __restrict__ Q, const int32_t* __restrict__ pos_q, int Tq, int Tk, int Tk_pad, int d, int Tmax,
                 const int8_t* __restrict__ Kc, const int8_t* __restrict__ Vt, const float* __restrict__ s_q,
                 const float* __restrict__ s_kcol, const float* __restrict__ s_v, int P, int qmin, int qmax, float levels,
                 int causal, void* __restrict__ O, uint32_t* __restrict__ status)
{
    // NQ consecutive queries of one head per CTA: every key and value code that is read serves all of them
    extern __shared__ __align__(16) uint8_t few_smem[];
    float* S = reinterpret_cast<float*>(few_smem);                       // [NQ][Tk_pad]
    uint8_t* Pc = few_smem + (size_t)NQ * Tk_pad * 4;                     // [NQ][Tk_pad] codes, zero beyond the visible keys
    uint32_t* q8 = reinterpret_cast<uint32_t*>(Pc + (size_t)NQ * Tk_pad); // [NQ][d / 4] packed query codes
    int* part = reinterpret_cast<int*>(q8 + NQ * (d / 4));                // [NQ][kFewThreads] partial sums of step 4
    __shared__ float scratch[kFewThreads / 32];
    __shared__ float sq_sh[NQ];
    const int nqb = (Tq + NQ - 1) / NQ;
    const int g = blockIdx.x / nqb, i0 = (blockIdx.x - g * nqb) * NQ;
    const int nq = min(NQ, Tq - i0);
    const int tid = threadIdx.x;
    // 1. query codes
    for (int t = tid; t < NQ * (d / 4); t += kFewThreads) {
        const int q = t / (d / 4), c4 = t - q * (d / 4);
        uint32_t w = 0;
        if (q < nq) {
            const int pos = pos_q[i0 + q];
            const bool ok = pos >= 0 && pos < P;
            if (!ok && c4 == 0 && g == 0) atomicOr(status, STWQ_DEV_POS_RANGE);
            const float sq = ok ? s_q[pos] : 0.0f;
            if (c4 == 0) sq_sh[q] = sq;
            if (ok) {
                const float rt = __frcp_rn(sq);
                const float4 x = reinterpret_cast<const float4*>(Q + ((int64_t)g * Tq + i0 + q) * d)[c4];
                w = (uint32_t)(stwq_code(__fmul_rn(x.x, rt), qmin, qmax) & 0xFF) | ((uint32_t)(stwq_code(__fmul_rn(x.y, rt), qmin, qmax) & 0xFF) << 8) |
                    ((uint32_t)(stwq_code(__fmul_rn(x.z, rt), qmin, qmax) & 0xFF) << 16) | ((uint32_t)(stwq_code(__fmul_rn(x.w, rt), qmin, qmax) & 0xFF) << 24);
            }
        } else if (c4 == 0) {
            sq_sh[q] = 0.0f;
        }
        q8[t] = w;
    }
    __syncthreads();
    // 2. scores: a thread per key, the key row dotted with every query
    int last[NQ];                                          // last visible key of each query
    float m[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        last[q] = q < nq ? (causal ? min(Tk - 1, i0 + q + (Tk - Tq)) : Tk - 1) : -1;
        m[q] = -INFINITY;
    }
    const int last_all = causal ? min(Tk - 1, i0 + nq - 1 + (Tk - Tq)) : Tk - 1;      // the latest query sees the most keys
    const int8_t* Kg = Kc + (int64_t)g * Tmax * d;
    for (int j = tid; j <= last_all; j += kFewThreads) {
        const uint4* krow = reinterpret_cast<const uint4*>(Kg + (int64_t)j * d);
        int acc[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) acc[q] = 0;
        for (int c = 0; c < d / 16; ++c) {
            const uint4 k = __ldg(krow + c);
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const uint4 qq = reinterpret_cast<const uint4*>(q8 + q * (d / 4))[c];
                acc[q] = dp4a_ss(qq.w, k.w, dp4a_ss(qq.z, k.z, dp4a_ss(qq.y, k.y, dp4a_ss(qq.x, k.x, acc[q]))));
            }
        }
        const float skc = s_kcol[j];
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            if (j <= last[q]) {
                const float sc = __fmul_rn((float)acc[q], __fmul_rn(sq_sh[q], skc));
                S[(size_t)q * Tk_pad + j] = sc;
                m[q] = fmaxf(m[q], sc);
            }
        }
    }
    // 3. softmax and codes, query by query
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        if (q >= nq) break;                                // uniform over the block
        float* Sq = S + (size_t)q * Tk_pad;
        uint8_t* Pq = Pc + (size_t)q * Tk_pad;
        const float mq = block_reduce(m[q], scratch, true);
        float sum = 0.0f;
        for (int j = tid; j <= last[q]; j += kFewThreads) sum += exp2f((Sq[j] - mq) * 1.4426950408889634f);
        sum = block_reduce(sum, scratch, false);
        const float scale = sum > 0.0f ? __fdiv_rn(levels, sum) : 0.0f;
        for (int j = tid; j < Tk_pad; j += kFewThreads) {
            float u = 0.0f;
            if (j <= last[q]) u = exp2f((Sq[j] - mq) * 1.4426950408889634f) * scale;
            Pq[j] = (uint8_t)min(max(__float2int_rn(u), 0), (int)levels);
        }
    }
    __syncthreads();
    // 4. O accumulators: thread = (part of the keys, channel); a part is a multiple of 16 keys
    const int parts = max(1, kFewThreads / d);
    const int n16 = Tk_pad / 16;                          // 16-key pieces; those beyond the last visible key hold zero codes
    const float delta_p = __fdiv_rn(1.0f, levels);
    for (int c0 = 0; c0 < d; c0 += kFewThreads) {         // one pass unless d > 256 threads
        const int c = c0 + (parts > 1 ? tid % d : tid);
        const int prt = parts > 1 ? tid / d : 0;
        int acc[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) acc[q] = 0;
        if (c < d && prt < parts) {
            const uint4* vrow = reinterpret_cast<const uint4*>(Vt + ((int64_t)g * d + c) * Tmax);
            const int per = (n16 + parts - 1) / parts;
            const int e = min(n16, (prt + 1) * per);
            for (int t = prt * per; t < e; ++t) {
                if (t * 16 > last_all) break;             // nothing but zero codes from here on
                const uint4 v = __ldg(vrow + t);
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    const uint4 pc = reinterpret_cast<const uint4*>(Pc + (size_t)q * Tk_pad)[t];
                    acc[q] = dp4a_us(pc.w, v.w, dp4a_us(pc.z, v.z, dp4a_us(pc.y, v.y, dp4a_us(pc.x, v.x, acc[q]))));
                }
            }
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < NQ; ++q) part[q * kFewThreads + tid] = acc[q];
        __syncthreads();
        if (c < d && prt == 0) {
            const float sc = __fmul_rn(delta_p, s_v[c]);
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                if (q >= nq) break;
                int total = acc[q];
                for (int w = 1; w < parts; ++w) total += part[q * kFewThreads + w * d + (tid % d)];
                // 5. dequantize
                const float o = __fmul_rn((float)total, sc);
                const int64_t idx = ((int64_t)g * Tq + i0 + q) * d + c;
                if (BF16) static_cast<__nv_bfloat16*>(O)[idx] = __float2bfloat16_rn(o);
                else static_cast<float*>(O)[idx] = o;
            }
        }
    }
}

int launch_rows(stwq_ctx* ctx, const float* X, int64_t rows, int d, const int32_t* pos_ids, int rows_per_g, int pos0,
                const float* s_tok, int P, int bits, int8_t* out, int64_t gs, int from_pos, cudaStream_t st)
{
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    const int64_t n_vec = rows * (d / 16);
    const int64_t blocks = (n_vec + kRowThreads - 1) / kRowThreads;
    if (blocks > 0x7fffffff) return STWQ_ERR_DIM;
    rowq_rows_kernel<<<(unsigned)blocks, kRowThreads, 0, st>>>(reinterpret_cast<const float4*>(X), n_vec, d / 16, pos_ids,
                                                               rows_per_g, pos0, s_tok, P, qmin, qmax, out, gs, from_pos,
                                                               ctx->d_status);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

int launch_transpose(stwq_ctx* ctx, const float* V, int G, int t_new, int d, int pos0, const float* s_v, int bits, int8_t* Vt,
                     int Tmax, cudaStream_t st)
{
    const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
    const int64_t n_thr = (int64_t)G * ((t_new + 31) / 32) * (d / 4) * 4;
    const int64_t blocks = (n_thr + kRowThreads - 1) / kRowThreads;
    if (blocks > 0x7fffffff) return STWQ_ERR_DIM;
    rowq_transpose_kernel<<<(unsigned)blocks, kRowThreads, 0, st>>>(reinterpret_cast<const float4*>(V), G, d / 4, t_new, pos0,
                                                                    reinterpret_cast<const float4*>(s_v), qmin, qmax, Vt, Tmax);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

struct DevGuard {
    int prev = -1;
    bool switched = false;
    explicit DevGuard(int dev)
    {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) {
            cudaSetDevice(dev);
            switched = true;
        }
    }
    ~DevGuard()
    {
        if (switched) cudaSetDevice(prev);
    }
};

// Workspace of one qattention call: codes of Q, scores, probability codes, the padded key-column
// scales and the probability step.
struct AttnWs {
    int8_t* Qq;
    float* S;
    uint8_t* Pq;
    float* skcol;
    float* delta_p;
    size_t bytes;
};
// staged = false: the one-kernel head keeps scores and probability codes on the SM
AttnWs attn_layout(void* base, int64_t G, int64_t Tq, int64_t Tk_pad, int64_t d, bool staged)
{
    AttnWs w;
    size_t off = 0;
    auto take = [&](size_t n) { size_t o = off; off = (size_t)round_up((int64_t)(off + n), 256); return o; };
    const size_t oq = take(staged ? (size_t)(G * Tq * d) : 0);
    const size_t os = take(staged ? (size_t)(G * Tq * Tk_pad) * 4 : 0);
    const size_t op = take(staged ? (size_t)(G * Tq * Tk_pad) : 0);
    const size_t ok = take((size_t)round_up(Tk_pad, 128) * 4);
    const size_t od = take(256);
    uint8_t* b = static_cast<uint8_t*>(base);
    w.Qq = reinterpret_cast<int8_t*>(b + oq);
    w.S = reinterpret_cast<float*>(b + os);
    w.Pq = b + op;
    w.skcol = reinterpret_cast<float*>(b + ok);
    w.delta_p = reinterpret_cast<float*>(b + od);
    w.bytes = off;
    return w;
}

}  // namespace

extern "C" {

int kv_append(stwq_ctx* ctx, const float* Knew, const float* Vnew, int G, int t_new, int d, int pos0, int Tmax,
              const float* s_k, const float* s_v, int P, int bits, int8_t* Kc, int8_t* Vt, void* stream)
{
    if (!ctx || !Knew || !Vnew || !s_k || !s_v || !Kc || !Vt) return STWQ_ERR_NULL;
    if (G <= 0 || t_new <= 0 || d <= 0 || Tmax <= 0 || P <= 0 || pos0 < 0) return STWQ_ERR_DIM;
    if ((int64_t)pos0 + t_new > Tmax || (int64_t)pos0 + t_new > P) return STWQ_ERR_DIM;
    if (bits != 8 && bits != 6) return STWQ_ERR_BITS;
    if ((d & 15) != 0 || (Tmax & 15) != 0 || !aligned16(Knew) || !aligned16(Vnew) || !aligned16(s_v) || !aligned16(Kc) || !aligned16(Vt))
        return STWQ_ERR_ALIGN;
    DevGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t rows = (int64_t)G * t_new;
    int rc = launch_rows(ctx, Knew, rows, d, nullptr, t_new, pos0, s_k, P, bits, Kc, (int64_t)Tmax * d, 1, st);
    if (rc != STWQ_OK) return rc;
    return launch_transpose(ctx, Vnew, G, t_new, d, pos0, s_v, bits, Vt, Tmax, st);
}

int stwq_reserve_attention(stwq_ctx* ctx, int G, int Tq, int Tk, int d)
{
    if (!ctx) return STWQ_ERR_NULL;
    if (G <= 0 || Tq <= 0 || Tk <= 0 || d <= 0) return STWQ_ERR_DIM;
    DevGuard g(ctx->device);
    const AttnWs w = attn_layout(nullptr, G, Tq, round_up(Tk, 16), d, ctx->debug == 9);
    return stwq_ensure_ws(ctx, &ctx->ws_attn, &ctx->ws_attn_bytes, w.bytes, nullptr, 0);
}

int qattention(stwq_ctx* ctx, const float* Q, const int32_t* pos_q, int G, int Tq, int Tk, int d, int Tmax,
               const int8_t* Kc, const int8_t* Vt, const float* s_q, const float* s_kcol, const float* s_v, int P,
               int bits, int causal, int out_dtype, void* O, void* stream)
{
    if (!ctx || !Q || !pos_q || !Kc || !Vt || !s_q || !s_kcol || !s_v || !O) return STWQ_ERR_NULL;
    if (G <= 0 || Tq <= 0 || Tk <= 0 || d <= 0 || Tmax <= 0 || P <= 0) return STWQ_ERR_DIM;
    if (Tk > Tmax || (causal && Tq > Tk) || d > 256) return STWQ_ERR_DIM;
    if (bits != 8 && bits != 6) return STWQ_ERR_BITS;
    if (out_dtype != STWQ_OUT_F32 && out_dtype != STWQ_OUT_BF16) return STWQ_ERR_BITS;
    if ((d & 15) != 0 || (Tmax & 15) != 0 || !aligned16(Q) || !aligned16(Kc) || !aligned16(Vt) || !aligned16(O) ||
        !aligned16(s_v))
        return STWQ_ERR_ALIGN;
    DevGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t Tk_pad = round_up(Tk, 16);
    const bool staged = ctx->debug == 9;                  // the three stages as separate kernels
    // a decode step: few queries against a long cache. Bound by reading the cache once, done by one
    // CTA per (head, query) without the tensor cores
    const int nq_cta = Tq == 1 ? 1 : (Tq == 2 ? 2 : 4);   // queries of a head that share one read of its cache
    const size_t few_smem = (size_t)nq_cta * ((size_t)Tk_pad * 5 + (size_t)d + kFewThreads * 4) + 16;
    const int64_t few_ctas = (int64_t)G * ((Tq + nq_cta - 1) / nq_cta);
    if (!staged && Tq <= 8 && few_smem <= 200 * 1024 && few_ctas <= 0x7fffffff) {
        const int qmax = (1 << (bits - 1)) - 1, qmin = -(1 << (bits - 1));
        const float lv = (float)((1 << bits) - 1);
        auto launch = [&](auto kern) -> int {
            cudaError_t e1 = cudaSuccess;
            if (few_smem > 48 * 1024) e1 = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            if (e1 != cudaSuccess) return stwq_cuda_fail(ctx, e1);
            kern<<<(unsigned)few_ctas, kFewThreads, few_smem, st>>>(Q, pos_q, Tq, Tk, (int)Tk_pad, d, Tmax, Kc, Vt, s_q, s_kcol, s_v, P, qmin,
                                                                   qmax, lv, causal ? 1 : 0, O, ctx->d_status);
            ctx->launches += 1;
            e1 = cudaGetLastError();
            return e1 == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e1);
        };
        const bool bf = out_dtype == STWQ_OUT_BF16;
        if (nq_cta == 1) return bf ? launch(qattn_few_kernel<true, 1>) : launch(qattn_few_kernel<false, 1>);
        if (nq_cta == 2) return bf ? launch(qattn_few_kernel<true, 2>) : launch(qattn_few_kernel<false, 2>);
        return bf ? launch(qattn_few_kernel<true, 4>) : launch(qattn_few_kernel<false, 4>);
    }
    AttnWs w = attn_layout(nullptr, G, Tq, Tk_pad, d, staged);
    int rc = stwq_ensure_ws(ctx, &ctx->ws_attn, &ctx->ws_attn_bytes, w.bytes, st, 0);
    if (rc != STWQ_OK) return rc;
    w = attn_layout(ctx->ws_attn, G, Tq, Tk_pad, d, staged);

    // key-column scales, padded with zeros (to the 16-column pitch of the score matrix; to whole
    // chunks of 128 keys for the one-kernel head)
    const int n_pad = (int)round_up(Tk_pad, 128);
    pad_scales_kernel<<<(n_pad + 255) / 256, 256, 0, st>>>(s_kcol, Tk, n_pad, w.skcol);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
    if (!staged)                                          // quantizes its queries itself
        return stwq_launch_qattn_fused(ctx, Q, pos_q, G, Tq, Tk, d, Tmax, Kc, Vt, s_q, w.skcol, s_v, P, bits, causal, out_dtype,
                                       O, st);
    // queries -> codes with their per-position scales
    rc = launch_rows(ctx, Q, (int64_t)G * Tq, d, pos_q, Tq, 0, s_q, P, bits, w.Qq, (int64_t)Tq * d, 0, st);
    if (rc != STWQ_OK) return rc;
    // S = dequantized Q K^T, one matrix per head: rows scaled by s_q[pos], columns by s_kcol
    stwq_batch bq = {G, (int64_t)d, (int64_t)Tmax * d, 0, 1, 0};
    rc = stwq_launch_qgemm2(ctx, w.Qq, pos_q, Tq, d, (int)Tk_pad, Kc, w.skcol, s_q, P, nullptr, STWQ_ACT_NONE, STWQ_OUT_F32,
                            w.S, false, nullptr, st, nullptr, &bq);
    if (rc != STWQ_OK) return rc;
    // probabilities -> unsigned codes (and the step 1 / (2^b - 1) for the second dequantizer)
    const float levels = (float)((1 << bits) - 1);
    const int64_t rows = (int64_t)G * Tq;
    softmax_quantize_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(w.S, rows, Tq, Tk, (int)Tk_pad, causal ? 1 : 0, levels,
                                                                       w.Pq, w.delta_p);
    ctx->launches += 1;
    e = cudaGetLastError();
    if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
    // O = dequantized P V: unsigned probability codes times the transposed value cache, scaled by
    // delta_p (one "position") and the value channels' scales
    stwq_batch bp = {G, (int64_t)Tmax, (int64_t)d * Tmax, 0, 1, 1};
    return stwq_launch_qgemm2(ctx, reinterpret_cast<const int8_t*>(w.Pq), nullptr, Tq, (int)Tk_pad, d, Vt, s_v, w.delta_p, 1,
                              nullptr, STWQ_ACT_NONE, out_dtype, O, false, nullptr, st, nullptr, &bp);
}

// The stages of qattention on their own (tests compare each with the CPU definition).
int qattn_softmax_quantize(stwq_ctx* ctx, const float* S, int64_t rows, int Tq, int Tk, int ld, int causal, int bits,
                           uint8_t* Pq, void* stream)
{
    if (!ctx || !S || !Pq) return STWQ_ERR_NULL;
    if (rows <= 0 || Tq <= 0 || Tk <= 0 || ld < Tk || (causal && Tq > Tk)) return STWQ_ERR_DIM;
    if (bits != 8 && bits != 6) return STWQ_ERR_BITS;
    DevGuard g(ctx->device);
    softmax_quantize_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        S, rows, Tq, Tk, ld, causal ? 1 : 0, (float)((1 << bits) - 1), Pq, nullptr);
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

int qattn_pv(stwq_ctx* ctx, const uint8_t* Pq, int G, int Tq, int Tk_pad, int d, int Tmax, const int8_t* Vt,
             const float* s_v, const float* delta_p, int out_dtype, void* O, void* stream)
{
    if (!ctx || !Pq || !Vt || !O) return STWQ_ERR_NULL;
    if (out_dtype != STWQ_OUT_INT32 && (!s_v || !delta_p)) return STWQ_ERR_NULL;
    if (G <= 0 || Tq <= 0 || Tk_pad <= 0 || d <= 0 || Tk_pad > Tmax || d > 256) return STWQ_ERR_DIM;
    if (out_dtype < STWQ_OUT_F32 || out_dtype > STWQ_OUT_INT32) return STWQ_ERR_BITS;
    if ((d & 15) != 0 || (Tmax & 15) != 0 || (Tk_pad & 15) != 0 || !aligned16(Pq) || !aligned16(Vt) || !aligned16(O) ||
        (s_v && !aligned16(s_v)))
        return STWQ_ERR_ALIGN;
    DevGuard g(ctx->device);
    stwq_batch bp = {G, (int64_t)Tmax, (int64_t)d * Tmax, 0, 1, 1};
    return stwq_launch_qgemm2(ctx, reinterpret_cast<const int8_t*>(Pq), nullptr, Tq, Tk_pad, d, Vt, s_v, delta_p, 1, nullptr,
                              STWQ_ACT_NONE, out_dtype, O, false, nullptr, static_cast<cudaStream_t>(stream), nullptr, &bp);
}

}  // extern "C"

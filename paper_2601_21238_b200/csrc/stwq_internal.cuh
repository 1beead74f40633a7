// Internal declarations shared by the translation units of libstwq.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "stwq.h"

// Bits of the device status word (OR-ed by kernels, read by stwq_device_status).
#define STWQ_DEV_POS_RANGE 1u
#define STWQ_DEV_NONFINITE 2u
#define STWQ_DEV_TIMEOUT 4u

struct stwq_ctx {
    int device;
    int sm_count;
    int l2_bytes;
    int last_cuda_error;
    int gemm_path;             // STWQ_OPT_GEMM_PATH
    int wait_limit_ms;         // STWQ_OPT_WAIT_LIMIT_MS
    int64_t launches;
    int force_bn;              // tuning: 0 = choose, 128 / 256 = force the tile width
    int debug;                 // tuning: variant of the pair GEMM (epilogue store mode, prefetch distance)
    int quant_blocks_per_sm;   // resident blocks per SM of the quantize kernel (0 = not yet queried)
    int quant_blocks_per_sm2;  // the same for its 256-column-span variant
    int quant_ring_configured; // the ring quantize kernel has its shared-memory attribute set
    int max_pairs;             // CTA pairs of the pair GEMM that can be resident at once (0 = not yet queried)
    uint64_t configured_mask;  // kernels whose shared-memory attribute is already set (single-CTA GEMM)
    uint64_t configured_pair[4]; // the same for the pair GEMM, one mask per kernel variant
    uint32_t* d_status;        // device status word
    int8_t* ws_xq;             // workspace: int8 copy of X for qlinear
    size_t ws_xq_bytes;
    void* ws_dyn;              // workspace of qlinear_dtwq: per-row scales [M] and row ids [M]
    size_t ws_dyn_bytes;
    void* ws_cal;              // workspace: calibration histograms and selection state
    size_t ws_cal_bytes;
    void* ws_dec;              // split-K workspace: arrival counters, then int32 partial sums
    size_t ws_dec_bytes;
    uint64_t configured_decode;
    void* ws_attn;             // workspace of qattention: codes of Q, scores, probability codes
    size_t ws_attn_bytes;
    int8_t* ws_w4;             // workspace: int8 copy of packed 4-bit weights (qlinear_w4 on the tiled route)
    size_t ws_w4_bytes;
    int force_ksplit;          // tuning: 0 = choose, else the number of K ranges of the few-row path
    uint64_t ws_generation;    // bumped whenever a workspace buffer is (re)allocated
    int probe_configured;      // the peak-probe kernel has its shared-memory attribute set
    int attn_configured;       // so has the one-kernel attention head
    int attn_few_configured;   // and the few-query attention kernel
    void* encode_tiled;        // cuTensorMapEncodeTiled, resolved at create
};

// The next layer's static quantizer, applied by the GEMM epilogue when the output type is 3
// (int8 codes for the next linear instead of Y): s_ch_next [N] or NULL, s_tok_next [P].
struct stwq_chain {
    const float* s_ch_next;
    const float* s_tok_next;
    int bits_next;
};

// Zero points of the asymmetric quantizer (Eq. 1 as printed) and the sums its correction needs.
struct stwq_asym {
    const int32_t* z_tok;      // [P] signed zero point per position
    const int32_t* z_w;        // [N] signed zero point per output channel
    const int32_t* colsum;     // [N] sum_k Wq[n,k]
    const int32_t* rowcorr;    // [M] sum_k Xq[m,k] - K z_tok[pos[m]]
};

// Batched operands of the CTA-pair GEMM (one matrix per attention head): A [G, M, K] and Y [G, M, N]
// dense; B [G, N, K] with rows ldb bytes apart and matrices b_gstride bytes apart.
struct stwq_batch {
    int G;
    int64_t ldb, b_gstride;
    int64_t sw_gstride;        // elements between the column-scale vectors of two matrices (0 = one vector for all)
    int pos_shared;            // pos_ids has M entries shared by all matrices (else G * M)
    int a_unsigned;            // A holds unsigned 8-bit codes (attention probabilities)
};

// Launchers (host). Each returns STWQ_OK or STWQ_ERR_CUDA and bumps ctx->launches.
int stwq_launch_quantize(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K,
                         const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq,
                         bool dependent, cudaStream_t st);
int stwq_launch_quantize_bf16(stwq_ctx* ctx, const void* X, const int32_t* pos_ids, int64_t M, int K,
                              const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq, cudaStream_t st);
int stwq_launch_fold_asym(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, int bits, int8_t* Wq,
                          float* s_w, int32_t* z_w, int32_t* colsum, cudaStream_t st);
int stwq_launch_quantize_asym(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, const float* s_ch,
                              const float* s_tok, const int32_t* z_tok, int P, int bits, int8_t* Xq, int32_t* rowcorr,
                              cudaStream_t st);
int stwq_launch_calibrate_asym(stwq_ctx* ctx, void* ws, const float* Xcal, const int32_t* pos_ids, int64_t rows, int K,
                               int P, const float* s_ch, int bits, uint32_t pct_ppm, float* s_tok, int32_t* z_tok,
                               cudaStream_t st);
int stwq_launch_fold_packed4(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, uint8_t* Wp, float* s_w,
                             cudaStream_t st);
int stwq_launch_unpack4(stwq_ctx* ctx, const uint8_t* Wp, int64_t packed_bytes, int8_t* Wq, cudaStream_t st);
int stwq_launch_fold(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, int bits,
                     int8_t* Wq, float* s_w, cudaStream_t st);
size_t stwq_calibrate_ws_bytes(int P);
size_t stwq_gps_ws_bytes(int K, int N);
size_t stwq_dgc_ws_bytes(int D);
int stwq_launch_qattn_fused(stwq_ctx* ctx, const float* Q, const int32_t* pos_q, int G, int Tq, int Tk, int d, int Tmax,
                            const int8_t* Kc, const int8_t* Vt, const float* s_q, const float* s_kcol_pad, const float* s_v,
                            int P, int bits, int causal, int out_dtype, void* O, cudaStream_t st);
int stwq_launch_dgc(stwq_ctx* ctx, void* ws, const float* F, int n, int D, int k, double ridge, double* rho,
                    int32_t* selected, cudaStream_t st);
int stwq_launch_gps(stwq_ctx* ctx, void* ws_cal, void* ws, const float* X, int64_t T, int K, const float* W, int N,
                    int bits, uint32_t pct_ppm, int variant, float* s, int32_t* k_star_out, cudaStream_t st);
int stwq_launch_calibrate(stwq_ctx* ctx, void* ws, const float* Xcal, const int32_t* pos_ids,
                          int64_t rows, int K, int P, const float* s_ch, int bits, uint32_t pct_ppm,
                          float* s_tok, cudaStream_t st);
int stwq_launch_qgemm(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K,
                      int N, const int8_t* Wq, const float* s_w, const float* s_tok, int P,
                      const float* bias, int act, int out_dtype, void* Y, cudaStream_t st);
bool stwq_qgemm2_supported(int N, int out_dtype, const float* s_w, const float* bias);
int stwq_launch_qgemm2(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K,
                       int N, const int8_t* Wq, const float* s_w, const float* s_tok, int P,
                       const float* bias, int act, int out_dtype, void* Y, bool after_quantize,
                       const struct stwq_chain* chain, cudaStream_t st, const struct stwq_asym* asym = nullptr,
                       const struct stwq_batch* batch = nullptr);
int stwq_launch_decode(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K,
                       int N, const int8_t* Wq, const float* s_w, const float* s_tok, int P,
                       const float* bias, int act, int out_dtype, void* Y, bool after_quantize, cudaStream_t st);

int stwq_launch_dtwq(stwq_ctx* ctx, const float* X, int64_t M, int K, const float* s_ch, int bits, int8_t* Xq,
                     float* s_row, int32_t* row_ids, cudaStream_t st);
size_t stwq_decode_split_bytes(const stwq_ctx* ctx, int K, int N);
int stwq_split_ws(stwq_ctx* ctx, size_t partial_bytes, size_t n_counters, uint32_t** counters, int32_t** partial,
                  cudaStream_t st);
// Grow one workspace buffer of the context to `bytes` (no-op if it is large enough). Refused with
// STWQ_ERR_CAPTURE while `st` is being captured; the first zero_prefix bytes of a new buffer are cleared.
int stwq_ensure_ws(stwq_ctx* ctx, void** buf, size_t* have, size_t bytes, cudaStream_t st, size_t zero_prefix);

static inline int stwq_cuda_fail(stwq_ctx* ctx, cudaError_t e)
{
    if (ctx) ctx->last_cuda_error = (int)e;
    return STWQ_ERR_CUDA;
}

#ifdef __CUDACC__
// delta of the symmetric b-bit quantizer with range [-a, a]: 2a / (2^b - 1) in IEEE fp32,
// 1 for a == 0, floored at 2^-64.
__device__ __forceinline__ float stwq_delta(float a, int bits)
{
    if (!(a > 0.0f)) return 1.0f;
    const float levels = (float)((1 << bits) - 1);
    float d = __fdiv_rn(__fadd_rn(a, a), levels);
    return fmaxf(d, 5.421010862427522e-20f);
}

// Eq. 1 as printed, for a range widened to contain 0: delta = (up - down) / (2^b - 1), z =
// round(-down / delta) clamped to [0, 2^b - 1]; returned as the signed zero point z - 2^(b-1)
// that goes with codes stored in signed containers.
__device__ __forceinline__ void stwq_asym_params(float lo, float hi, int bits, float& delta, int& zs)
{
    const float levels = (float)((1 << bits) - 1);
    if (lo > 0.0f) lo = 0.0f;
    if (hi < 0.0f) hi = 0.0f;
    float d = __fdiv_rn(__fsub_rn(hi, lo), levels);
    if (!(d > 0.0f)) d = 1.0f;
    d = fmaxf(d, 5.421010862427522e-20f);
    float z = rintf(__fdiv_rn(-lo, d));
    z = fminf(fmaxf(z, 0.0f), levels);
    delta = d;
    zs = (int)z - (1 << (bits - 1));
}
// signed asymmetric code: clamp(round(u) + zs) (NaN -> round 0; the rounded value saturates at +-2^20 first)
__device__ __forceinline__ int stwq_code_asym(float u, int zs, int qmin, int qmax)
{
    const int r = max(min(__float2int_rn(u), 1048576), -1048576);
    return max(min(r + zs, qmax), qmin);
}

// round to nearest even (NaN -> 0, +-Inf and large values saturate), clamp to the b-bit range.
// Rounding then clamping equals clamping then rounding because the bounds are integers.
__device__ __forceinline__ int stwq_code(float u, int qmin, int qmax)
{
    return max(min(__float2int_rn(u), qmax), qmin);
}
#endif

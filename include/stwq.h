/*
 * libstwq - static-token-wise-quantized (STWQ) linear layer for NVIDIA B200 (sm_100a).
 *
 * The inference hot path of PTQ4ARVG's quantized decoder, as a C library:
 *
 *   offline   stwq_calibrate   per-token-position activation scales      (Section 4.2)
 *   offline   gps_scales       the per-channel scaling vector s of Eq. 2        (Section 4.1, Algorithm 1)
 *   offline   gps_fold         fold the per-channel scale into W, quantize W (Eq. 2, Appendix B)
 *   online    stwq_quantize    X -> int8 codes with the static scales     (Eq. 1, Eq. 2, Section 4.2)
 *   online    qlinear          quantize -> int8 GEMM -> dequantize (+bias, +GELU)
 *   online    qlinear_q        the same from precomputed codes
 * and, beside the path: chained layers, bf16 activations, the asymmetric quantizer, the dynamic
 * token-wise baseline, packed 4-bit weights, quantized attention with a quantized KV cache, and the
 * selection of calibration samples (each documented at its declaration below).
 *
 * Notation: M rows (tokens x batch), K input channels (the paper's n), N output
 * channels (the paper's m), P token positions (the paper's T), b in {8, 6} bits,
 * qmin = -2^(b-1), qmax = 2^(b-1) - 1, D = 2^b - 1.
 *
 * Conventions for every call
 *  - Every pointer is a DEVICE pointer owned by the caller unless it is said to be a host
 *    pointer. The library never frees or keeps caller memory. Matrices are row-major and
 *    dense: X [M,K], W and Wq [N,K] (the nn.Linear layout, i.e. the paper's W transposed),
 *    Y [M,N].
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Calls
 *    enqueue work and return; they do not synchronise, except where stated.
 *  - Return value: STWQ_OK (0) or a negative STWQ_ERR_* code. Argument errors are detected
 *    on the host before anything is enqueued. Errors only the device can see (a pos_id
 *    outside [0,P), a non-finite calibration value, a device-side wait that ran out) are
 *    recorded in the context and read with stwq_device_status().
 *  - A context may be used from one host thread at a time, and its calls share its workspace
 *    (the int8 copy of X, per-row scratch, calibration and split-K buffers): calls on one
 *    context that could overlap on the device (different streams without an ordering between
 *    them) race. Use one context per stream that runs concurrently.
 *  - Alignment: X, Xq, Wq, Y 16-byte aligned; K a multiple of 16.
 */
#ifndef STWQ_H
#define STWQ_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default)   /* the entry points below are the library's only exports */
#endif

typedef struct stwq_ctx stwq_ctx;

enum {
    STWQ_OK = 0,
    STWQ_ERR_NULL = -1,           /* a required pointer is NULL                              */
    STWQ_ERR_DIM = -2,            /* a size is zero, negative or beyond what is supported    */
    STWQ_ERR_ALIGN = -3,          /* pointer or K alignment rule violated                    */
    STWQ_ERR_BITS = -4,           /* bits not 6 or 8 (4 too for weights), or act / out_dtype / pct invalid */
    STWQ_ERR_ARCH = -5,           /* the device is not compute capability 10.x               */
    STWQ_ERR_CUDA = -6,           /* a CUDA call failed; see stwq_last_cuda_error()          */
    STWQ_ERR_DEVICE_TIMEOUT = -7, /* a bounded device-side wait expired; output is invalid   */
    STWQ_ERR_POS_RANGE = -8,      /* a pos_id was outside [0,P); that row was written as 0   */
    STWQ_ERR_NONFINITE = -9,      /* calibration saw NaN or Inf                              */
    STWQ_ERR_NOMEM = -10,         /* workspace allocation failed                             */
    STWQ_ERR_CAPTURE = -11        /* the call would have to (re)allocate workspace while its stream is being
                                     captured into a CUDA graph; reserve the workspace before capturing */
};

/*
 * Activation applied by the epilogue.
 *   STWQ_ACT_GELU_ERF   y = z Phi(z), with Phi(-|z|) = erfc(|z| / sqrt2) / 2 as one exp2 of a fitted
 *                       polynomial (absolute error on Phi below 1.5e-7), for every output type.
 *   STWQ_ACT_GELU_TANH  y = z/2 (1 + tanh(sqrt(2/pi)(z + 0.044715 z^3))), evaluated as z sigmoid(2u) in fp32.
 *   STWQ_ACT_GELU_FAST  the tanh form with the hardware's approximate tanh (relative error about 2^-11 on
 *                       tanh, i.e. up to 6e-4 |z| on y): six instructions per element instead of about
 *                       twenty. Meant for bf16 output (rounding unit 2^-9), where it stays inside the 1e-2
 *                       tolerance of either GELU form; chained codes computed with it can differ by one
 *                       from those of the exact activation.
 */
enum { STWQ_ACT_NONE = 0, STWQ_ACT_GELU_ERF = 1, STWQ_ACT_GELU_TANH = 2, STWQ_ACT_GELU_FAST = 3 };
/* element type of Y. INT32 returns the raw accumulators (no scale, bias or activation). */
enum { STWQ_OUT_F32 = 0, STWQ_OUT_BF16 = 1, STWQ_OUT_INT32 = 2 };

/*
 * Create a context on `device` (a CUDA ordinal). Synchronous. Allocates a small status
 * word and, lazily, workspace (the int8 copy of X used by qlinear, calibration histograms).
 * Fails with STWQ_ERR_ARCH unless the device is compute capability 10.x.
 * stwq_destroy frees everything the context allocated; it synchronises the device.
 */
int stwq_create(stwq_ctx** out, int device);
void stwq_destroy(stwq_ctx* ctx);

/*
 * Workspace. A context keeps five buffers: the int8 copy of X, the int8 copy of packed 4-bit
 * weights (qlinear_w4), per-row scratch (row scales of
 * qlinear_dtwq, row corrections of qlinear_asym, column statistics of gps_scales), calibration
 * histograms, and int32 partial sums for the calls that split K. Each is allocated on first use and
 * re-allocated (cudaFree + cudaMalloc, which synchronise the device) when a call needs more.
 *  - stwq_reserve sizes the first and third for an [M,K] activation and P positions;
 *    stwq_reserve_layer sizes all five for every call this header declares on an [M,K] x [N,K] layer
 *    with P positions. After either, calls within those sizes allocate nothing.
 *  - A call that would have to grow a buffer while its stream is being captured into a CUDA graph
 *    returns STWQ_ERR_CAPTURE and enqueues nothing (an allocation would invalidate the capture).
 *  - Growth moves the buffer: a graph captured earlier still holds the old, freed address and must
 *    not be replayed. stwq_workspace_generation() changes whenever any buffer was (re)allocated, so
 *    a caller that keeps graphs can compare the value it saw at capture time before each replay.
 * Both reserve calls are synchronous and may allocate.
 */
int stwq_reserve(stwq_ctx* ctx, int64_t M, int K, int P);
int stwq_reserve_layer(stwq_ctx* ctx, int64_t M, int K, int N, int P);
uint64_t stwq_workspace_generation(const stwq_ctx* ctx);

/*
 * Static token-wise calibration (Section 4.2: one set of quantization parameters per token
 * position, fixed offline by percentile calibration).
 * For each position p, over every row r with pos_ids[r] == p and every channel k:
 *     v = | Xcal[r,k] * (1 / s_ch[k]) |          (fp32; s_ch == NULL means no scaling)
 *     a_p = the value of rank ceil(pct_ppm * n_p / 1e6) among the n_p values, ascending
 *           (nearest rank, no interpolation; pct_ppm = 1000000 is min-max calibration)
 *     s_tok[p] = 2 a_p / D   (fp32 division; 1 if a_p == 0 or no row has position p;
 *                             floored at 2^-64)
 * Xcal [rows,K] fp32, pos_ids [rows] int32 in [0,P), s_tok [P] fp32 out.
 * pct_ppm in 1..1000000. Exact (an order statistic), independent of row order.
 */
int stwq_calibrate(stwq_ctx* ctx, const float* Xcal, const int32_t* pos_ids, int64_t rows, int K,
                   int P, const float* s_ch, int bits, uint32_t pct_ppm, float* s_tok,
                   void* stream);

/*
 * Gain-Projected Scaling (Section 4.1, Eq. 13-16; Algorithm 1 of Appendix F): the per-input-channel
 * scaling vector s of Eq. 2 from calibration activations and the layer's weights.
 *   1. Q(X) per tensor, its range the nearest-rank percentile pct_ppm of |Xcal| (as stwq_calibrate
 *      with one position), Q(W) per output channel with min-max range, both with the symmetric
 *      quantizer of `bits` bits; dX = X - Q(X), dW = W - Q(W).
 *   2. k* = the channel with the largest activation range max_t X[t,k] - min_t X[t,k] (lowest index
 *      on ties); s[k*] = sqrt(R_x[k*] / R_w[k*]), R_w[k*] the range of column k* of W.
 *   3. every other channel i:
 *        variant 0 (Eq. 16):   s[i] = s[k*] sqrt(sum_t sum_n |dW[n,i] X[t,i]|) / sqrt(sum_t sum_n |W[n,i] dX[t,i]|)
 *        variant 1 (the stationary point of the gain of Eq. 15):
 *                              s[i] = s[k*] (sum dW^2 X^2 / sum W^2 dX^2)^(1/4)
 *      A zero numerator, denominator or weight range gives 1; s is clamped to [1e-4, 1e4].
 * Xcal [rows,K] fp32, W [N,K] fp32, s_ch [K] fp32 out, k_star (device int32, may be NULL) receives k*.
 * Sums are accumulated in fp64 in a fixed order: repeatable, and within rounding of any other
 * order of summation. Uses context workspace (allocated on first use or growth).
 */
int gps_scales(stwq_ctx* ctx, const float* Xcal, int64_t rows, int K, const float* W, int N, int bits,
               uint32_t pct_ppm, int variant, float* s_ch, int32_t* k_star, void* stream);

/*
 * Distribution-Guided Calibration (Section 4.3, Eq. 17): the Mahalanobis distance of every sample of a
 * set to the set's own distribution, rho(x) = sqrt((x - u)^T S^-1 (x - u)) with u the mean and S the
 * (population) covariance of the set, and the choice of the ceil(keep_ppm n / 1e6) samples with the
 * largest rho (the paper keeps the top 50 %) as the calibration set. The paper does not say which
 * vector stands for a sample: F [n, D] fp32 holds one feature vector per sample, D <= 1024.
 * ridge >= 0: ridge * trace(S) / D is added to the diagonal of S before it is factorised (0 = Eq. 17 as
 * printed; a covariance that is then not positive definite, e.g. D >= n, gives rho = 0 for every
 * sample). rho [n] fp64 out; selected (int32, ceil(keep n) entries, may be NULL) receives the indices
 * of the kept samples, largest rho first, equal rho in index order. All in fp64 on the GPU.
 */
int dgc_select(stwq_ctx* ctx, const float* F, int n, int D, uint32_t keep_ppm, double ridge, double* rho,
               int32_t* selected, void* stream);

/*
 * Equivalent scaling, weight side (Eq. 2: Y = (X / s)(s * W)), then per-output-channel
 * min-max weight quantization with the symmetric form of Eq. 1:
 *     W'[n,k] = W[n,k] * s_ch[k]                  (s_ch == NULL: W' = W)
 *     a_n = max_k |W'[n,k]|,   s_w[n] = 2 a_n / D  (1 if a_n == 0)
 *     Wq[n,k] = clamp(round(W'[n,k] / s_w[n]), qmin, qmax)      (IEEE division, ties to even)
 * W [N,K] fp32 in, Wq [N,K] int8 out, s_w [N] fp32 out. bits in {8, 6, 4}: 4-bit weights (the W4A8
 * setting of Table 11) are codes in [-8, 7] in the same int8 containers, so every GEMM call takes them
 * unchanged together with 8-bit activations.
 */
int gps_fold(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, int bits, int8_t* Wq,
             float* s_w, void* stream);

/*
 * 4-bit weights stored two per byte (the W4A8 setting of Appendix J, Table 11: 4-bit weights, 8-bit
 * activations). The paper fixes the bit width, not a storage format; this one is the plain one:
 *     byte[n, j] = (Wq[n, 2j] & 0xF) | ((Wq[n, 2j+1] & 0xF) << 4)
 * i.e. two's complement nibbles, the even input channel in the low nibble, codes in [-8, 7], with
 * Wq and s_w exactly those of gps_fold(bits = 4). A weight matrix then takes N K / 2 bytes of HBM.
 *  - gps_fold_packed4: W [N,K] fp32 -> Wp [N, K/2] bytes, s_w [N]. K a multiple of 32.
 *  - stwq_unpack4: Wp -> Wq [N,K] int8 (for callers that want the containers back).
 *  - qlinear_w4: qlinear on packed weights: same arithmetic and results as qlinear on the unpacked
 *    codes (the activations keep `bits` in {8, 6}). The codes are widened to int8 on the GPU before
 *    the tensor cores read them; the widened copy lives in context workspace.
 */
int gps_fold_packed4(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, uint8_t* Wp, float* s_w,
                     void* stream);
int stwq_unpack4(stwq_ctx* ctx, const uint8_t* Wp, int N, int K, int8_t* Wq, void* stream);
int qlinear_w4(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, int N, const uint8_t* Wp,
               const float* s_w, const float* s_tok, int P, const float* s_ch, const float* bias, int bits, int act,
               int out_dtype, void* Y, void* stream);

/*
 * Activation quantization with static per-position scales (Eq. 1 on the left factor of
 * Eq. 2; Section 4.2):
 *     Xq[m,k] = clamp(round((X[m,k] * rc[k]) * rt[pos_ids[m]]), qmin, qmax)
 * rc[k] = 1 / s_ch[k] (1 if s_ch == NULL), rt[p] = 1 / s_tok[p], both IEEE fp32; the two
 * multiplies are rounded separately in this order; ties to even; NaN -> 0, +-Inf saturate.
 * X [M,K] fp32, pos_ids [M] int32, s_ch [K] or NULL, s_tok [P], Xq [M,K] int8 out.
 * A row whose pos_id is outside [0,P) is written as zeros and STWQ_ERR_POS_RANGE is recorded.
 */
int stwq_quantize(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K,
                  const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq, void* stream);

/* stwq_quantize for activations held in bf16 (X [M,K] bf16): every bf16 value is an fp32 value,
 * and the codes are those stwq_quantize gives on the widened input. */
int stwq_quantize_bf16(stwq_ctx* ctx, const void* X, const int32_t* pos_ids, int64_t M, int K,
                       const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq, void* stream);

/*
 * qlinear for activations held in bf16 (what a bf16 model hands from layer to layer): the same
 * quantizer on the widened values (Eq. 1, Section 4.2; see stwq_quantize_bf16), then the GEMM and
 * epilogue of qlinear. X [M,K] bf16, 16-byte aligned; everything else as qlinear. Reads 2 bytes per
 * activation instead of 4.
 */
int qlinear_bf16(stwq_ctx* ctx, const void* X, const int32_t* pos_ids, int64_t M, int K, int N,
                 const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* s_ch,
                 const float* bias, int bits, int act, int out_dtype, void* Y, void* stream);

/*
 * The quantized linear layer: stwq_quantize into context workspace, then
 *     acc[m,n] = sum_k Xq[m,k] * Wq[n,k]                          (int32, exact)
 *     z = float(acc) * (s_tok[pos_ids[m]] * s_w[n]) + bias[n]     (fp32: one multiply for the
 *                                                   scale, one fused multiply-add; Appendix A.1)
 *     Y[m,n] = act(z)  cast to out_dtype
 * bias == NULL means zero. out_dtype STWQ_OUT_INT32 stores acc itself.
 * Calls with few rows (M <= 256, the raster-order decode step where a batch advances one
 * token position at a time) are routed to a variant that streams Wq once across all SMs, split
 * along K where N alone does not give every SM work; the result is the same. That variant, and
 * the tiled GEMM when it splits a partly filled last wave along K, keep int32 partial sums in
 * context workspace that is allocated (synchronously) the first time a shape needs it.
 * The two kernels of a call are launched as programmatic dependents of their predecessor in the
 * stream; each waits for that predecessor to complete before its first dependent access, so the
 * effects are ordered as with ordinary launches.
 * Extra alignment: N a multiple of 8 for bf16 output gives vector stores; other N work but
 * store element by element.
 */
int qlinear(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, int N,
            const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* s_ch,
            const float* bias, int bits, int act, int out_dtype, void* Y, void* stream);

/* GEMM + epilogue of qlinear from codes the caller already holds (Xq [M,K] int8). */
int qlinear_q(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K, int N,
              const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* bias,
              int act, int out_dtype, void* Y, void* stream);

/*
 * Chained layers (Section 5 quantizes every linear of a block, so one quantized linear feeds
 * the next one's quantizer): qlinear whose epilogue applies the NEXT layer's static activation
 * quantizer instead of storing Y, so that the activation never makes the round trip through
 * memory in floating point:
 *     z = float(acc) * (s_tok[pos] * s_w[n]) + bias[n],  y = act(z)                 (fp32)
 *     Xq_next[m,n] = clamp(round((y * rc_next[n]) * rt_next[pos_ids[m]]), qmin, qmax)
 * rc_next = 1 / s_ch_next (1 if NULL), rt_next = 1 / s_tok_next, bits_next in {8, 6}; positions
 * are those of this layer (a linear keeps the token order). Xq_next [M,N] int8 is what
 * stwq_quantize would give on Y kept in fp32; feed it to qlinear_q / qlinear_chain_q of the next
 * layer. GELU is evaluated in the short form used for bf16 output (error on y below 6e-4 |z|),
 * so a code can differ by one from the exact activation's where u lies that close to a tie.
 * Always runs the tiled CTA-pair GEMM: N a multiple of 16, s_w / bias / s_ch_next 16-byte aligned
 * (STWQ_ERR_ALIGN otherwise).
 */
int qlinear_chain(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, int N,
                  const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* s_ch,
                  const float* bias, int bits, int act, const float* s_ch_next, const float* s_tok_next,
                  int bits_next, int8_t* Xq_next, void* stream);
int qlinear_chain_q(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K, int N,
                    const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* bias, int act,
                    const float* s_ch_next, const float* s_tok_next, int bits_next, int8_t* Xq_next, void* stream);

/*
 * The asymmetric quantizer, Eq. 1 as printed (Appendix B: channel-wise asymmetric weights,
 * asymmetric activations), next to the symmetric one that the calls above use:
 *     delta = (x_up - x_down) / D,  z = round(-x_down / delta),  c = clamp(round(x / delta) + z, 0, D)
 * with the range widened to contain 0 (so 0 <= z <= D). Codes live in the same signed containers,
 * cs = c - 2^(b-1), together with the signed zero point zs = z - 2^(b-1): x_hat = delta (cs - zs).
 *  - stwq_calibrate_asym: per position, x_up = the value of rank ceil(pct n) among the signed
 *    values X / s_ch, x_down = the value of rank n + 1 - ceil(pct n); s_tok[p] = delta, z_tok[p] = zs.
 *  - gps_fold_asym: per output channel the min-max range of W * s_ch; also colsum[n] = sum_k Wq[n,k].
 *  - stwq_quantize_asym: cs = clamp(round((X * rc) * rt) + z_tok[pos], qmin, qmax) and
 *    rowcorr[m] = sum_k cs[m,k] - K z_tok[pos[m]].
 *  - qlinear_asym: quantize, integer GEMM, then the exact zero-point correction
 *        acc' = acc - z_w[n] rowcorr[m] - z_tok[pos[m]] colsum[n]     (= sum_k (cs - zx)(ws - zw))
 *    and z = float(acc') * (s_tok[pos] * s_w[n]) + bias[n], activation, cast. STWQ_OUT_INT32 stores acc'.
 *    Runs the tiled CTA-pair GEMM for every M: N a multiple of 4 (8 for bf16), s_w / bias / z_w /
 *    colsum 16-byte aligned, K <= 32768 (STWQ_ERR_ALIGN / STWQ_ERR_DIM otherwise).
 */
int stwq_calibrate_asym(stwq_ctx* ctx, const float* Xcal, const int32_t* pos_ids, int64_t rows, int K, int P,
                        const float* s_ch, int bits, uint32_t pct_ppm, float* s_tok, int32_t* z_tok, void* stream);
int gps_fold_asym(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, int bits, int8_t* Wq, float* s_w,
                  int32_t* z_w, int32_t* colsum, void* stream);
int stwq_quantize_asym(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, const float* s_ch,
                       const float* s_tok, const int32_t* z_tok, int P, int bits, int8_t* Xq, int32_t* rowcorr,
                       void* stream);
int qlinear_asym(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, int N, const int8_t* Wq,
                 const float* s_w, const int32_t* z_w, const int32_t* colsum, const float* s_tok, const int32_t* z_tok,
                 int P, const float* s_ch, const float* bias, int bits, int act, int out_dtype, void* Y, void* stream);

/*
 * Dynamic token-wise quantization, the baseline that the static scales replace (Section 1,
 * Section 4.2, Table 5: the range of every token is found by a min-max pass at run time). Kept
 * to be timed beside stwq_quantize / qlinear, and for layers without calibrated scales:
 *     v = X[m,k] * rc[k],  a_m = max_k |v|,  s_row[m] = 2 a_m / D  (1 if a_m == 0),
 *     Xq[m,k] = clamp(round(v * (1 / s_row[m])), qmin, qmax)
 * NaN values do not take part in the maximum and give code 0. K <= 8192.
 * X [M,K] fp32, s_ch [K] or NULL, Xq [M,K] int8 out, s_row [M] fp32 out.
 * qlinear_dtwq is qlinear with this quantizer: the dequantizer uses s_row[m] in place of
 * s_tok[pos_ids[m]]; codes, scales and row ids live in context workspace.
 */
int dtwq_quantize(stwq_ctx* ctx, const float* X, int64_t M, int K, const float* s_ch, int bits, int8_t* Xq,
                  float* s_row, void* stream);
int qlinear_dtwq(stwq_ctx* ctx, const float* X, int64_t M, int K, int N, const int8_t* Wq, const float* s_w,
                 const float* s_ch, const float* bias, int bits, int act, int out_dtype, void* Y, void* stream);

/*
 * Quantized attention matmuls and the quantized KV cache (Section 5: "all linear layers and matrix
 * multiplications" run in 6 or 8 bits; Appendix C: "including the KV cache"). G = batch x heads
 * independent heads, head dimension d, Tq queries, Tk keys, token positions in [0, P).
 * Readings, since the paper names the operands but not their quantizers:
 *  - queries and keys: the static per-position quantizer of stwq_quantize without channel scales,
 *    codes = clamp(round(x * (1 / s[pos]))); in S = Q K^T the two scales leave the integer sum:
 *        S[i,j] = acc_qk[i,j] * (s_q[pos_q[i]] * s_kcol[j]),   s_kcol[j] = s_k[pos of key j] * softmax scale
 *  - values: one static scale per head channel, codes = clamp(round(x * (1 / s_v[c]))) (a scale that varied
 *    along the keys could not leave the sum over keys);
 *  - probabilities: Eq. 1 on the fixed range [0, 1]: delta_p = 1 / (2^b - 1), zero point 0, UNSIGNED codes
 *    0 .. 2^b - 1, P = softmax over the visible keys of row i (fp32); causal != 0 hides key j from query
 *    i unless j <= i + (Tk - Tq);
 *  - O[i,c] = acc_pv[i,c] * (delta_p * s_v[c]),  acc_pv = sum_j Pcode[i,j] Vq[j,c]   (unsigned x signed, int32).
 * Cache layout: Kc [G, Tmax, d] int8 (row = position), Vt [G, d, Tmax] int8 (the value codes transposed,
 * column = position), so that both matmuls read operands whose contraction index is contiguous.
 * d and Tmax multiples of 16, d <= 256.
 *  - kv_append: quantize t_new new key / value rows per head (Knew, Vnew [G, t_new, d] fp32, at positions
 *    pos0 .. pos0 + t_new - 1) into the caches. s_k [P], s_v [d]. Knew, Vnew, s_v, Kc and Vt
 *    16-byte aligned (STWQ_ERR_ALIGN otherwise).
 *  - qattention: Q [G, Tq, d] fp32, pos_q [Tq] (shared by all heads), keys / values = the first Tk
 *    positions of the caches, s_q [P], s_kcol [Tk], s_v [d]; O [G, Tq, d] fp32 or bf16. Quantizes Q, then
 *    one kernel per 128 queries of a head runs both matmuls on the tensor cores with the softmax and the
 *    quantizer of the probabilities in between, scores and probability codes staying on the SM (the keys
 *    are walked twice: row maxima and sums first, codes second). STWQ_OPT_VARIANT 9 runs the three stages
 *    as separate kernels instead (batched integer GEMMs with the scores, fp32, and the codes in context
 *    workspace). The two differ only where a probability sits on a rounding tie of its code. With at most
 *    eight queries (a decode step) one CTA per head and group of four queries reads the head's cache once and
 *    does the dot products by dp4a; same definitions, same tolerance.
 *    stwq_reserve_attention sizes the workspace ahead of time for the variant in force; growth during
 *    stream capture is refused like everywhere else.
 *  - qattn_softmax_quantize, qattn_pv: the second and third stage on their own (S [rows, ld] fp32 with
 *    rows = G Tq and ld >= Tk a multiple of 16; Pq [G, Tq, Tk_pad] codes; STWQ_OUT_INT32 stores acc_pv).
 */
int kv_append(stwq_ctx* ctx, const float* Knew, const float* Vnew, int G, int t_new, int d, int pos0, int Tmax,
              const float* s_k, const float* s_v, int P, int bits, int8_t* Kc, int8_t* Vt, void* stream);
int qattention(stwq_ctx* ctx, const float* Q, const int32_t* pos_q, int G, int Tq, int Tk, int d, int Tmax,
               const int8_t* Kc, const int8_t* Vt, const float* s_q, const float* s_kcol, const float* s_v, int P,
               int bits, int causal, int out_dtype, void* O, void* stream);
int stwq_reserve_attention(stwq_ctx* ctx, int G, int Tq, int Tk, int d);
int qattn_softmax_quantize(stwq_ctx* ctx, const float* S, int64_t rows, int Tq, int Tk, int ld, int causal, int bits,
                           uint8_t* Pq, void* stream);
int qattn_pv(stwq_ctx* ctx, const uint8_t* Pq, int G, int Tq, int Tk_pad, int d, int Tmax, const int8_t* Vt,
             const float* s_v, const float* delta_p, int out_dtype, void* O, void* stream);

/*
 * qlinear without any allocation. (The paper has no counterpart to this call; it exists for the
 * way the library gets embedded.) qlinear needs a context, whose creation allocates, and keeps
 * the int8 copy of X in workspace that may be (re)allocated during a call. Hosts that cannot
 * reach an allocator at that point - a loop with a hard latency budget, a process whose device
 * memory is wholly owned by another runtime's pool, a deployment that forbids allocation after
 * start-up - call this instead. It takes no context, runs on the CURRENT device, and computes
 * exactly what qlinear computes (tiled tensor-core GEMM for every M), with the int8 copy of X
 * held in a fixed array of STWQ_STATIC_MAX_CODES bytes that is part of the library image on
 * every GPU that loads it (4 MiB + 256 bytes per GPU until the process exits).
 *  - M * K must not exceed STWQ_STATIC_MAX_CODES; larger problems return STWQ_ERR_DIM and
 *    nothing is enqueued. All other argument rules are those of qlinear.
 *  - The first call on each device looks up the array's device address and the driver entry
 *    point for tensor maps (no allocation, but several runtime queries): make that call once
 *    during start-up, before any stream capture begins on that device.
 *  - All calls on a device share the one array, which keeps the codes of the last call. Two
 *    calls whose kernels can overlap on the GPU (different streams without an ordering between
 *    them) race on it; order them. Nothing in it needs clearing between calls: each call
 *    overwrites the M * K bytes it later reads.
 *  - Device-side conditions (a pos_id outside [0,P) - that row is computed as zeros - or an
 *    expired device wait) are not reported by this call.
 */
#define STWQ_STATIC_MAX_CODES (4 * 1024 * 1024)
int qlinear_static(const float* X, const int32_t* pos_ids, int64_t M, int K, int N, const int8_t* Wq,
                   const float* s_w, const float* s_tok, int P, const float* s_ch, const float* bias,
                   int bits, int act, int out_dtype, void* Y, void* stream);

/*
 * Synchronise `stream`, then return and clear the status recorded by device code since the
 * last call: STWQ_OK, STWQ_ERR_POS_RANGE, STWQ_ERR_NONFINITE or STWQ_ERR_DEVICE_TIMEOUT.
 */
int stwq_device_status(stwq_ctx* ctx, void* stream);

/*
 * Self-test of the bounded device-side wait (the paper has no counterpart; failure handling of the
 * library). Launches one small CTA that waits, with the wait routine and the limit
 * (STWQ_OPT_WAIT_LIMIT_MS, at most one second here) of the GEMM kernels, for a barrier that nothing
 * completes. The wait gives up, the kernel records the timeout in the context's status word and
 * returns; stwq_device_status() then reports STWQ_ERR_DEVICE_TIMEOUT once. waited_ns (device pointer
 * to one uint64, may be NULL) receives the time the wait lasted. The context stays usable.
 */
int stwq_selftest_wait_expiry(stwq_ctx* ctx, uint64_t* waited_ns, void* stream);

/*
 * Options (for tests and tuning). STWQ_OPT_GEMM_PATH: 0 = choose by shape (default),
 * 1 = always a tiled tensor-core GEMM, 2 = always the few-row (decode) variant (M <= 256 only),
 * 3 = always the single-CTA tiled GEMM (the fallback used when N or the s_w / bias pointers
 * do not meet the 16-byte rules of the CTA-pair kernel).
 * STWQ_OPT_WAIT_LIMIT_MS: limit of every device-side wait in milliseconds (default 2000).
 * The remaining options choose between kernel variants that compute the same results (the parity
 * tests use them to reach every variant; 0 = the library's own choice; any other value than those
 * listed is refused with STWQ_ERR_DIM):
 * STWQ_OPT_TILE_N: 128 or 256 = tile width of the CTA-pair GEMM.
 * STWQ_OPT_VARIANT: 1 / 2 = CTA-pair GEMM epilogue through staged TMA stores / straight from
 *   registers; 5 = ordinary launches instead of programmatic dependent ones; 7 / 8 = the
 *   register-streaming / the TMA-ring quantize kernel; 9 = qattention as three separate stages (batched
 *   GEMM, softmax-and-quantize pass, batched GEMM) instead of the one-kernel head.
 * STWQ_OPT_KSPLIT (-1 .. 64): n > 0 = cut the tiles of the last wave of the CTA-pair GEMM (every work item of
 *   the few-row kernel) into n ranges of K; -1 = the few-row kernel never cuts. The CTA-pair GEMM
 *   cuts only on request.
 */
enum { STWQ_OPT_GEMM_PATH = 1, STWQ_OPT_WAIT_LIMIT_MS = 2, STWQ_OPT_TILE_N = 100, STWQ_OPT_VARIANT = 101,
       STWQ_OPT_KSPLIT = 102 };
int stwq_set_option(stwq_ctx* ctx, int option, int value);

/*
 * Peak probe of the int8 tensor path (measurement aid; the paper has no counterpart). Launches one
 * kernel in which `cta_pairs` CTA pairs (0 = as many as are resident at once, one pair per two SMs)
 * each issue kblocks x 4 tcgen05.mma.cta_group::2.kind::i8 instructions (M 256, N 256, K 32) on operand
 * tiles that stay in shared memory: no global traffic, no epilogue. *ops_per_launch (HOST pointer, may
 * be NULL) receives pairs * kblocks * 4 * 2 * 256 * 256 * 32. The caller times the launch with events;
 * ops / time is the rate the pipe delivers at the clocks the GPU holds. kblocks in 1 .. 2^22.
 */
int stwq_probe_int8_peak(stwq_ctx* ctx, int kblocks, int cta_pairs, int64_t* ops_per_launch, void* stream);

/* Number of kernels this context has launched since creation (for launch accounting). */
int64_t stwq_launch_count(const stwq_ctx* ctx);

/* Text for a status code; the cudaError_t of the last STWQ_ERR_CUDA on this context. */
const char* stwq_strerror(int status);
int stwq_last_cuda_error(const stwq_ctx* ctx);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* STWQ_H */

/*
 * CPU oracle for the static-token-wise-quantized (STWQ) linear layer of PTQ4ARVG.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain definition of what the
 * GPU library must compute. It shares no code with the CUDA path and is never on
 * the product path: only the tests, the smoke check and the benchmark's CPU
 * baseline leg may load it.
 *
 * Every function names the passage of the paper it follows. Where the paper is
 * silent the reading taken is stated next to the code. Parity status: every
 * function here is pinned by the CPU tests (closed forms, brute force, textbook
 * special cases); none is "parity unpinned".
 *
 * Layout conventions: X is [rows, K] row-major (K = the paper's n input
 * channels), W is [N, K] row-major (the transpose of the paper's n x m W, N =
 * the paper's m output channels), Y is [rows, N] row-major.
 *
 * Arithmetic: fp32 where a decision (a code, a scale) is taken, because the
 * deployed path takes it in fp32; fp64 for the dequantized output. Build with
 * -O2 -ffp-contract=off and without fast-math so every fp32 operation below is
 * one IEEE-754 operation in the order written.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------- */
/* Code range of a b-bit signed container.                                    */
static int orc_qmax(int bits) { return (1 << (bits - 1)) - 1; }
static int orc_qmin(int bits) { return -(1 << (bits - 1)); }

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/*
 * Eq. 1, general (asymmetric) form, exactly as printed:
 *   delta = (x_up - x_down) / (2^b - 1),  z = round(-x_down / delta),
 *   code  = clamp(round(x / delta) + z, 0, 2^b - 1),
 * and the dequantizer of Appendix A.1:  x_hat = delta * (code - z).
 * round() is round-to-nearest; ties go to even (the paper does not fix the tie
 * rule; this is the IEEE default and what hardware converts do).
 * Outputs: codes in [0, 2^b-1] as int32, and (optionally) delta and z.
 */
void orc_eq1_quantize(const float* x, int64_t n, float x_down, float x_up, int bits,
                      int32_t* code, float* delta_out, int32_t* z_out)
{
    const float levels = (float)((1 << bits) - 1);
    float delta = (x_up - x_down) / levels;
    if (!(delta > 0.0f)) delta = 1.0f;
    const int32_t z = (int32_t)nearbyintf(-x_down / delta);
    for (int64_t i = 0; i < n; ++i) {
        float r = nearbyintf(x[i] / delta) + (float)z;
        if (r < 0.0f) r = 0.0f;
        if (r > levels) r = levels;
        code[i] = (int32_t)r;
    }
    if (delta_out) *delta_out = delta;
    if (z_out) *z_out = z;
}

void orc_eq1_dequantize(const int32_t* code, int64_t n, float delta, int32_t z, float* x_hat)
{
    for (int64_t i = 0; i < n; ++i) x_hat[i] = delta * (float)(code[i] - z);
}

/* ------------------------------------------------------------------------- */
/*
 * Symmetric specialisation of Eq. 1 used by the deployed path: the range is
 * [-a, a], so R = 2a and delta = 2a / (2^b - 1). The zero point of Eq. 1 is then
 * round((2^b - 1) / 2) = 2^(b-1); subtracting it from the unsigned code gives a
 * signed code in [-2^(b-1), 2^(b-1) - 1], i.e. [-128,127] for b = 8 and
 * [-32,31] for b = 6, and the dequantizer becomes x_hat = delta * code.
 * Guards (the paper gives none): a == 0 gives delta = 1; delta is floored at
 * 2^-64 so that its reciprocal is finite.
 */
float orc_delta(float a, int bits)
{
    const float levels = (float)((1 << bits) - 1);
    if (!(a > 0.0f)) return 1.0f;
    float delta = (a + a) / levels;
    const float floor_ = 5.421010862427522e-20f; /* 2^-64 */
    if (delta < floor_) delta = floor_;
    return delta;
}

/* round-to-nearest-even then clamp to the signed b-bit range; NaN gives 0. */
static int32_t orc_code(float u, int bits)
{
    if (u != u) return 0;
    float r = nearbyintf(u);
    const float lo = (float)orc_qmin(bits), hi = (float)orc_qmax(bits);
    if (r < lo) r = lo;
    if (r > hi) r = hi;
    return (int32_t)r;
}

/* q(x) = clamp(round(x / delta)) with a true division (Eq. 1), signed codes. */
void orc_quantize_div(const float* x, int64_t n, float delta, int bits, int8_t* q)
{
    for (int64_t i = 0; i < n; ++i) q[i] = (int8_t)orc_code(x[i] / delta, bits);
}

/* ------------------------------------------------------------------------- */
/*
 * Equivalent scaling, weight side (Eq. 2: Y = (X / s)(s * W)) followed by
 * per-output-channel weight quantization (Appendix B: channel-wise weights) with
 * min-max range calibration (Section 3), in the symmetric form above:
 *   W'[n,k] = W[n,k] * s_ch[k]        (s_ch == NULL means all ones)
 *   a_n     = max_k |W'[n,k]|
 *   s_w[n]  = delta(a_n)
 *   Wq[n,k] = clamp(round(W'[n,k] / s_w[n]))     (true division)
 */
void orc_gps_fold(const float* W, int N, int K, const float* s_ch, int bits,
                  int8_t* Wq, float* s_w)
{
    for (int n = 0; n < N; ++n) {
        const float* w = W + (int64_t)n * K;
        float a = 0.0f;
        for (int k = 0; k < K; ++k) {
            float v = s_ch ? w[k] * s_ch[k] : w[k];
            float av = fabsf(v);
            if (av > a) a = av;
        }
        const float d = orc_delta(a, bits);
        s_w[n] = d;
        for (int k = 0; k < K; ++k) {
            float v = s_ch ? w[k] * s_ch[k] : w[k];
            Wq[(int64_t)n * K + k] = (int8_t)orc_code(v / d, bits);
        }
    }
}

/* ------------------------------------------------------------------------- */
/*
 * STWQ calibration (Section 4.2): one static quantization range per token
 * position, set offline by percentile calibration over the calibration samples.
 * For position p the population is |X[r,k] * rc[k]| over every calibration row r
 * with pos_ids[r] == p and every channel k, where rc[k] = 1 / s_ch[k] is the
 * activation side of Eq. 2 (s_ch == NULL: no scaling). The range half-width a_p
 * is the nearest-rank percentile: with n_p values sorted ascending, the value of
 * rank ceil(pct * n_p) (1-based), pct given in parts per million; no
 * interpolation. pct = 100 % is min-max calibration. s_tok[p] = delta(a_p).
 * A position with no rows gets s_tok = 1.
 * Returns 0, or -1 if a pos_id is outside [0, P), -2 on a non-finite value.
 */
static int orc_cmp_float(const void* a, const void* b)
{
    const float fa = *(const float*)a, fb = *(const float*)b;
    return (fa > fb) - (fa < fb);
}

int orc_stwq_calibrate(const float* X, const int32_t* pos_ids, int64_t rows, int K, int P,
                       const float* s_ch, int bits, uint32_t pct_ppm, float* s_tok)
{
    int64_t* count = (int64_t*)calloc((size_t)P, sizeof(int64_t));
    for (int64_t r = 0; r < rows; ++r) {
        if (pos_ids[r] < 0 || pos_ids[r] >= P) { free(count); return -1; }
        count[pos_ids[r]] += 1;
    }
    float* rc = (float*)malloc(sizeof(float) * (size_t)K);
    for (int k = 0; k < K; ++k) rc[k] = s_ch ? 1.0f / s_ch[k] : 1.0f;

    int status = 0;
    for (int p = 0; p < P; ++p) {
        const int64_t n_p = count[p] * (int64_t)K;
        if (n_p == 0) { s_tok[p] = 1.0f; continue; }
        float* v = (float*)malloc(sizeof(float) * (size_t)n_p);
        int64_t j = 0;
        for (int64_t r = 0; r < rows; ++r) {
            if (pos_ids[r] != p) continue;
            for (int k = 0; k < K; ++k) {
                const float x = X[r * K + k];
                const float t = s_ch ? x * rc[k] : x;
                if (!isfinite(t)) status = -2;
                v[j++] = fabsf(t);
            }
        }
        qsort(v, (size_t)n_p, sizeof(float), orc_cmp_float);
        uint64_t rank = ((uint64_t)pct_ppm * (uint64_t)n_p + 999999ull) / 1000000ull;
        if (rank < 1) rank = 1;
        if (rank > (uint64_t)n_p) rank = (uint64_t)n_p;
        s_tok[p] = orc_delta(v[rank - 1], bits);
        free(v);
    }
    free(rc);
    free(count);
    return status;
}

/* ------------------------------------------------------------------------- */
/*
 * Step 1 of the quantized linear: activation quantization with the static
 * per-position scale (Eq. 1 applied to the left factor of Eq. 2, Section 4.2).
 *   Xq[m,k] = clamp(round( (X[m,k] * rc[k]) * rt[pos[m]] ))
 * with rc[k] = 1/s_ch[k] and rt[p] = 1/s_tok[p] formed once in fp32. The
 * deployed path multiplies by reciprocals instead of dividing twice per element;
 * the product is taken in this order, each multiply rounded to fp32.
 * NaN gives code 0; +-Inf saturate.
 * Returns 0, or -1 if a pos_id is outside [0, P).
 */
int orc_quantize(const float* X, const int32_t* pos_ids, int64_t M, int K,
                 const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq)
{
    float* rc = (float*)malloc(sizeof(float) * (size_t)K);
    for (int k = 0; k < K; ++k) rc[k] = s_ch ? 1.0f / s_ch[k] : 1.0f;
    int status = 0;
    for (int64_t m = 0; m < M; ++m) {
        const int32_t p = pos_ids[m];
        if (p < 0 || p >= P) { status = -1; break; }
        const float rt = 1.0f / s_tok[p];
        for (int k = 0; k < K; ++k) {
            const float x = X[m * K + k];
            const float t = s_ch ? x * rc[k] : x;
            const float u = t * rt;
            Xq[m * K + k] = (int8_t)orc_code(u, bits);
        }
    }
    free(rc);
    return status;
}

/*
 * Dynamic token-wise quantization, the baseline that the static scheme replaces
 * (Section 1 and Section 4.2: the quantization range of every token is found at
 * run time by a min-max pass over that token; Table 5 prices it at 473.9 ms
 * against 397.9 ms for the static scales). Per row m:
 *   v[k]  = X[m,k] * rc[k]                       (rc = 1 / s_ch, or 1)
 *   a_m   = max_k |v[k]|                         (NaN entries do not take part)
 *   s_m   = delta(a_m) = 2 a_m / (2^b - 1)       (the symmetric quantizer above)
 *   Xq    = clamp(round(v[k] * (1 / s_m)))       (reciprocal form, as on the static path)
 * s_row[m] = s_m is returned so that the dequantizer can use it in place of the
 * static s_tok[pos[m]].
 */
void orc_dtwq_quantize(const float* X, int64_t M, int K, const float* s_ch, int bits, int8_t* Xq,
                       float* s_row)
{
    float* rc = (float*)malloc(sizeof(float) * (size_t)K);
    for (int k = 0; k < K; ++k) rc[k] = s_ch ? 1.0f / s_ch[k] : 1.0f;
    for (int64_t m = 0; m < M; ++m) {
        float a = 0.0f;
        for (int k = 0; k < K; ++k) {
            const float x = X[m * K + k];
            const float v = s_ch ? x * rc[k] : x;
            const float av = fabsf(v);
            if (av > a) a = av;                       /* false for NaN */
        }
        const float s = orc_delta(a, bits);
        const float rt = 1.0f / s;
        s_row[m] = s;
        for (int k = 0; k < K; ++k) {
            const float x = X[m * K + k];
            const float v = s_ch ? x * rc[k] : x;
            Xq[m * K + k] = (int8_t)orc_code(v * rt, bits);
        }
    }
    free(rc);
}

/*
 * The same step with two true divisions per element, (x / s_ch[k]) / s_tok[p]:
 * the literal reading of Eq. 1 and Eq. 2. Information only (how many codes the
 * reciprocal form moves); not the parity definition.
 */
int orc_quantize_exact_div(const float* X, const int32_t* pos_ids, int64_t M, int K,
                           const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq)
{
    for (int64_t m = 0; m < M; ++m) {
        const int32_t p = pos_ids[m];
        if (p < 0 || p >= P) return -1;
        for (int k = 0; k < K; ++k) {
            const double x = X[m * K + k];
            const double t = s_ch ? x / (double)s_ch[k] : x;
            const float u = (float)(t / (double)s_tok[p]);
            Xq[m * K + k] = (int8_t)orc_code(u, bits);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/*
 * Step 2: Y = X W of Section 3 on the integer codes, int32 accumulation:
 *   acc[m,n] = sum_k Xq[m,k] * Wq[n,k].
 * |acc| <= K * 2^14, so int32 cannot overflow for K < 131072.
 */
void orc_igemm(const int8_t* Xq, const int8_t* Wq, int64_t M, int N, int K, int32_t* acc)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        const int8_t* x = Xq + m * K;
        for (int n = 0; n < N; ++n) {
            const int8_t* w = Wq + (int64_t)n * K;
            int32_t s = 0;
            for (int k = 0; k < K; ++k) s += (int32_t)x[k] * (int32_t)w[k];
            acc[m * N + n] = s;
        }
    }
}

/* ------------------------------------------------------------------------- */
/*
 * Step 3: dequantization (Appendix A.1, x_hat = delta * code, applied to the
 * product of two quantized factors), bias, optional GELU; in double.
 *   z = acc * (s_tok[pos[m]] * s_w[n]) + bias[n]
 *   act 0: y = z
 *   act 1: y = z * 0.5 * (1 + erf(z / sqrt 2))                    (GELU, erf form)
 *   act 2: y = z * 0.5 * (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3))) (GELU, tanh form)
 * mag (optional) receives |acc * s_tok * s_w| + |bias|, the magnitude the
 * tolerance of the parity tests is relative to.
 */
int orc_epilogue(const int32_t* acc, const int32_t* pos_ids, int64_t M, int N,
                 const float* s_tok, int P, const float* s_w, const float* bias, int act,
                 double* Y, double* mag)
{
    for (int64_t m = 0; m < M; ++m) {
        const int32_t p = pos_ids[m];
        if (p < 0 || p >= P) return -1;
        const double st = (double)s_tok[p];
        for (int n = 0; n < N; ++n) {
            const double prod = (double)acc[m * N + n] * (st * (double)s_w[n]);
            const double b = bias ? (double)bias[n] : 0.0;
            const double z = prod + b;
            double y = z;
            if (act == 1) y = z * 0.5 * (1.0 + erf(z / sqrt(2.0)));
            else if (act == 2)
                y = z * 0.5 * (1.0 + tanh(sqrt(2.0 / M_PI) * (z + 0.044715 * z * z * z)));
            Y[m * N + n] = y;
            if (mag) mag[m * N + n] = fabs(prod) + fabs(b);
        }
    }
    return 0;
}

/*
 * Chained layers: the paper quantizes every linear of a block (Section 5), so the
 * output of one quantized linear is the input of the next one's static
 * quantizer. This is Step 3 followed at once by Step 1 of the next layer:
 *   z = fmaf(float(acc), s_tok[pos] * s_w[n], bias[n])        in fp32, this order
 *   y = act(z)         (the activation itself evaluated in double, rounded to fp32)
 *   u = (y * rc_next[n]) * rt_next[pos]                       two fp32 multiplies
 *   code = clamp(round(u))
 * A code is an integer decided by floating point, so the decision is taken in the
 * precision of the deployed path (fp32), not in double. u_out (optional) receives
 * u and zmag_out (optional) |z * rc_next * rt_next|, which bounds how far an
 * approximate activation can move u.
 */
int orc_chain_codes(const int32_t* acc, const int32_t* pos_ids, int64_t M, int N,
                    const float* s_tok, int P, const float* s_w, const float* bias, int act,
                    const float* s_ch_next, const float* s_tok_next, int bits_next,
                    int8_t* codes, float* u_out, float* zmag_out)
{
    for (int64_t m = 0; m < M; ++m) {
        const int32_t p = pos_ids[m];
        if (p < 0 || p >= P) return -1;
        const float st = s_tok[p];
        const float rt = 1.0f / s_tok_next[p];
        for (int n = 0; n < N; ++n) {
            const float scale = st * s_w[n];
            const float z = fmaf((float)acc[m * N + n], scale, bias ? bias[n] : 0.0f);
            float y = z;
            const double zd = (double)z;
            if (act == 1) y = (float)(zd * 0.5 * (1.0 + erf(zd / sqrt(2.0))));
            else if (act == 2)
                y = (float)(zd * 0.5 * (1.0 + tanh(sqrt(2.0 / M_PI) * (zd + 0.044715 * zd * zd * zd))));
            const float rc = s_ch_next ? 1.0f / s_ch_next[n] : 1.0f;
            const float t = y * rc;
            const float u = t * rt;
            codes[m * N + n] = (int8_t)orc_code(u, bits_next);
            if (u_out) u_out[m * N + n] = u;
            if (zmag_out) zmag_out[m * N + n] = fabsf((z * rc) * rt);
        }
    }
    return 0;
}

/*
 * The whole quantized linear: quantize -> integer GEMM -> dequantize.
 * Xq_out, acc_out and mag may be NULL. Returns 0 or -1 (bad pos_id).
 */
int orc_qlinear(const float* X, const int32_t* pos_ids, int64_t M, int K, int N,
                const int8_t* Wq, const float* s_w, const float* s_tok, int P,
                const float* s_ch, const float* bias, int bits, int act,
                double* Y, int8_t* Xq_out, int32_t* acc_out, double* mag)
{
    int8_t* Xq = Xq_out ? Xq_out : (int8_t*)malloc((size_t)(M * K));
    int32_t* acc = acc_out ? acc_out : (int32_t*)malloc(sizeof(int32_t) * (size_t)(M * N));
    int st = orc_quantize(X, pos_ids, M, K, s_ch, s_tok, P, bits, Xq);
    if (st == 0) {
        orc_igemm(Xq, Wq, M, N, K, acc);
        st = orc_epilogue(acc, pos_ids, M, N, s_tok, P, s_w, bias, act, Y, mag);
    }
    if (!Xq_out) free(Xq);
    if (!acc_out) free(acc);
    return st;
}

/* ------------------------------------------------------------------------- */
/*
 * The asymmetric quantizer, Eq. 1 as printed (Appendix B deploys "channel-wise
 * asymmetric" weights and asymmetric activations), in the form the integer
 * pipeline needs.
 *   delta = (x_up - x_down) / (2^b - 1),  z = round(-x_down / delta),
 *   c = clamp(round(x / delta) + z, 0, 2^b - 1),  x_hat = delta (c - z).
 * Readings: the range is widened to contain 0 (x_down <= 0 <= x_up), which keeps
 * z inside [0, 2^b - 1] and zero exactly representable; a degenerate range gives
 * delta = 1; delta is floored at 2^-64. Codes are stored in signed containers by
 * subtracting h = 2^(b-1): cs = c - h in [-h, h-1], with the signed zero point
 * zs = z - h, so that x_hat = delta (cs - zs). orc_asym_params gives (delta, zs).
 */
void orc_asym_params(float x_down, float x_up, int bits, float* delta_out, int32_t* zs_out)
{
    const float levels = (float)((1 << bits) - 1);
    if (x_down > 0.0f) x_down = 0.0f;
    if (x_up < 0.0f) x_up = 0.0f;
    float delta = (x_up - x_down) / levels;
    if (!(delta > 0.0f)) delta = 1.0f;
    const float floor_ = 5.421010862427522e-20f;
    if (delta < floor_) delta = floor_;
    float z = nearbyintf(-x_down / delta);
    if (z < 0.0f) z = 0.0f;
    if (z > levels) z = levels;
    *delta_out = delta;
    *zs_out = (int32_t)z - (1 << (bits - 1));
}

/* cs = clamp(round(u) + zs, -h, h-1); NaN gives round(u) = 0; huge u saturates first. */
static int32_t orc_code_asym(float u, int32_t zs, int bits)
{
    float r = (u != u) ? 0.0f : nearbyintf(u);
    if (r > 1048576.0f) r = 1048576.0f;
    if (r < -1048576.0f) r = -1048576.0f;
    int32_t c = (int32_t)r + zs;
    if (c < orc_qmin(bits)) c = orc_qmin(bits);
    if (c > orc_qmax(bits)) c = orc_qmax(bits);
    return c;
}

/*
 * Weights, asymmetric per output channel (Eq. 2 weight side, then Eq. 1 with the
 * min-max range of the scaled row): Wq signed codes, s_w = delta_n, z_w = zs_n,
 * and colsum[n] = sum_k Wq[n,k], which the zero-point correction of the
 * integer product needs.
 */
void orc_gps_fold_asym(const float* W, int N, int K, const float* s_ch, int bits,
                       int8_t* Wq, float* s_w, int32_t* z_w, int32_t* colsum)
{
    for (int n = 0; n < N; ++n) {
        const float* w = W + (int64_t)n * K;
        float lo = 0.0f, hi = 0.0f;
        for (int k = 0; k < K; ++k) {
            const float v = s_ch ? w[k] * s_ch[k] : w[k];
            if (v < lo) lo = v;
            if (v > hi) hi = v;
        }
        float d; int32_t zs;
        orc_asym_params(lo, hi, bits, &d, &zs);
        s_w[n] = d;
        z_w[n] = zs;
        int32_t sum = 0;
        for (int k = 0; k < K; ++k) {
            const float v = s_ch ? w[k] * s_ch[k] : w[k];
            const int32_t c = orc_code_asym(v / d, zs, bits);
            Wq[(int64_t)n * K + k] = (int8_t)c;
            sum += c;
        }
        colsum[n] = sum;
    }
}

/*
 * Static token-wise calibration, asymmetric: per position the range is
 * [x_down, x_up] with x_up the nearest-rank percentile of the signed values
 * (rank r = ceil(pct n), ascending) and x_down the mirrored one (rank n + 1 - r);
 * pct = 100 % is min-max. s_tok[p] = delta_p, z_tok[p] = zs_p. A position with
 * no rows gets (1, -h + 0) from the degenerate range [0, 0].
 */
int orc_stwq_calibrate_asym(const float* X, const int32_t* pos_ids, int64_t rows, int K, int P,
                            const float* s_ch, int bits, uint32_t pct_ppm, float* s_tok, int32_t* z_tok)
{
    int64_t* count = (int64_t*)calloc((size_t)P, sizeof(int64_t));
    for (int64_t r = 0; r < rows; ++r) {
        if (pos_ids[r] < 0 || pos_ids[r] >= P) { free(count); return -1; }
        count[pos_ids[r]] += 1;
    }
    float* rc = (float*)malloc(sizeof(float) * (size_t)K);
    for (int k = 0; k < K; ++k) rc[k] = s_ch ? 1.0f / s_ch[k] : 1.0f;
    int status = 0;
    for (int p = 0; p < P; ++p) {
        const int64_t n_p = count[p] * (int64_t)K;
        if (n_p == 0) { orc_asym_params(0.0f, 0.0f, bits, &s_tok[p], &z_tok[p]); continue; }
        float* v = (float*)malloc(sizeof(float) * (size_t)n_p);
        int64_t j = 0;
        for (int64_t r = 0; r < rows; ++r) {
            if (pos_ids[r] != p) continue;
            for (int k = 0; k < K; ++k) {
                const float x = X[r * K + k];
                const float t = s_ch ? x * rc[k] : x;
                if (!isfinite(t)) status = -2;
                v[j++] = t;
            }
        }
        qsort(v, (size_t)n_p, sizeof(float), orc_cmp_float);
        uint64_t rank = ((uint64_t)pct_ppm * (uint64_t)n_p + 999999ull) / 1000000ull;
        if (rank < 1) rank = 1;
        if (rank > (uint64_t)n_p) rank = (uint64_t)n_p;
        orc_asym_params(v[(uint64_t)n_p - rank], v[rank - 1], bits, &s_tok[p], &z_tok[p]);
        free(v);
    }
    free(rc);
    free(count);
    return status;
}

/*
 * Activation quantization, asymmetric static per position, reciprocal form as on
 * the symmetric path: u = (X * rc) * rt, cs = clamp(round(u) + zs[pos], -h, h-1).
 * rowcorr[m] = sum_k cs[m,k] - K zs[pos[m]] is returned for the correction below.
 */
int orc_quantize_asym(const float* X, const int32_t* pos_ids, int64_t M, int K, const float* s_ch,
                      const float* s_tok, const int32_t* z_tok, int P, int bits, int8_t* Xq, int32_t* rowcorr)
{
    float* rc = (float*)malloc(sizeof(float) * (size_t)K);
    for (int k = 0; k < K; ++k) rc[k] = s_ch ? 1.0f / s_ch[k] : 1.0f;
    int status = 0;
    for (int64_t m = 0; m < M; ++m) {
        const int32_t p = pos_ids[m];
        if (p < 0 || p >= P) { status = -1; break; }
        const float rt = 1.0f / s_tok[p];
        int32_t sum = 0;
        for (int k = 0; k < K; ++k) {
            const float x = X[m * K + k];
            const float t = s_ch ? x * rc[k] : x;
            const int32_t c = orc_code_asym(t * rt, z_tok[p], bits);
            Xq[m * K + k] = (int8_t)c;
            sum += c;
        }
        rowcorr[m] = sum - K * z_tok[p];
    }
    free(rc);
    return status;
}

/*
 * The integer product of two asymmetric factors. With x_hat = dx (cs - zx) and
 * w_hat = dw (ws - zw):
 *   sum_k x_hat w_hat = dx dw [ acc - zw (sum_k cs - K zx) - zx sum_k ws ]
 *                     = dx dw [ acc - zw[n] rowcorr[m] - zx[pos[m]] colsum[n] ]
 * acc_corr (optional) receives the bracket (an exact integer); then bias and
 * activation as in orc_epilogue, in double.
 */
int orc_epilogue_asym(const int32_t* acc, const int32_t* pos_ids, int64_t M, int N, const float* s_tok,
                      const int32_t* z_tok, int P, const float* s_w, const int32_t* z_w, const int32_t* colsum,
                      const int32_t* rowcorr, const float* bias, int act, double* Y, double* mag,
                      int32_t* acc_corr)
{
    for (int64_t m = 0; m < M; ++m) {
        const int32_t p = pos_ids[m];
        if (p < 0 || p >= P) return -1;
        const double st = (double)s_tok[p];
        for (int n = 0; n < N; ++n) {
            const int64_t a = (int64_t)acc[m * N + n] - (int64_t)z_w[n] * rowcorr[m] - (int64_t)z_tok[p] * colsum[n];
            if (acc_corr) acc_corr[m * N + n] = (int32_t)a;
            const double prod = (double)a * (st * (double)s_w[n]);
            const double b = bias ? (double)bias[n] : 0.0;
            const double z = prod + b;
            double y = z;
            if (act == 1) y = z * 0.5 * (1.0 + erf(z / sqrt(2.0)));
            else if (act == 2)
                y = z * 0.5 * (1.0 + tanh(sqrt(2.0 / M_PI) * (z + 0.044715 * z * z * z)));
            Y[m * N + n] = y;
            if (mag) mag[m * N + n] = fabs(prod) + fabs(b);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/*
 * Gain-Projected Scaling, Algorithm 1 (Appendix F), with Eq. 13-16 of Section 4.1.
 * Inputs: calibration activations X [T, K], weights W [N, K] (paper: n x m,
 * transposed here), bit width, percentile for the activation range.
 *
 * 1. Quantize X per tensor (Step 3 of Section 4.1 assumes per-tensor activation
 *    quantization; range by percentile calibration) and W per output channel
 *    (min-max), both with the symmetric quantizer above; dX = X - Q(X),
 *    dW = W - Q(W).
 * 2. R_x[k] = max_t X[t,k] - min_t X[t,k]; k* = the channel with the largest
 *    range (lowest index on ties).
 * 3. s_k* = sqrt(R_x[k*] / R_w[k*]), where R_w[k*] is the range of the weights
 *    that multiply channel k* (max_n W[n,k*] - min_n W[n,k*]): the only slice
 *    that s_k* rescales, so that R_x/s = R_w*s holds after scaling.
 * 4. For every other channel i (Eq. 16 as printed, variant 0):
 *      s_i = s_k* * sqrt(sum_t sum_n |dW[n,i] X[t,i]|) / sqrt(sum_t sum_n |W[n,i] dX[t,i]|)
 *    the sums also running over the calibration rows t (the expectation in
 *    Eq. 5-6). Variant 1 is the exact stationary point of the gain of Eq. 15:
 *      s_i = s_k* * (sum dW^2 X^2 / sum W^2 dX^2)^(1/4).
 *    The two agree when there is one output channel and one row (Eq. 14).
 * Guards (the paper gives none): a zero numerator, denominator or weight range
 * gives s_i = 1; s is clamped to [1e-4, 1e4].
 * k_star_out (optional) receives k*.
 */
void orc_gps(const float* X, int64_t T, int K, const float* W, int N, int bits,
             uint32_t pct_ppm, int variant, float* s, int32_t* k_star_out)
{
    /* 1. quantization errors */
    const int64_t nx = T * (int64_t)K;
    float* ax = (float*)malloc(sizeof(float) * (size_t)nx);
    for (int64_t i = 0; i < nx; ++i) ax[i] = fabsf(X[i]);
    qsort(ax, (size_t)nx, sizeof(float), orc_cmp_float);
    uint64_t rank = ((uint64_t)pct_ppm * (uint64_t)nx + 999999ull) / 1000000ull;
    if (rank < 1) rank = 1;
    if (rank > (uint64_t)nx) rank = (uint64_t)nx;
    const float dx_scale = orc_delta(ax[rank - 1], bits);
    free(ax);

    double* dX = (double*)malloc(sizeof(double) * (size_t)nx);
    for (int64_t i = 0; i < nx; ++i) {
        const float xhat = dx_scale * (float)orc_code(X[i] / dx_scale, bits);
        dX[i] = (double)X[i] - (double)xhat;
    }
    double* dW = (double*)malloc(sizeof(double) * (size_t)N * (size_t)K);
    for (int n = 0; n < N; ++n) {
        float a = 0.0f;
        for (int k = 0; k < K; ++k) {
            const float av = fabsf(W[(int64_t)n * K + k]);
            if (av > a) a = av;
        }
        const float d = orc_delta(a, bits);
        for (int k = 0; k < K; ++k) {
            const float w = W[(int64_t)n * K + k];
            const float what = d * (float)orc_code(w / d, bits);
            dW[(int64_t)n * K + k] = (double)w - (double)what;
        }
    }

    /* 2. channel with the largest activation range */
    int kstar = 0;
    double best = -1.0;
    for (int k = 0; k < K; ++k) {
        double hi = -INFINITY, lo = INFINITY;
        for (int64_t t = 0; t < T; ++t) {
            const double v = X[t * K + k];
            if (v > hi) hi = v;
            if (v < lo) lo = v;
        }
        const double r = hi - lo;
        if (r > best) { best = r; kstar = k; }
    }

    /* 3. s_k* equalises the two ranges */
    double whi = -INFINITY, wlo = INFINITY;
    for (int n = 0; n < N; ++n) {
        const double v = W[(int64_t)n * K + kstar];
        if (v > whi) whi = v;
        if (v < wlo) wlo = v;
    }
    const double rw = whi - wlo;
    double sk = (rw > 0.0 && best > 0.0) ? sqrt(best / rw) : 1.0;

    /* 4. the remaining channels */
#pragma omp parallel for schedule(static)
    for (int i = 0; i < K; ++i) {
        double si;
        if (i == kstar) {
            si = sk;
        } else {
            double num = 0.0, den = 0.0;
            for (int64_t t = 0; t < T; ++t) {
                const double x = X[t * K + i];
                const double dx = dX[t * K + i];
                for (int n = 0; n < N; ++n) {
                    const double w = W[(int64_t)n * K + i];
                    const double dw = dW[(int64_t)n * K + i];
                    if (variant == 0) {
                        num += fabs(dw * x);
                        den += fabs(w * dx);
                    } else {
                        num += (dw * x) * (dw * x);
                        den += (w * dx) * (w * dx);
                    }
                }
            }
            if (!(num > 0.0) || !(den > 0.0)) si = 1.0;
            else if (variant == 0) si = sk * sqrt(num) / sqrt(den);
            else si = sk * sqrt(sqrt(num / den));
        }
        if (si < 1e-4) si = 1e-4;
        if (si > 1e4) si = 1e4;
        s[i] = (float)si;
    }
    if (k_star_out) *k_star_out = kstar;
    free(dX);
    free(dW);
}

/*
 * The scaling gain of Eq. 13 / Eq. 15 for one channel i, as a function of a
 * trial s_i with s_k* fixed; summed over outputs and calibration rows. Used by
 * the tests to check that the closed form is where this function peaks.
 *   g(s_i) = 1/2 sum (W^2 dX^2 + dW^2 X^2) - s_i^2/(2 s_k^2) sum W^2 dX^2
 *            - s_k^2/(2 s_i^2) sum dW^2 X^2
 * The caller passes the two sums: A = sum W^2 dX^2, B = sum dW^2 X^2.
 */
double orc_gps_gain(double A, double B, double s_k, double s_i)
{
    return 0.5 * (A + B) - (s_i * s_i) / (2.0 * s_k * s_k) * A
           - (s_k * s_k) / (2.0 * s_i * s_i) * B;
}

/* ------------------------------------------------------------------------- */
/*
 * Packed storage of 4-bit weight codes (the W4A8 setting of Appendix J, Table 11:
 * 4-bit weights with 8-bit activations). The paper fixes the bit width, not a
 * storage format; the format here is the plain one: two signed 4-bit codes in
 * [-8, 7] per byte, two's complement nibbles, the code of the EVEN input channel
 * in the low nibble and the code of the following ODD channel in the high one:
 *   byte = (c[2j] & 0xF) | ((c[2j+1] & 0xF) << 4).
 * Unpacking sign-extends each nibble. A row of K codes (K even) takes K/2 bytes.
 * orc_pack4 returns -1 if a code lies outside [-8, 7] (nothing is clamped here:
 * clamping is the quantizer's job).
 */
int orc_pack4(const int8_t* codes, int64_t n_pairs, uint8_t* bytes)
{
    for (int64_t j = 0; j < n_pairs; ++j) {
        const int lo = codes[2 * j], hi = codes[2 * j + 1];
        if (lo < -8 || lo > 7 || hi < -8 || hi > 7) return -1;
        bytes[j] = (uint8_t)((lo & 0xF) | ((hi & 0xF) << 4));
    }
    return 0;
}

void orc_unpack4(const uint8_t* bytes, int64_t n_pairs, int8_t* codes)
{
    for (int64_t j = 0; j < n_pairs; ++j) {
        const int lo = bytes[j] & 0xF, hi = (bytes[j] >> 4) & 0xF;
        codes[2 * j] = (int8_t)(lo >= 8 ? lo - 16 : lo);
        codes[2 * j + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
    }
}

/* ------------------------------------------------------------------------- */
/*
 * Quantized attention matmuls and the quantized KV cache (Section 5: 6- or 8-bit
 * quantization of "all linear layers and matrix multiplications"; Appendix C: the
 * KV cache is quantized too). The paper gives no quantizer for these operands
 * beyond static, calibrated parameters (Appendix B; Section 4.2), so the reading
 * is stated here and in the design notes:
 *   - queries and keys: static scale per token position (the STWQ quantizer of
 *     orc_quantize with s_ch = NULL); in S = Q K^T the scale of a query row and of
 *     a key column factor out of the integer sum, so
 *       S[i,j] = acc_qk[i,j] * (s_q[pos_i] * s_kcol[j]),  s_kcol[j] = s_k[pos_j] * softmax_scale
 *     which is orc_epilogue with s_w = s_kcol, no bias, no activation;
 *   - values: one static scale per head channel (orc_quantize with s_ch = s_v and
 *     unit position scales): a scale that varied along the keys could not be taken
 *     out of the sum over keys;
 *   - attention probabilities: Eq. 1 on the fixed range [0, 1]: delta_p = 1/(2^b - 1),
 *     zero point 0, UNSIGNED codes 0 .. 2^b - 1 (orc_softmax_quantize);
 *   - O[i,c] = acc_pv[i,c] * (delta_p * s_v[c]) with acc_pv = sum_j P[i,j] Vq[j,c]
 *     (orc_igemm_u8s8), again orc_epilogue (one "position" with scale delta_p).
 */

/*
 * Row softmax followed by the quantizer of the probabilities. S is [Tq, Tk] fp32
 * (the dequantized scores). causal != 0 masks key j for query i unless
 * j <= i + (Tk - Tq) (the last query sees every key). Computed in double:
 *   m_i = max_j S[i,j],  e_ij = exp(S[i,j] - m_i),  P_ij = e_ij / sum_j e_ij   (masked: 0)
 *   u = P_ij * (2^b - 1),  code = clamp(round(u), 0, 2^b - 1)
 * A row with every key masked gives zeros. u_out (optional) receives u.
 */
void orc_softmax_quantize(const float* S, int Tq, int Tk, int causal, int bits, uint8_t* codes, double* u_out)
{
    const double D = (double)((1 << bits) - 1);
    for (int i = 0; i < Tq; ++i) {
        const int last = causal ? i + (Tk - Tq) : Tk - 1;      /* last visible key */
        double m = -INFINITY;
        for (int j = 0; j < Tk && j <= last; ++j)
            if ((double)S[(int64_t)i * Tk + j] > m) m = (double)S[(int64_t)i * Tk + j];
        double sum = 0.0;
        for (int j = 0; j < Tk && j <= last; ++j) sum += exp((double)S[(int64_t)i * Tk + j] - m);
        for (int j = 0; j < Tk; ++j) {
            double u = 0.0;
            if (j <= last && sum > 0.0) u = exp((double)S[(int64_t)i * Tk + j] - m) / sum * D;
            double r = nearbyint(u);
            if (r < 0.0) r = 0.0;
            if (r > D) r = D;
            codes[(int64_t)i * Tk + j] = (uint8_t)r;
            if (u_out) u_out[(int64_t)i * Tk + j] = u;
        }
    }
}

/* acc[i,c] = sum_j P[i,j] * Vq[j,c], P unsigned 8-bit codes, Vq signed; int32 exact
 * (|acc| <= Tk * 255 * 128). P is [Tq, Tk], Vq is [Tk, C] (key-major, as the values are produced). */
void orc_igemm_u8s8(const uint8_t* P, const int8_t* Vq, int Tq, int Tk, int C, int32_t* acc)
{
    for (int i = 0; i < Tq; ++i)
        for (int c = 0; c < C; ++c) {
            int32_t s = 0;
            for (int j = 0; j < Tk; ++j) s += (int32_t)P[(int64_t)i * Tk + j] * (int32_t)Vq[(int64_t)j * C + c];
            acc[(int64_t)i * C + c] = s;
        }
}

/* ------------------------------------------------------------------------- */
/*
 * Distribution-Guided Calibration (Section 4.3, Eq. 17): the Mahalanobis distance of every
 * sample of a set to the set's own distribution,
 *     rho(x) = sqrt((x - u)^T S^-1 (x - u)),   u = mean, S = covariance of the set,
 * and the selection of the fraction of samples with the largest rho (the paper keeps the top
 * 50 %) as the calibration set. The paper does not say which vector represents a sample; the
 * caller supplies one feature vector per sample, F [n, D].
 * Readings: S is the population covariance (divide by n; the ranking does not depend on the
 * factor); S may be singular (D >= n, constant features), so ridge * trace(S) / D is added to its
 * diagonal (ridge = 0 gives Eq. 17 as printed; a zero-variance set gives rho = 0); S^-1 is applied
 * through the Cholesky factor S = L L^T: rho^2 = |L^-1 (x - u)|^2. k = ceil(keep_ppm * n / 1e6)
 * samples are kept, the largest rho first, equal rho in index order. All in double.
 * Returns 0, or -1 if the (ridged) covariance is not positive definite.
 */
int orc_dgc_select(const float* F, int n, int D, uint32_t keep_ppm, double ridge, double* rho, int32_t* selected)
{
    double* u = (double*)calloc((size_t)D, sizeof(double));
    double* S = (double*)calloc((size_t)D * D, sizeof(double));
    double* y = (double*)malloc(sizeof(double) * (size_t)D);
    int status = 0;
    for (int i = 0; i < n; ++i)
        for (int a = 0; a < D; ++a) u[a] += (double)F[(int64_t)i * D + a];
    for (int a = 0; a < D; ++a) u[a] /= (double)n;
    for (int i = 0; i < n; ++i)
        for (int a = 0; a < D; ++a)
            for (int b = 0; b <= a; ++b)
                S[(int64_t)a * D + b] += ((double)F[(int64_t)i * D + a] - u[a]) * ((double)F[(int64_t)i * D + b] - u[b]);
    double tr = 0.0;
    for (int a = 0; a < D; ++a) {
        for (int b = 0; b <= a; ++b) S[(int64_t)a * D + b] /= (double)n;
        tr += S[(int64_t)a * D + a];
    }
    for (int a = 0; a < D; ++a) S[(int64_t)a * D + a] += ridge * tr / (double)D;
    if (!(tr > 0.0)) {                                   /* every sample equals the mean */
        for (int i = 0; i < n; ++i) rho[i] = 0.0;
    } else {
        /* Cholesky, lower triangle in place: L[a][b] for b <= a */
        for (int k = 0; k < D && status == 0; ++k) {
            double dkk = S[(int64_t)k * D + k];
            for (int b = 0; b < k; ++b) dkk -= S[(int64_t)k * D + b] * S[(int64_t)k * D + b];
            if (!(dkk > 0.0)) { status = -1; break; }
            const double lkk = sqrt(dkk);
            S[(int64_t)k * D + k] = lkk;
            for (int a = k + 1; a < D; ++a) {
                double v = S[(int64_t)a * D + k];
                for (int b = 0; b < k; ++b) v -= S[(int64_t)a * D + b] * S[(int64_t)k * D + b];
                S[(int64_t)a * D + k] = v / lkk;
            }
        }
        for (int i = 0; i < n && status == 0; ++i) {     /* forward substitution L y = x - u */
            double r2 = 0.0;
            for (int a = 0; a < D; ++a) {
                double v = (double)F[(int64_t)i * D + a] - u[a];
                for (int b = 0; b < a; ++b) v -= S[(int64_t)a * D + b] * y[b];
                y[a] = v / S[(int64_t)a * D + a];
                r2 += y[a] * y[a];
            }
            rho[i] = sqrt(r2);
        }
    }
    if (status == 0 && selected) {
        int64_t k = ((int64_t)keep_ppm * n + 999999) / 1000000;
        if (k < 1) k = 1;
        if (k > n) k = n;
        /* selection by rank: sample i is kept if fewer than k samples come before it */
        for (int i = 0; i < n; ++i) {
            int64_t before = 0;
            for (int j = 0; j < n; ++j)
                if (rho[j] > rho[i] || (rho[j] == rho[i] && j < i)) ++before;
            if (before < k) selected[before] = i;
        }
    }
    free(u);
    free(S);
    free(y);
    return status;
}

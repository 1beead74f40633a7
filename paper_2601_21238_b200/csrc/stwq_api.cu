// C ABI of libstwq: context management, argument validation, and the composition of the
// kernels into the calls declared in stwq.h. No arithmetic of the method lives here.
#include <cuda.h>

#include <new>

#include "stwq_internal.cuh"

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_bits(int bits) { return (bits == 8 || bits == 6) ? STWQ_OK : STWQ_ERR_BITS; }
// weights may also be 4-bit (W4A8, Table 11): the codes still travel in int8 containers
int check_wbits(int bits) { return (bits == 8 || bits == 6 || bits == 4) ? STWQ_OK : STWQ_ERR_BITS; }

}  // namespace

// One workspace buffer of the context, grown on demand: free + allocate (both synchronise the
// device). Growth is refused while the stream is being captured into a CUDA graph (an allocation
// there would break the capture) and it bumps the context's workspace generation, because graphs
// captured earlier hold the old address.
int stwq_ensure_ws(stwq_ctx* ctx, void** buf, size_t* have, size_t bytes, cudaStream_t st, size_t zero_prefix)
{
    if (*have >= bytes) return STWQ_OK;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) {
        (void)cudaGetLastError();
        return STWQ_ERR_CAPTURE;        // the query itself fails while another stream of the thread captures
    }
    if (cap != cudaStreamCaptureStatusNone) return STWQ_ERR_CAPTURE;
    if (*buf) {
        cudaError_t e = cudaFree(*buf);                 // synchronises
        if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
        *buf = nullptr;
        *have = 0;
    }
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, bytes);
    if (e == cudaSuccess && zero_prefix > 0) e = cudaMemset(p, 0, zero_prefix);
    if (e != cudaSuccess) {
        ctx->last_cuda_error = (int)e;
        (void)cudaGetLastError();
        if (p) cudaFree(p);
        return STWQ_ERR_NOMEM;
    }
    *buf = p;
    *have = bytes;
    ctx->ws_generation += 1;
    return STWQ_OK;
}

namespace {

int ensure_xq(stwq_ctx* ctx, size_t bytes, cudaStream_t st)
{
    return stwq_ensure_ws(ctx, reinterpret_cast<void**>(&ctx->ws_xq), &ctx->ws_xq_bytes, bytes, st, 0);
}
int ensure_cal(stwq_ctx* ctx, int P, cudaStream_t st)
{
    return stwq_ensure_ws(ctx, &ctx->ws_cal, &ctx->ws_cal_bytes, stwq_calibrate_ws_bytes(P), st, 0);
}
// Per-row workspace of qlinear_dtwq (row scales + row ids) and qlinear_asym (row corrections).
int ensure_dyn(stwq_ctx* ctx, size_t bytes, cudaStream_t st)
{
    return stwq_ensure_ws(ctx, &ctx->ws_dyn, &ctx->ws_dyn_bytes, bytes, st, 0);
}

// Make the context's device current for the duration of a call.
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) {
            cudaSetDevice(dev);
            switched = true;
        }
    }
    ~DeviceGuard()
    {
        if (switched) cudaSetDevice(prev);
    }
};

int check_gemm_args(const void* A, const int32_t* pos_ids, int64_t M, int K, int N, const int8_t* Wq,
                    const float* s_w, const float* s_tok, int P, int act, int out_dtype, const void* Y)
{
    if (!A || !Wq || !Y) return STWQ_ERR_NULL;
    if (out_dtype != STWQ_OUT_INT32 && (!pos_ids || !s_w || !s_tok)) return STWQ_ERR_NULL;
    if (M <= 0 || K <= 0 || N <= 0 || P <= 0) return STWQ_ERR_DIM;
    if (M > (int64_t)0x7fffff00 || K >= 131072) return STWQ_ERR_DIM;   // int32 accumulation bound
    if ((K & 15) != 0 || !aligned16(A) || !aligned16(Wq) || !aligned16(Y)) return STWQ_ERR_ALIGN;
    if (act < STWQ_ACT_NONE || act > STWQ_ACT_GELU_FAST) return STWQ_ERR_BITS;
    if (out_dtype < STWQ_OUT_F32 || out_dtype > STWQ_OUT_INT32) return STWQ_ERR_BITS;
    return STWQ_OK;
}

int run_gemm(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K, int N,
             const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* bias, int act,
             int out_dtype, void* Y, bool after_quantize, cudaStream_t st)
{
    const bool can_decode = M <= 256;
    // the few-row kernel gives each CTA pair one 128-column slice; with more slices than pairs it
    // would run in two rounds and re-read Xq once per slice, and the tiled GEMM with its
    // 256-column tiles is the faster one (M 256, N 16384, K 4096: 22 against 34 us)
    bool decode = can_decode && (N + 127) / 128 <= ctx->sm_count / 2;
    if (ctx->gemm_path == 1 || ctx->gemm_path == 3) decode = false;
    if (ctx->gemm_path == 2 && !can_decode) return STWQ_ERR_DIM;
    if (ctx->gemm_path == 2) decode = true;
    if (decode)
        return stwq_launch_decode(ctx, Xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype, Y,
                                  after_quantize, st);
    if (ctx->gemm_path != 3 && stwq_qgemm2_supported(N, out_dtype, s_w, bias))
        return stwq_launch_qgemm2(ctx, Xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype, Y,
                                  after_quantize, nullptr, st);
    return stwq_launch_qgemm(ctx, Xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype, Y, st);
}

}  // namespace

extern "C" {

int stwq_create(stwq_ctx** out, int device)
{
    if (!out) return STWQ_ERR_NULL;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        (void)cudaGetLastError();
        return STWQ_ERR_CUDA;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return STWQ_ERR_CUDA;
    if (prop.major != 10) return STWQ_ERR_ARCH;
    stwq_ctx* ctx = new (std::nothrow) stwq_ctx();
    if (!ctx) return STWQ_ERR_NOMEM;
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->l2_bytes = prop.l2CacheSize;
    ctx->gemm_path = 0;
    ctx->wait_limit_ms = 2000;
    DeviceGuard g(device);
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&ctx->d_status), 256);
    if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, 256);
    if (e != cudaSuccess) {
        delete ctx;
        return STWQ_ERR_CUDA;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
        cudaFree(ctx->d_status);
        delete ctx;
        return STWQ_ERR_CUDA;
    }
    ctx->encode_tiled = fn;
    *out = ctx;
    return STWQ_OK;
}

void stwq_destroy(stwq_ctx* ctx)
{
    if (!ctx) return;
    DeviceGuard g(ctx->device);
    cudaDeviceSynchronize();
    if (ctx->ws_xq) cudaFree(ctx->ws_xq);
    if (ctx->ws_cal) cudaFree(ctx->ws_cal);
    if (ctx->ws_dec) cudaFree(ctx->ws_dec);
    if (ctx->ws_dyn) cudaFree(ctx->ws_dyn);
    if (ctx->ws_w4) cudaFree(ctx->ws_w4);
    if (ctx->ws_attn) cudaFree(ctx->ws_attn);
    if (ctx->d_status) cudaFree(ctx->d_status);
    delete ctx;
}

int stwq_reserve(stwq_ctx* ctx, int64_t M, int K, int P)
{
    if (!ctx) return STWQ_ERR_NULL;
    if (M < 0 || K < 0 || P < 0) return STWQ_ERR_DIM;
    DeviceGuard g(ctx->device);
    int rc = STWQ_OK;
    if (M > 0 && K > 0) rc = ensure_xq(ctx, (size_t)M * (size_t)K, nullptr);
    if (rc == STWQ_OK && P > 0) rc = ensure_cal(ctx, P, nullptr);
    return rc;
}

int stwq_reserve_layer(stwq_ctx* ctx, int64_t M, int K, int N, int P)
{
    if (!ctx) return STWQ_ERR_NULL;
    if (M <= 0 || K <= 0 || N <= 0 || P <= 0) return STWQ_ERR_DIM;
    DeviceGuard g(ctx->device);
    int rc = ensure_xq(ctx, (size_t)M * (size_t)K, nullptr);
    if (rc == STWQ_OK) rc = ensure_cal(ctx, P, nullptr);
    // per-row scratch of qlinear_dtwq / qlinear_asym, column statistics of gps_scales
    size_t dyn = (size_t)M * 8;
    if (stwq_gps_ws_bytes(K, N) > dyn) dyn = stwq_gps_ws_bytes(K, N);
    if (rc == STWQ_OK) rc = ensure_dyn(ctx, dyn, nullptr);
    // int8 copy of packed 4-bit weights (qlinear_w4)
    if (rc == STWQ_OK)
        rc = stwq_ensure_ws(ctx, reinterpret_cast<void**>(&ctx->ws_w4), &ctx->ws_w4_bytes, (size_t)N * (size_t)K, nullptr, 0);
    // int32 partial sums of the few-row path when it splits K
    if (rc == STWQ_OK && M <= 256) {
        const size_t split = stwq_decode_split_bytes(ctx, K, N);
        uint32_t* c = nullptr;
        int32_t* part = nullptr;
        if (split > 0) {
            rc = stwq_split_ws(ctx, split, 1, &c, &part, nullptr);
            if (rc == STWQ_ERR_DIM) rc = STWQ_OK;
        }
    }
    return rc;
}

int stwq_set_option(stwq_ctx* ctx, int option, int value)
{
    if (!ctx) return STWQ_ERR_NULL;
    if (option == STWQ_OPT_GEMM_PATH && value >= 0 && value <= 3) {
        ctx->gemm_path = value;
        return STWQ_OK;
    }
    if (option == STWQ_OPT_WAIT_LIMIT_MS && value >= 1 && value <= 60000) {
        ctx->wait_limit_ms = value;
        return STWQ_OK;
    }
    if (option == STWQ_OPT_TILE_N && (value == 0 || value == 128 || value == 256)) {
        ctx->force_bn = value;
        return STWQ_OK;
    }
    if (option == STWQ_OPT_VARIANT && (value == 0 || value == 1 || value == 2 || value == 5 || value == 7 || value == 8 || value == 9)) {
        ctx->debug = value;
        return STWQ_OK;
    }
    if (option == STWQ_OPT_KSPLIT && value >= -1 && value <= 64) {
        ctx->force_ksplit = value;
        return STWQ_OK;
    }
    return STWQ_ERR_DIM;
}

int stwq_calibrate(stwq_ctx* ctx, const float* Xcal, const int32_t* pos_ids, int64_t rows, int K, int P,
                   const float* s_ch, int bits, uint32_t pct_ppm, float* s_tok, void* stream)
{
    if (!ctx || !Xcal || !pos_ids || !s_tok) return STWQ_ERR_NULL;
    if (rows <= 0 || K <= 0 || P <= 0 || P > (1 << 20)) return STWQ_ERR_DIM;
    if (check_bits(bits) != STWQ_OK || pct_ppm < 1u || pct_ppm > 1000000u) return STWQ_ERR_BITS;
    DeviceGuard g(ctx->device);
    int rc = ensure_cal(ctx, P, static_cast<cudaStream_t>(stream));
    if (rc != STWQ_OK) return rc;
    return stwq_launch_calibrate(ctx, ctx->ws_cal, Xcal, pos_ids, rows, K, P, s_ch, bits, pct_ppm, s_tok,
                                 static_cast<cudaStream_t>(stream));
}

int gps_scales(stwq_ctx* ctx, const float* Xcal, int64_t rows, int K, const float* W, int N, int bits,
               uint32_t pct_ppm, int variant, float* s_ch, int32_t* k_star, void* stream)
{
    if (!ctx || !Xcal || !W || !s_ch) return STWQ_ERR_NULL;
    if (rows <= 0 || K <= 0 || N <= 0) return STWQ_ERR_DIM;
    if (check_bits(bits) != STWQ_OK || pct_ppm < 1u || pct_ppm > 1000000u) return STWQ_ERR_BITS;
    if (variant != 0 && variant != 1) return STWQ_ERR_BITS;
    DeviceGuard g(ctx->device);
    int rc = ensure_cal(ctx, 1, static_cast<cudaStream_t>(stream));
    if (rc == STWQ_OK) rc = ensure_dyn(ctx, stwq_gps_ws_bytes(K, N), static_cast<cudaStream_t>(stream));
    if (rc != STWQ_OK) return rc;
    return stwq_launch_gps(ctx, ctx->ws_cal, ctx->ws_dyn, Xcal, rows, K, W, N, bits, pct_ppm, variant, s_ch, k_star,
                           static_cast<cudaStream_t>(stream));
}

int dgc_select(stwq_ctx* ctx, const float* F, int n, int D, uint32_t keep_ppm, double ridge, double* rho,
               int32_t* selected, void* stream)
{
    if (!ctx || !F || !rho) return STWQ_ERR_NULL;
    if (n <= 0 || D <= 0 || D > 1024 || n > (1 << 20)) return STWQ_ERR_DIM;
    if (keep_ppm < 1u || keep_ppm > 1000000u || !(ridge >= 0.0)) return STWQ_ERR_BITS;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = ensure_dyn(ctx, stwq_dgc_ws_bytes(D), st);
    if (rc != STWQ_OK) return rc;
    int64_t k = ((int64_t)keep_ppm * n + 999999) / 1000000;
    if (k < 1) k = 1;
    if (k > n) k = n;
    return stwq_launch_dgc(ctx, ctx->ws_dyn, F, n, D, (int)k, ridge, rho, selected, st);
}

int gps_fold(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, int bits, int8_t* Wq,
             float* s_w, void* stream)
{
    if (!ctx || !W || !Wq || !s_w) return STWQ_ERR_NULL;
    if (N <= 0 || K <= 0) return STWQ_ERR_DIM;
    if (check_wbits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    DeviceGuard g(ctx->device);
    return stwq_launch_fold(ctx, W, N, K, s_ch, bits, Wq, s_w, static_cast<cudaStream_t>(stream));
}

int gps_fold_packed4(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, uint8_t* Wp, float* s_w,
                     void* stream)
{
    if (!ctx || !W || !Wp || !s_w) return STWQ_ERR_NULL;
    if (N <= 0 || K <= 0) return STWQ_ERR_DIM;
    if ((K & 31) != 0 || !aligned16(Wp)) return STWQ_ERR_ALIGN;     // rows of K / 2 bytes stay 16-byte aligned
    DeviceGuard g(ctx->device);
    return stwq_launch_fold_packed4(ctx, W, N, K, s_ch, Wp, s_w, static_cast<cudaStream_t>(stream));
}

int stwq_unpack4(stwq_ctx* ctx, const uint8_t* Wp, int N, int K, int8_t* Wq, void* stream)
{
    if (!ctx || !Wp || !Wq) return STWQ_ERR_NULL;
    if (N <= 0 || K <= 0) return STWQ_ERR_DIM;
    if ((K & 31) != 0 || !aligned16(Wp) || !aligned16(Wq)) return STWQ_ERR_ALIGN;
    DeviceGuard g(ctx->device);
    return stwq_launch_unpack4(ctx, Wp, (int64_t)N * (K / 2), Wq, static_cast<cudaStream_t>(stream));
}

int qlinear_w4(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, int N, const uint8_t* Wp,
               const float* s_w, const float* s_tok, int P, const float* s_ch, const float* bias, int bits, int act,
               int out_dtype, void* Y, void* stream)
{
    if (!ctx) return STWQ_ERR_NULL;
    if (!pos_ids || !s_tok || !s_w) return STWQ_ERR_NULL;
    int rc = check_gemm_args(X, pos_ids, M, K, N, reinterpret_cast<const int8_t*>(Wp), s_w, s_tok, P, act, out_dtype, Y);
    if (rc != STWQ_OK) return rc;
    if (check_bits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    if ((K & 31) != 0) return STWQ_ERR_ALIGN;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = ensure_xq(ctx, (size_t)M * (size_t)K, st);
    if (rc == STWQ_OK)
        rc = stwq_ensure_ws(ctx, reinterpret_cast<void**>(&ctx->ws_w4), &ctx->ws_w4_bytes, (size_t)N * (size_t)K, st, 0);
    if (rc != STWQ_OK) return rc;
    // the weights travel through HBM as half a byte per code; the tensor cores take int8, so the
    // codes are widened into workspace first (N K bytes written once, then read from L2 / HBM by the GEMM)
    rc = stwq_launch_unpack4(ctx, Wp, (int64_t)N * (K / 2), ctx->ws_w4, st);
    if (rc != STWQ_OK) return rc;
    rc = stwq_launch_quantize(ctx, X, pos_ids, M, K, s_ch, s_tok, P, bits, ctx->ws_xq, false, st);
    if (rc != STWQ_OK) return rc;
    return run_gemm(ctx, ctx->ws_xq, pos_ids, M, K, N, ctx->ws_w4, s_w, s_tok, P, bias, act, out_dtype, Y, ctx->debug != 5, st);
}

int stwq_quantize(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K,
                  const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq, void* stream)
{
    if (!ctx || !X || !pos_ids || !s_tok || !Xq) return STWQ_ERR_NULL;
    if (M <= 0 || K <= 0 || P <= 0) return STWQ_ERR_DIM;
    if (check_bits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    if ((K & 15) != 0 || !aligned16(X) || !aligned16(Xq)) return STWQ_ERR_ALIGN;
    DeviceGuard g(ctx->device);
    return stwq_launch_quantize(ctx, X, pos_ids, M, K, s_ch, s_tok, P, bits, Xq, false,
                                static_cast<cudaStream_t>(stream));
}

int stwq_quantize_bf16(stwq_ctx* ctx, const void* X, const int32_t* pos_ids, int64_t M, int K,
                       const float* s_ch, const float* s_tok, int P, int bits, int8_t* Xq, void* stream)
{
    if (!ctx || !X || !pos_ids || !s_tok || !Xq) return STWQ_ERR_NULL;
    if (M <= 0 || K <= 0 || P <= 0) return STWQ_ERR_DIM;
    if (check_bits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    if ((K & 15) != 0 || !aligned16(X) || !aligned16(Xq)) return STWQ_ERR_ALIGN;
    DeviceGuard g(ctx->device);
    return stwq_launch_quantize_bf16(ctx, X, pos_ids, M, K, s_ch, s_tok, P, bits, Xq, static_cast<cudaStream_t>(stream));
}

int qlinear_q(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K, int N,
              const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* bias, int act,
              int out_dtype, void* Y, void* stream)
{
    if (!ctx) return STWQ_ERR_NULL;
    int rc = check_gemm_args(Xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, act, out_dtype, Y);
    if (rc != STWQ_OK) return rc;
    DeviceGuard g(ctx->device);
    return run_gemm(ctx, Xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype, Y, false,
                    static_cast<cudaStream_t>(stream));
}

int qlinear(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, int N,
            const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* s_ch,
            const float* bias, int bits, int act, int out_dtype, void* Y, void* stream)
{
    if (!ctx) return STWQ_ERR_NULL;
    if (!pos_ids || !s_tok || !s_w) return STWQ_ERR_NULL;
    int rc = check_gemm_args(X, pos_ids, M, K, N, Wq, s_w, s_tok, P, act, out_dtype, Y);
    if (rc != STWQ_OK) return rc;
    if (check_bits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    DeviceGuard g(ctx->device);
    rc = ensure_xq(ctx, (size_t)M * (size_t)K, static_cast<cudaStream_t>(stream));
    if (rc != STWQ_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Both kernels are launched as programmatic dependents of their predecessor in the stream:
    // each executes griddepcontrol.wait before it reads or writes anything the predecessor could
    // have produced, so the order of effects is that of ordinary launches; what overlaps is the
    // launch itself and the GEMM's prologue.
    const bool pdl = ctx->debug != 5;                     // tuning: 5 = ordinary launches
    rc = stwq_launch_quantize(ctx, X, pos_ids, M, K, s_ch, s_tok, P, bits, ctx->ws_xq, pdl, st);
    if (rc != STWQ_OK) return rc;
    return run_gemm(ctx, ctx->ws_xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype, Y, pdl, st);
}

int qlinear_bf16(stwq_ctx* ctx, const void* X, const int32_t* pos_ids, int64_t M, int K, int N,
                 const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* s_ch,
                 const float* bias, int bits, int act, int out_dtype, void* Y, void* stream)
{
    if (!ctx) return STWQ_ERR_NULL;
    if (!pos_ids || !s_tok || !s_w) return STWQ_ERR_NULL;
    int rc = check_gemm_args(X, pos_ids, M, K, N, Wq, s_w, s_tok, P, act, out_dtype, Y);
    if (rc != STWQ_OK) return rc;
    if (check_bits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    DeviceGuard g(ctx->device);
    rc = ensure_xq(ctx, (size_t)M * (size_t)K, static_cast<cudaStream_t>(stream));
    if (rc != STWQ_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = stwq_launch_quantize_bf16(ctx, X, pos_ids, M, K, s_ch, s_tok, P, bits, ctx->ws_xq, st);
    if (rc != STWQ_OK) return rc;
    // the GEMM is a programmatic dependent of the quantize kernel, as in qlinear
    return run_gemm(ctx, ctx->ws_xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype, Y, ctx->debug != 5, st);
}

static int chain_args(const void* A, const int32_t* pos_ids, int64_t M, int K, int N, const int8_t* Wq,
                      const float* s_w, const float* s_tok, int P, const float* bias, int act,
                      const float* s_ch_next, const float* s_tok_next, int bits_next, const int8_t* Xq_next)
{
    if (!pos_ids || !s_tok || !s_w || !s_tok_next) return STWQ_ERR_NULL;
    int rc = check_gemm_args(A, pos_ids, M, K, N, Wq, s_w, s_tok, P, act, STWQ_OUT_F32, Xq_next);
    if (rc != STWQ_OK) return rc;
    if (check_bits(bits_next) != STWQ_OK) return STWQ_ERR_BITS;
    // the fused epilogue lives in the CTA-pair kernel only: 16-byte rows of codes, aligned vectors
    if ((N & 15) != 0 || !stwq_qgemm2_supported(N, 3, s_w, bias)) return STWQ_ERR_ALIGN;
    if (s_ch_next != nullptr && (reinterpret_cast<uintptr_t>(s_ch_next) & 15u) != 0) return STWQ_ERR_ALIGN;
    return STWQ_OK;
}

int qlinear_chain_q(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K, int N,
                    const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* bias, int act,
                    const float* s_ch_next, const float* s_tok_next, int bits_next, int8_t* Xq_next, void* stream)
{
    if (!ctx) return STWQ_ERR_NULL;
    int rc = chain_args(Xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, s_ch_next, s_tok_next, bits_next, Xq_next);
    if (rc != STWQ_OK) return rc;
    DeviceGuard g(ctx->device);
    const stwq_chain chain = {s_ch_next, s_tok_next, bits_next};
    return stwq_launch_qgemm2(ctx, Xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, 3, Xq_next, false, &chain,
                              static_cast<cudaStream_t>(stream));
}

int qlinear_chain(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, int N,
                  const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* s_ch,
                  const float* bias, int bits, int act, const float* s_ch_next, const float* s_tok_next,
                  int bits_next, int8_t* Xq_next, void* stream)
{
    if (!ctx) return STWQ_ERR_NULL;
    int rc = chain_args(X, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, s_ch_next, s_tok_next, bits_next, Xq_next);
    if (rc != STWQ_OK) return rc;
    if (check_bits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    DeviceGuard g(ctx->device);
    rc = ensure_xq(ctx, (size_t)M * (size_t)K, static_cast<cudaStream_t>(stream));
    if (rc != STWQ_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool pdl = ctx->debug != 5;
    rc = stwq_launch_quantize(ctx, X, pos_ids, M, K, s_ch, s_tok, P, bits, ctx->ws_xq, pdl, st);
    if (rc != STWQ_OK) return rc;
    const stwq_chain chain = {s_ch_next, s_tok_next, bits_next};
    return stwq_launch_qgemm2(ctx, ctx->ws_xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, 3, Xq_next, pdl, &chain, st);
}

// ---- asymmetric quantizer (Eq. 1 as printed)
int stwq_calibrate_asym(stwq_ctx* ctx, const float* Xcal, const int32_t* pos_ids, int64_t rows, int K, int P,
                        const float* s_ch, int bits, uint32_t pct_ppm, float* s_tok, int32_t* z_tok, void* stream)
{
    if (!ctx || !Xcal || !pos_ids || !s_tok || !z_tok) return STWQ_ERR_NULL;
    if (rows <= 0 || K <= 0 || P <= 0 || P > (1 << 20)) return STWQ_ERR_DIM;
    if (check_bits(bits) != STWQ_OK || pct_ppm < 1u || pct_ppm > 1000000u) return STWQ_ERR_BITS;
    DeviceGuard g(ctx->device);
    int rc = ensure_cal(ctx, P, static_cast<cudaStream_t>(stream));
    if (rc != STWQ_OK) return rc;
    return stwq_launch_calibrate_asym(ctx, ctx->ws_cal, Xcal, pos_ids, rows, K, P, s_ch, bits, pct_ppm, s_tok, z_tok,
                                      static_cast<cudaStream_t>(stream));
}

int gps_fold_asym(stwq_ctx* ctx, const float* W, int N, int K, const float* s_ch, int bits, int8_t* Wq, float* s_w,
                  int32_t* z_w, int32_t* colsum, void* stream)
{
    if (!ctx || !W || !Wq || !s_w || !z_w || !colsum) return STWQ_ERR_NULL;
    if (N <= 0 || K <= 0) return STWQ_ERR_DIM;
    if (check_wbits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    DeviceGuard g(ctx->device);
    return stwq_launch_fold_asym(ctx, W, N, K, s_ch, bits, Wq, s_w, z_w, colsum, static_cast<cudaStream_t>(stream));
}

int stwq_quantize_asym(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, const float* s_ch,
                       const float* s_tok, const int32_t* z_tok, int P, int bits, int8_t* Xq, int32_t* rowcorr,
                       void* stream)
{
    if (!ctx || !X || !pos_ids || !s_tok || !z_tok || !Xq || !rowcorr) return STWQ_ERR_NULL;
    if (M <= 0 || K <= 0 || P <= 0) return STWQ_ERR_DIM;
    if (check_bits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    if ((K & 15) != 0 || !aligned16(X) || !aligned16(Xq)) return STWQ_ERR_ALIGN;
    DeviceGuard g(ctx->device);
    return stwq_launch_quantize_asym(ctx, X, pos_ids, M, K, s_ch, s_tok, z_tok, P, bits, Xq, rowcorr,
                                     static_cast<cudaStream_t>(stream));
}

int qlinear_asym(stwq_ctx* ctx, const float* X, const int32_t* pos_ids, int64_t M, int K, int N, const int8_t* Wq,
                 const float* s_w, const int32_t* z_w, const int32_t* colsum, const float* s_tok, const int32_t* z_tok,
                 int P, const float* s_ch, const float* bias, int bits, int act, int out_dtype, void* Y, void* stream)
{
    if (!ctx || !pos_ids || !s_tok || !s_w || !z_w || !colsum || !z_tok) return STWQ_ERR_NULL;
    int rc = check_gemm_args(X, pos_ids, M, K, N, Wq, s_w, s_tok, P, act, out_dtype, Y);
    if (rc != STWQ_OK) return rc;
    if (check_bits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    if (K > 32768 || M > (int64_t)0x7fffffff) return STWQ_ERR_DIM;     // the corrections stay inside int32
    // the corrected epilogue lives in the CTA-pair kernel: 16-byte rows of Y, aligned per-column vectors
    if (!stwq_qgemm2_supported(N, out_dtype, s_w, bias) || (N & 3) != 0 || !aligned16(z_w) || !aligned16(colsum))
        return STWQ_ERR_ALIGN;
    DeviceGuard g(ctx->device);
    rc = ensure_xq(ctx, (size_t)M * (size_t)K, static_cast<cudaStream_t>(stream));
    if (rc != STWQ_OK) return rc;
    rc = ensure_dyn(ctx, (size_t)M * 8, static_cast<cudaStream_t>(stream));
    if (rc != STWQ_OK) return rc;
    int32_t* rowcorr = static_cast<int32_t*>(ctx->ws_dyn);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = stwq_launch_quantize_asym(ctx, X, pos_ids, M, K, s_ch, s_tok, z_tok, P, bits, ctx->ws_xq, rowcorr, st);
    if (rc != STWQ_OK) return rc;
    const stwq_asym asym = {z_tok, z_w, colsum, rowcorr};
    // the GEMM is a programmatic dependent of the quantize kernel, as in qlinear
    return stwq_launch_qgemm2(ctx, ctx->ws_xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype, Y,
                              ctx->debug != 5, nullptr, st, &asym);
}

int dtwq_quantize(stwq_ctx* ctx, const float* X, int64_t M, int K, const float* s_ch, int bits, int8_t* Xq,
                  float* s_row, void* stream)
{
    if (!ctx || !X || !Xq || !s_row) return STWQ_ERR_NULL;
    if (M <= 0 || K <= 0 || K > 8192) return STWQ_ERR_DIM;
    if (check_bits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    if ((K & 15) != 0 || !aligned16(X) || !aligned16(Xq)) return STWQ_ERR_ALIGN;
    DeviceGuard g(ctx->device);
    return stwq_launch_dtwq(ctx, X, M, K, s_ch, bits, Xq, s_row, nullptr, static_cast<cudaStream_t>(stream));
}

int qlinear_dtwq(stwq_ctx* ctx, const float* X, int64_t M, int K, int N, const int8_t* Wq, const float* s_w,
                 const float* s_ch, const float* bias, int bits, int act, int out_dtype, void* Y, void* stream)
{
    if (!ctx || !s_w) return STWQ_ERR_NULL;
    static const int32_t dummy_pos = 0;
    static const float dummy_tok = 1.0f;
    int rc = check_gemm_args(X, &dummy_pos, M, K, N, Wq, s_w, &dummy_tok, 1, act, out_dtype, Y);
    if (rc != STWQ_OK) return rc;
    if (check_bits(bits) != STWQ_OK) return STWQ_ERR_BITS;
    if (K > 8192 || M > (int64_t)0x7fffffff) return STWQ_ERR_DIM;
    DeviceGuard g(ctx->device);
    rc = ensure_xq(ctx, (size_t)M * (size_t)K, static_cast<cudaStream_t>(stream));
    if (rc != STWQ_OK) return rc;
    rc = ensure_dyn(ctx, (size_t)M * 8, static_cast<cudaStream_t>(stream));
    if (rc != STWQ_OK) return rc;
    float* s_row = static_cast<float*>(ctx->ws_dyn);
    int32_t* row_ids = reinterpret_cast<int32_t*>(s_row + M);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = stwq_launch_dtwq(ctx, X, M, K, s_ch, bits, ctx->ws_xq, s_row, row_ids, st);
    if (rc != STWQ_OK) return rc;
    // the dequantizer takes the row's own scale: position id = row index, table = the scales just computed
    return run_gemm(ctx, ctx->ws_xq, row_ids, M, K, N, Wq, s_w, s_row, (int)M, bias, act, out_dtype, Y, false, st);
}

int stwq_device_status(stwq_ctx* ctx, void* stream)
{
    if (!ctx) return STWQ_ERR_NULL;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t h = 0;
    cudaError_t e = cudaMemcpyAsync(&h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(h), st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
    if (h & STWQ_DEV_TIMEOUT) return STWQ_ERR_DEVICE_TIMEOUT;
    if (h & STWQ_DEV_POS_RANGE) return STWQ_ERR_POS_RANGE;
    if (h & STWQ_DEV_NONFINITE) return STWQ_ERR_NONFINITE;
    return STWQ_OK;
}

int64_t stwq_launch_count(const stwq_ctx* ctx) { return ctx ? ctx->launches : 0; }

uint64_t stwq_workspace_generation(const stwq_ctx* ctx) { return ctx ? ctx->ws_generation : 0; }

int stwq_last_cuda_error(const stwq_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

const char* stwq_strerror(int status)
{
    switch (status) {
        case STWQ_OK: return "ok";
        case STWQ_ERR_NULL: return "a required pointer is NULL";
        case STWQ_ERR_DIM: return "a size is out of range";
        case STWQ_ERR_ALIGN: return "alignment rule violated (16-byte pointers, K multiple of 16)";
        case STWQ_ERR_BITS: return "unsupported bits / activation / output type / percentile";
        case STWQ_ERR_ARCH: return "device is not compute capability 10.x";
        case STWQ_ERR_CUDA: return "a CUDA call failed";
        case STWQ_ERR_DEVICE_TIMEOUT: return "a device-side wait expired";
        case STWQ_ERR_POS_RANGE: return "a position id was outside [0, P)";
        case STWQ_ERR_NONFINITE: return "calibration input contains NaN or Inf";
        case STWQ_ERR_NOMEM: return "workspace allocation failed";
        case STWQ_ERR_CAPTURE: return "workspace would have to grow during stream capture (reserve it first)";
        default: return "unknown status";
    }
}

}  // extern "C"

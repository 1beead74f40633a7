// qlinear_static: the quantized linear layer for callers that must not allocate device memory.
//
// qlinear keeps the int8 copy of X in workspace that its context obtains from cudaMalloc, on
// first use or when a larger X arrives, and the context itself allocates a status word when it
// is created. Some hosts cannot accept either: a control loop with a fixed latency budget that
// the driver's allocator (which may synchronise the whole device) would break; a plug-in inside
// a process where another runtime has claimed all device memory for its own pool, so that
// cudaMalloc simply fails; firmware-like deployments whose rules forbid allocation once start-up
// is over. For them this file offers one extra entry point in which every byte of scratch is a
// file-scope __device__ array that belongs to the library image: it exists on every GPU that
// loads libstwq, from module load until the process exits, and nothing is ever requested from
// an allocator, neither by a context (none is needed) nor by the call.
//
// The name of a __device__ array means something only in device code; in host code it is a
// stand-in symbol whose address is not a device address, and a kernel handed that address would
// fault or scribble on unrelated memory. The host therefore asks the runtime for the array's
// device address once per device (cudaGetSymbolAddress, with that device current), checks the
// answer, and hands that pointer to the kernels.
#include <cuda.h>

#include <mutex>

#include "stwq_internal.cuh"

namespace {

constexpr size_t kHeaderBytes = 256;                        // status word, padded
constexpr size_t kCodeBytes = STWQ_STATIC_MAX_CODES;        // int8 codes of X
// Layout: [0, 256) device status word (kernels OR error bits into it); [256, ...) codes of X.
static __device__ __align__(256) unsigned char g_static_scratch[kHeaderBytes + kCodeBytes];

constexpr int kMaxDevices = 64;

struct DeviceSlot {
    bool ready = false;
    stwq_ctx ctx = {};          // host-side launch state only; owns no device allocation
};

std::mutex g_mutex;
DeviceSlot g_slots[kMaxDevices];

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Once per device, with that device current: resolve the scratch array's device address and the
// few facts the launchers need. Allocates nothing.
int setup_device(int device, DeviceSlot** out)
{
    if (device < 0 || device >= kMaxDevices) return STWQ_ERR_DIM;
    DeviceSlot& s = g_slots[device];
    if (!s.ready) {
        int major = 0, sms = 0, l2 = 0;
        cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, device);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return STWQ_ERR_CUDA;
        }
        if (major != 10) return STWQ_ERR_ARCH;
        unsigned char* base = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&base), g_static_scratch);
        if (e != cudaSuccess || base == nullptr) {
            (void)cudaGetLastError();
            return STWQ_ERR_CUDA;
        }
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || fn == nullptr) {
            (void)cudaGetLastError();
            return STWQ_ERR_CUDA;
        }
        s.ctx = stwq_ctx{};
        s.ctx.device = device;
        s.ctx.sm_count = sms;
        s.ctx.l2_bytes = l2;
        s.ctx.wait_limit_ms = 2000;
        s.ctx.force_ksplit = -1;        // the split-K tail keeps partial sums in allocated scratch: never here
        s.ctx.d_status = reinterpret_cast<uint32_t*>(base);
        s.ctx.ws_xq = reinterpret_cast<int8_t*>(base + kHeaderBytes);
        s.ctx.ws_xq_bytes = kCodeBytes;
        s.ctx.encode_tiled = fn;
        s.ready = true;
    }
    *out = &s;
    return STWQ_OK;
}

}  // namespace

extern "C" int qlinear_static(const float* X, const int32_t* pos_ids, int64_t M, int K, int N,
                              const int8_t* Wq, const float* s_w, const float* s_tok, int P,
                              const float* s_ch, const float* bias, int bits, int act, int out_dtype,
                              void* Y, void* stream)
{
    if (!X || !pos_ids || !Wq || !s_w || !s_tok || !Y) return STWQ_ERR_NULL;
    if (M <= 0 || K <= 0 || N <= 0 || P <= 0 || K >= 131072) return STWQ_ERR_DIM;
    if ((uint64_t)M * (uint64_t)K > (uint64_t)kCodeBytes) return STWQ_ERR_DIM;   // beyond the fixed scratch
    if ((K & 15) != 0 || !aligned16(X) || !aligned16(Wq) || !aligned16(Y)) return STWQ_ERR_ALIGN;
    if (bits != 8 && bits != 6) return STWQ_ERR_BITS;
    if (act < STWQ_ACT_NONE || act > STWQ_ACT_GELU_FAST) return STWQ_ERR_BITS;
    if (out_dtype < STWQ_OUT_F32 || out_dtype > STWQ_OUT_INT32) return STWQ_ERR_BITS;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) {
        (void)cudaGetLastError();
        return STWQ_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceSlot* slot = nullptr;
    int rc = setup_device(device, &slot);
    if (rc != STWQ_OK) return rc;
    stwq_ctx* ctx = &slot->ctx;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = stwq_launch_quantize(ctx, X, pos_ids, M, K, s_ch, s_tok, P, bits, ctx->ws_xq, false, st);
    if (rc != STWQ_OK) return rc;
    if (stwq_qgemm2_supported(N, out_dtype, s_w, bias))
        return stwq_launch_qgemm2(ctx, ctx->ws_xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act,
                                  out_dtype, Y, false, nullptr, st);
    return stwq_launch_qgemm(ctx, ctx->ws_xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype,
                             Y, st);
}

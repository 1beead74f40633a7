// Few-row (decode-step) variant of the quantized linear. Placeholder routing: until the
// bandwidth-bound kernel lands, few-row calls use the tiled tensor-core GEMM.
#include "stwq_internal.cuh"

int stwq_launch_decode(stwq_ctx* ctx, const int8_t* Xq, const int32_t* pos_ids, int64_t M, int K, int N,
                       const int8_t* Wq, const float* s_w, const float* s_tok, int P, const float* bias,
                       int act, int out_dtype, void* Y, cudaStream_t st)
{
    return stwq_launch_qgemm(ctx, Xq, pos_ids, M, K, N, Wq, s_w, s_tok, P, bias, act, out_dtype, Y, st);
}

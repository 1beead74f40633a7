// Distribution-Guided Calibration (Section 4.3, Eq. 17): rho(x) = sqrt((x - u)^T S^-1 (x - u)) for
// every sample of a set against the set's own mean u and covariance S, and the selection of the
// fraction of samples with the largest rho as the calibration set. Offline, small (a few hundred
// samples, a few hundred features), in fp64 throughout:
//
//   dgc_mean_kernel   u[a] = mean over samples                         (one thread per feature)
//   dgc_cov_kernel    S[a][b] = mean of (x_a - u_a)(x_b - u_b), lower triangle, then the ridge
//   dgc_chol_kernel   S = L L^T in place, one block (right-looking, a barrier per column)
//   dgc_rho_kernel    forward substitution L y = x - u, one warp per sample; rho = |y|
//   dgc_rank_kernel   rank by (rho descending, index ascending); the first k ranks are the selection
//
// Sums run over samples and features in index order inside each thread; only the dot products
// of the substitution are split across lanes, so rho agrees with a sequential evaluation to
// rounding (relative 1e-12) and the selection is the same except between samples whose distances
// agree to that precision.
#include "stwq_internal.cuh"

namespace {

__global__ void dgc_mean_kernel(const float* __restrict__ F, int n, int D, double* __restrict__ u)
{
    const int a = blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= D) return;
    double s = 0.0;
    for (int i = 0; i < n; ++i) s += (double)F[(int64_t)i * D + a];
    u[a] = s / (double)n;
}

__global__ void dgc_cov_kernel(const float* __restrict__ F, int n, int D, const double* __restrict__ u,
                               double* __restrict__ S)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    const int a = blockIdx.y;
    if (b > a || b >= D) return;
    const double ua = u[a], ub = u[b];
    double s = 0.0;
    for (int i = 0; i < n; ++i) s += ((double)F[(int64_t)i * D + a] - ua) * ((double)F[(int64_t)i * D + b] - ub);
    S[(int64_t)a * D + b] = s / (double)n;
}

// One block. Adds ridge * trace / D to the diagonal, then factorises the lower triangle in place.
// flag: 1 = the set has no variance (rho is 0 everywhere), 2 = not positive definite.
__global__ void __launch_bounds__(1024) dgc_chol_kernel(double* __restrict__ S, int D, double ridge, int* __restrict__ flag)
{
    __shared__ double tr_sh;
    __shared__ int bad;
    if (threadIdx.x == 0) {
        double tr = 0.0;
        for (int a = 0; a < D; ++a) tr += S[(int64_t)a * D + a];
        tr_sh = tr;
        bad = tr > 0.0 ? 0 : 1;
    }
    __syncthreads();
    if (bad) {
        if (threadIdx.x == 0) *flag = 1;
        return;
    }
    for (int a = threadIdx.x; a < D; a += blockDim.x) S[(int64_t)a * D + a] += ridge * tr_sh / (double)D;
    __syncthreads();
    for (int k = 0; k < D; ++k) {
        if (threadIdx.x == 0) {
            const double dkk = S[(int64_t)k * D + k];
            if (!(dkk > 0.0)) bad = 2;
            else S[(int64_t)k * D + k] = sqrt(dkk);
        }
        __syncthreads();
        if (bad) {
            if (threadIdx.x == 0) *flag = 2;
            return;
        }
        const double lkk = S[(int64_t)k * D + k];
        for (int a = k + 1 + threadIdx.x; a < D; a += blockDim.x) S[(int64_t)a * D + k] /= lkk;
        __syncthreads();
        // trailing update of the lower triangle: S[a][b] -= L[a][k] L[b][k], k < b <= a
        const int m = D - k - 1;
        for (int64_t t = threadIdx.x; t < (int64_t)m * m; t += blockDim.x) {
            const int a = k + 1 + (int)(t / m), b = k + 1 + (int)(t % m);
            if (b <= a) S[(int64_t)a * D + b] -= S[(int64_t)a * D + k] * S[(int64_t)b * D + k];
        }
        __syncthreads();
    }
}

// One warp per sample; y lives in shared memory (D doubles per warp).
__global__ void __launch_bounds__(128) dgc_rho_kernel(const float* __restrict__ F, int n, int D, const double* __restrict__ u,
                                                      const double* __restrict__ L, const int* __restrict__ flag,
                                                      double* __restrict__ rho)
{
    extern __shared__ double ysh[];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int i = blockIdx.x * 4 + w;
    if (i >= n) return;
    if (*flag != 0) {
        if (lane == 0) rho[i] = 0.0;
        return;
    }
    double* y = ysh + (size_t)w * D;
    double r2 = 0.0;
    for (int a = 0; a < D; ++a) {
        double part = 0.0;
        for (int b = lane; b < a; b += 32) part += L[(int64_t)a * D + b] * y[b];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        const double v = ((double)F[(int64_t)i * D + a] - u[a] - part) / L[(int64_t)a * D + a];
        if (lane == 0) y[a] = v;
        __syncwarp();
        r2 += v * v;
    }
    if (lane == 0) rho[i] = sqrt(r2);
}

__global__ void dgc_rank_kernel(const double* __restrict__ rho, int n, int k, int32_t* __restrict__ selected)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const double ri = rho[i];
    int before = 0;
    for (int j = 0; j < n; ++j) {
        const double rj = rho[j];
        if (rj > ri || (rj == ri && j < i)) ++before;
    }
    if (before < k) selected[before] = i;
}

}  // namespace

size_t stwq_dgc_ws_bytes(int D) { return ((size_t)D * D + (size_t)D + 32) * sizeof(double); }

int stwq_launch_dgc(stwq_ctx* ctx, void* ws, const float* F, int n, int D, int k, double ridge, double* rho,
                    int32_t* selected, cudaStream_t st)
{
    double* S = static_cast<double*>(ws);
    double* u = S + (size_t)D * D;
    int* flag = reinterpret_cast<int*>(u + D);
    cudaError_t e = cudaMemsetAsync(flag, 0, sizeof(int), st);
    if (e != cudaSuccess) return stwq_cuda_fail(ctx, e);
    dgc_mean_kernel<<<(D + 127) / 128, 128, 0, st>>>(F, n, D, u);
    dgc_cov_kernel<<<dim3((D + 127) / 128, D), 128, 0, st>>>(F, n, D, u, S);
    dgc_chol_kernel<<<1, 1024, 0, st>>>(S, D, ridge, flag);
    dgc_rho_kernel<<<(n + 3) / 4, 128, (size_t)4 * D * sizeof(double), st>>>(F, n, D, u, S, flag, rho);
    if (selected != nullptr) dgc_rank_kernel<<<(n + 127) / 128, 128, 0, st>>>(rho, n, k, selected);
    ctx->launches += selected != nullptr ? 5 : 4;
    e = cudaGetLastError();
    return e == cudaSuccess ? STWQ_OK : stwq_cuda_fail(ctx, e);
}

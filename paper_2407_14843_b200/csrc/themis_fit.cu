// Least-squares fit of the paper's latency profile (Eq. 1)
//     l(b, c) = gamma * b / c + epsilon / c + delta * b + eta
// to measured (batch size, cores, latency) samples, one model per warp, and the
// latency table the solver consumes, evaluated from the fitted coefficients.
// Normal equations in double precision: 4 x 4, accumulated with a warp reduction,
// solved by Gaussian elimination with partial pivoting.
#include "themis_internal.h"

namespace themis {
namespace {

constexpr int kFitThreads = 128;     // 4 models per block

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

__global__ void __launch_bounds__(kFitThreads)
fit_profiles_kernel(int n_models, int n_samples, const int32_t *sample_b, const int32_t *sample_c,
                    const double *latency_ms, int c_max, int n_batch, const int32_t *batch_sizes,
                    double *coeffs, int32_t *lat_us, int32_t *status)
{
    const int lane = threadIdx.x & 31;
    const int m = blockIdx.x * (kFitThreads / 32) + (threadIdx.x >> 5);
    if (m >= n_models) return;
    // A = X^T X (upper triangle, 10 entries), y = X^T l with rows x = (b/c, 1/c, b, 1)
    double a[10], y[4];
#pragma unroll
    for (int i = 0; i < 10; ++i) a[i] = 0.0;
#pragma unroll
    for (int i = 0; i < 4; ++i) y[i] = 0.0;
    const double *lm = latency_ms + (size_t)m * n_samples;
    for (int i = lane; i < n_samples; i += 32) {
        const double b = (double)sample_b[i], c = (double)sample_c[i];
        const double x[4] = {b / c, 1.0 / c, b, 1.0};
        const double l = lm[i];
        int k = 0;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            y[r] += x[r] * l;
#pragma unroll
            for (int q = r; q < 4; ++q) a[k++] += x[r] * x[q];
        }
    }
#pragma unroll
    for (int i = 0; i < 10; ++i) a[i] = warp_sum(a[i]);
#pragma unroll
    for (int i = 0; i < 4; ++i) y[i] = warp_sum(y[i]);

    // every lane solves the same 4 x 4 system (augmented matrix M | y)
    double M[4][5];
    {
        int k = 0;
        for (int r = 0; r < 4; ++r)
            for (int q = r; q < 4; ++q) { M[r][q] = a[k]; M[q][r] = a[k]; ++k; }
        for (int r = 0; r < 4; ++r) M[r][4] = y[r];
    }
    bool singular = false;
    for (int col = 0; col < 4; ++col) {
        int piv = col;
        for (int r = col + 1; r < 4; ++r)
            if (fabs(M[r][col]) > fabs(M[piv][col])) piv = r;
        if (fabs(M[piv][col]) < 1e-300) { singular = true; break; }
        if (piv != col)
            for (int q = 0; q < 5; ++q) { const double t = M[col][q]; M[col][q] = M[piv][q]; M[piv][q] = t; }
        for (int r = col + 1; r < 4; ++r) {
            const double f = M[r][col] / M[col][col];
            for (int q = col; q < 5; ++q) M[r][q] -= f * M[col][q];
        }
    }
    double beta[4] = {0.0, 0.0, 0.0, 0.0};
    if (!singular) {
        for (int r = 3; r >= 0; --r) {
            double v = M[r][4];
            for (int q = r + 1; q < 4; ++q) v -= M[r][q] * beta[q];
            beta[r] = v / M[r][r];
        }
    }
    if (lane < 4) coeffs[(size_t)m * 4 + lane] = beta[lane];
    if (lane == 0) status[m] = singular ? THEMIS_STATUS_BAD_INPUT : THEMIS_STATUS_OK;
    // latency table [c_max][n_batch] in microseconds, rounded up, at least 1
    int32_t *tab = lat_us + (size_t)m * c_max * n_batch;
    for (int e = lane; e < c_max * n_batch; e += 32) {
        const double c = (double)(e / n_batch + 1), b = (double)batch_sizes[e % n_batch];
        const double l_ms = beta[0] * b / c + beta[1] / c + beta[2] * b + beta[3];
        const double us = ceil(l_ms * 1000.0);
        tab[e] = singular ? 0 : (int32_t)fmin(fmax(us, 1.0), 2147483647.0);
    }
}

}  // namespace

cudaError_t launch_fit_profiles(int n_models, int n_samples, const int32_t *sample_b, const int32_t *sample_c,
                                const double *latency_ms, int c_max, int n_batch, const int32_t *d_batch_sizes,
                                double *coeffs, int32_t *lat_us, int32_t *status, cudaStream_t st)
{
    const int per_block = kFitThreads / 32;
    fit_profiles_kernel<<<(n_models + per_block - 1) / per_block, kFitThreads, 0, st>>>(
        n_models, n_samples, sample_b, sample_c, latency_ms, c_max, n_batch, d_batch_sizes, coeffs, lat_us, status);
    return cudaGetLastError();
}

}  // namespace themis

// Bookkeeping kernels of Algorithm 1's last branch (no configuration serves the
// whole load): per-instance bisection on the arrival rate over search points
// k * resolution, then extra replicas for the rest of the load.  One thread per
// instance; the solves between these steps are the ordinary vertical solver.
#include "themis_internal.h"

namespace themis {
namespace {

constexpr int kThreads = 256;

// After the solve at the full rate: instances without a configuration start a
// search with lo = 0 (nothing served), hi = ceil(lambda / resolution) (not served).
__global__ void fb_init_kernel(int N, uint32_t res, const int32_t *status, const uint32_t *lambda,
                               uint32_t *lo, uint32_t *hi, int32_t *active)
{
    const int n = blockIdx.x * kThreads + threadIdx.x;
    if (n >= N) return;
    const bool search = status[n] == THEMIS_STATUS_INFEASIBLE;
    lo[n] = 0;
    hi[n] = search ? (uint32_t)(((unsigned long long)lambda[n] + res - 1) / res) : 0u;
    active[n] = search ? 1 : 0;
}

// Next trial rate of every instance whose interval is still open.
__global__ void fb_trial_kernel(int N, uint32_t res, const uint32_t *lo, const uint32_t *hi,
                                const int32_t *active, int32_t *iter_active, uint32_t *trial_lambda)
{
    const int n = blockIdx.x * kThreads + threadIdx.x;
    if (n >= N) return;
    const bool open = active[n] && hi[n] - lo[n] > 1u;
    iter_active[n] = open ? 1 : 0;
    trial_lambda[n] = open ? (lo[n] + (hi[n] - lo[n]) / 2u) * res : res;
}

__global__ void fb_update_kernel(int N, uint32_t *lo, uint32_t *hi, const int32_t *iter_active,
                                 const int32_t *trial_status)
{
    const int n = blockIdx.x * kThreads + threadIdx.x;
    if (n >= N || !iter_active[n]) return;
    const uint32_t mid = lo[n] + (hi[n] - lo[n]) / 2u;
    if (trial_status[n] == THEMIS_STATUS_OK) lo[n] = mid; else hi[n] = mid;
}

// The rate the final vertical solve runs at, and who takes part in it.
__global__ void fb_final_trial_kernel(int N, uint32_t res, const uint32_t *lo, const int32_t *active,
                                      int32_t *iter_active, uint32_t *trial_lambda)
{
    const int n = blockIdx.x * kThreads + threadIdx.x;
    if (n >= N) return;
    const bool go = active[n] && lo[n] > 0u;
    iter_active[n] = go ? 1 : 0;
    trial_lambda[n] = go ? lo[n] * res : res;
}

// lambda_vertical, extra replicas and the final status.
__global__ void fb_finish_kernel(const Params p, uint32_t res, const uint32_t *lo, const uint32_t *hi,
                                 const int32_t *active, uint32_t *lambda_vertical, int32_t *extra)
{
    const int n = blockIdx.x * kThreads + threadIdx.x;
    const int N = p.prob.n_instances, S = p.prob.n_stages;
    if (n >= N) return;
    int32_t *e = extra + (size_t)n * S;
    for (int s = 0; s < S; ++s) e[s] = 0;
    const uint32_t lam = p.lambda_mrps[n];
    if (!active[n]) { lambda_vertical[n] = lam; return; }
    if (hi[n] - lo[n] > 1u) {              // the caller's bound on lambda was too low for this one
        lambda_vertical[n] = 0;
        p.out.status[n] = THEMIS_STATUS_BAD_INPUT;
        return;
    }
    if (lo[n] == 0u) { lambda_vertical[n] = 0; return; }      // stays THEMIS_STATUS_INFEASIBLE
    const uint32_t lv = lo[n] * res;
    lambda_vertical[n] = lv;
    if (p.out.status[n] != THEMIS_STATUS_OK) return;          // device-side error of the last solve
    p.out.status[n] = THEMIS_STATUS_SPLIT;
    const unsigned long long rest = (unsigned long long)lam - lv;
    const int pid = p.profile_id ? p.profile_id[n] : 0;
    const int C = p.prob.c_max, NB = p.prob.n_batch;
    const int32_t *lat = p.lat_us + (size_t)pid * S * C * NB;
    for (int s = 0; s < S; ++s) {
        const int c = p.out.c[(size_t)n * S + s], b = p.out.b[(size_t)n * S + s];
        int bi = 0;
        while (bi < NB - 1 && p.prob.batch_sizes[bi] != b) ++bi;
        const unsigned long long l_us = (unsigned long long)lat[((size_t)s * C + (c - 1)) * NB + bi];
        const unsigned long long per = (unsigned long long)b * 1000000000ull;
        e[s] = (int32_t)((rest * l_us + per - 1ull) / per);
    }
}

// stable[n] = 1 iff both solves succeeded and chose the same (h, c, b) at every stage.
__global__ void configs_equal_kernel(int N, int S, themis_result_t a, themis_result_t b, int32_t *stable)
{
    const int n = blockIdx.x * kThreads + threadIdx.x;
    if (n >= N) return;
    int same = a.status[n] == THEMIS_STATUS_OK && b.status[n] == THEMIS_STATUS_OK;
    for (int s = 0; s < S && same; ++s) {
        const size_t i = (size_t)n * S + s;
        same = a.h[i] == b.h[i] && a.c[i] == b.c[i] && a.b[i] == b.b[i];
    }
    stable[n] = same;
}

}  // namespace

cudaError_t launch_configs_equal(int N, int S, themis_result_t a, themis_result_t b, int32_t *stable, cudaStream_t st)
{
    configs_equal_kernel<<<(N + kThreads - 1) / kThreads, kThreads, 0, st>>>(N, S, a, b, stable);
    return cudaGetLastError();
}

cudaError_t launch_fb_init(int N, uint32_t res, const int32_t *status, const uint32_t *lambda, uint32_t *lo,
                           uint32_t *hi, int32_t *active, cudaStream_t st)
{
    fb_init_kernel<<<(N + kThreads - 1) / kThreads, kThreads, 0, st>>>(N, res, status, lambda, lo, hi, active);
    return cudaGetLastError();
}

cudaError_t launch_fb_trial(int N, uint32_t res, const uint32_t *lo, const uint32_t *hi, const int32_t *active,
                            int32_t *iter_active, uint32_t *trial_lambda, cudaStream_t st)
{
    fb_trial_kernel<<<(N + kThreads - 1) / kThreads, kThreads, 0, st>>>(N, res, lo, hi, active, iter_active,
                                                                        trial_lambda);
    return cudaGetLastError();
}

cudaError_t launch_fb_update(int N, uint32_t *lo, uint32_t *hi, const int32_t *iter_active,
                             const int32_t *trial_status, cudaStream_t st)
{
    fb_update_kernel<<<(N + kThreads - 1) / kThreads, kThreads, 0, st>>>(N, lo, hi, iter_active, trial_status);
    return cudaGetLastError();
}

cudaError_t launch_fb_final_trial(int N, uint32_t res, const uint32_t *lo, const int32_t *active,
                                  int32_t *iter_active, uint32_t *trial_lambda, cudaStream_t st)
{
    fb_final_trial_kernel<<<(N + kThreads - 1) / kThreads, kThreads, 0, st>>>(N, res, lo, active, iter_active,
                                                                              trial_lambda);
    return cudaGetLastError();
}

cudaError_t launch_fb_finish(const Params &p, uint32_t res, const uint32_t *lo, const uint32_t *hi,
                             const int32_t *active, uint32_t *lambda_vertical, int32_t *extra, cudaStream_t st)
{
    const int N = p.prob.n_instances;
    fb_finish_kernel<<<(N + kThreads - 1) / kThreads, kThreads, 0, st>>>(p, res, lo, hi, active, lambda_vertical,
                                                                         extra);
    return cudaGetLastError();
}

}  // namespace themis

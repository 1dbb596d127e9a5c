// Algorithm 1's last branch (no configuration serves the whole load): per-instance
// bisection on the arrival rate over search points k * resolution, then extra replicas
// for the rest of the load.  A search point only has to be classified as served or not,
// and the replicas in place serve a rate exactly when the fastest feasible candidates of
// all stages fit the budget together (the recurrence finds a configuration iff one
// exists), so the whole search of an instance runs in one block of one kernel without
// the recurrence; the solves before and after it are the ordinary vertical solver.
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

// The bisection of one instance (one block): `rounds` halvings of [lo, hi), each deciding
// whether the rate mid * res is served.  Per trial rate the block fills, per (stage, batch size),
//   Q    = ceil((b-1) * m * 1e9 / (lambda * w)),  m = replicas or 1     (Eq. 4 in buckets)
//   Lmax = floor(replicas * b * 1e9 / lambda)                            (Eq. 6)
// and takes per stage the smallest ceil(l / w) + Q over the pairs (c, b) with l <= Lmax.
__global__ void __launch_bounds__(128)
fb_bisect_kernel(const Params p, int rounds, uint32_t res, const int32_t *active, uint32_t *lo_out, uint32_t *hi_out)
{
    __shared__ uint32_t q_tab[THEMIS_MAX_STAGES * THEMIS_MAX_BATCH_SIZES];
    __shared__ uint32_t lmax_tab[THEMIS_MAX_STAGES * THEMIS_MAX_BATCH_SIZES];
    __shared__ uint32_t stage_min[THEMIS_MAX_STAGES];
    const int n = blockIdx.x;
    if (!active[n]) return;
    const int tid = threadIdx.x;
    const int S = p.prob.n_stages, C = p.prob.c_max, NB = p.prob.n_batch, T = p.T;
    const int CB = C * NB;
    const uint32_t w_us = (uint32_t)p.prob.bucket_us;
    const int pid = p.profile_id ? p.profile_id[n] : 0;
    const int32_t *lat = p.lat_us + (size_t)pid * S * CB;
    const int32_t *rep = p.replicas + (size_t)n * S;
    uint32_t lo = lo_out[n], hi = hi_out[n];
    for (int r = 0; r < rounds && hi - lo > 1u; ++r) {      // lo, hi are block-uniform
        const uint32_t mid = lo + (hi - lo) / 2u;
        const unsigned long long lambda_m = (unsigned long long)mid * res;
        for (int e = tid; e < S * NB; e += blockDim.x) {
            const int s = e / NB, bi = e - s * NB;
            const unsigned long long h = (unsigned long long)rep[s], b = (unsigned long long)p.prob.batch_sizes[bi];
            const unsigned long long m = (p.prob.flags & THEMIS_QUEUE_PER_REPLICA) ? h : 1ull;
            const unsigned long long q_den = lambda_m * w_us;
            const unsigned long long q = ((b - 1ull) * m * 1000000000ull + q_den - 1ull) / q_den;
            const unsigned long long lm = h * b * 1000000000ull / lambda_m;
            q_tab[e] = q > (unsigned long long)T ? (uint32_t)T + 1u : (uint32_t)q;
            lmax_tab[e] = lm > 0x7FFFFFFFull ? 0x7FFFFFFFu : (uint32_t)lm;
        }
        if (tid < S) stage_min[tid] = 0xFFFFFFFFu;
        __syncthreads();
        for (int s = 0; s < S; ++s) {
            uint32_t best = 0xFFFFFFFFu;
            for (int pair = tid; pair < CB; pair += blockDim.x) {
                const int bi = pair % NB;
                const uint32_t l_us = (uint32_t)lat[(size_t)s * CB + pair];
                if (l_us <= lmax_tab[s * NB + bi]) best = min(best, (l_us + w_us - 1u) / w_us + q_tab[s * NB + bi]);
            }
            best = __reduce_min_sync(0xFFFFFFFFu, best);
            if ((tid & 31) == 0 && best != 0xFFFFFFFFu) atomicMin(&stage_min[s], best);
        }
        __syncthreads();
        unsigned long long fastest = 0;
        for (int s = 0; s < S; ++s) fastest += stage_min[s] == 0xFFFFFFFFu ? (unsigned long long)T + 1ull : stage_min[s];
        if (fastest <= (unsigned long long)T) lo = mid; else hi = mid;
        __syncthreads();                                     // stage_min is rewritten next round
    }
    if (tid == 0) { lo_out[n] = lo; hi_out[n] = hi; }
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

cudaError_t launch_fb_bisect(const Params &p, int rounds, uint32_t res, const int32_t *active, uint32_t *lo,
                             uint32_t *hi, cudaStream_t st)
{
    fb_bisect_kernel<<<p.prob.n_instances, 128, 0, st>>>(p, rounds, res, active, lo, hi);
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

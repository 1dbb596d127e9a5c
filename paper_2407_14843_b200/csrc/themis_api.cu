// C ABI of libthemis: argument validation, workspace carving, kernel launches.
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "themis_internal.h"
#include "themis_probe.h"

namespace themis {
namespace {

thread_local cudaError_t t_last_cuda = cudaSuccess;
thread_local char t_msg[256];
// Which problem a launch solves and for which instances.
enum Mode { kJoint = 0, kVertical = 1, kHorizontal = 2 };
struct SolveOpts {
    Mode mode = kJoint;
    const int32_t *active = nullptr;   // [N] device mask, or nullptr: every instance
};

// Kernel choice and tile of a call, from the flags of its problem description.
inline uint32_t kernel_of(const themis_problem_t *pr)
{
    const uint32_t k = pr->flags & THEMIS_KERNEL_MASK;
    return k == THEMIS_KERNEL_DEFAULT ? THEMIS_KERNEL_PACKED16 : k;
}
inline int tile_of(const themis_problem_t *pr)
{
    switch (pr->flags & THEMIS_TILE_MASK) {
        case THEMIS_TILE_4: return 4;
        case THEMIS_TILE_8: return 8;
        case THEMIS_TILE_16: return 16;
        default: return 0;
    }
}

constexpr size_t kAlign = 256;
inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

int fail_cuda(cudaError_t e)
{
    t_last_cuda = e;
    return THEMIS_E_CUDA;
}

// Host-side validation of the scalar description.  Fills T, K.
int validate(const themis_problem_t *pr, int vertical, int32_t *T_out, int32_t *K_out)
{
    if (!pr) return THEMIS_E_INVALID_ARG;
    if (pr->n_instances < 1 || pr->n_stages < 1 || pr->n_profiles < 1 || pr->c_max < 1 || pr->n_batch < 1)
        return THEMIS_E_INVALID_ARG;
    if (pr->slo_us < 1 || pr->bucket_us < 1) return THEMIS_E_INVALID_ARG;
    if (pr->flags & ~(THEMIS_QUEUE_PER_REPLICA | THEMIS_KERNEL_MASK | THEMIS_TILE_MASK)) return THEMIS_E_INVALID_ARG;
    if ((pr->flags & THEMIS_KERNEL_MASK) > THEMIS_KERNEL_PACKED16_BLOCK) return THEMIS_E_INVALID_ARG;
    if (!vertical && pr->h_max < 1) return THEMIS_E_INVALID_ARG;
    if (pr->n_batch > THEMIS_MAX_BATCH_SIZES) return THEMIS_E_UNSUPPORTED_SIZE;
    for (int i = 0; i < pr->n_batch; ++i) {
        if (pr->batch_sizes[i] < 1 || pr->batch_sizes[i] > 65536) return THEMIS_E_INVALID_ARG;
        if (i > 0 && pr->batch_sizes[i] <= pr->batch_sizes[i - 1]) return THEMIS_E_INVALID_ARG;
    }
    if (pr->n_stages > THEMIS_MAX_STAGES) return THEMIS_E_UNSUPPORTED_SIZE;
    const int64_t T = pr->slo_us / pr->bucket_us;
    if (T < 1) return THEMIS_E_INVALID_ARG;
    if (T > THEMIS_MAX_T) return THEMIS_E_UNSUPPORTED_SIZE;
    const int64_t h = vertical ? 1 : pr->h_max;
    const int64_t K = h * pr->c_max * pr->n_batch;
    if (K > THEMIS_MAX_CANDIDATES) return THEMIS_E_UNSUPPORTED_SIZE;
    // joint: the largest possible total must stay below the "unreachable" cost;
    // vertical: the same bound is checked on the device against replicas[].
    if (!vertical && (int64_t)pr->n_stages * pr->h_max * pr->c_max > THEMIS_MAX_TOTAL_COST)
        return THEMIS_E_UNSUPPORTED_SIZE;
    if (vertical && (int64_t)pr->n_stages * pr->c_max > THEMIS_MAX_TOTAL_COST) return THEMIS_E_UNSUPPORTED_SIZE;
    // shared-memory tables of the scoring kernel: n_batch * h entries, two tables
    if ((int64_t)pr->n_batch * h > 8192) return THEMIS_E_UNSUPPORTED_SIZE;
    *T_out = (int32_t)T;
    *K_out = (int32_t)K;
    return THEMIS_OK;
}

inline size_t list_words_of(const themis_problem_t *pr)
{
    return (size_t)score_list_layout(pr->c_max, pr->n_batch).words;
}

int layout_of(const themis_problem_t *pr, int vertical, themis_workspace_layout_t *L)
{
    int32_t T, K;
    int rc = validate(pr, vertical, &T, &K);
    if (rc != THEMIS_OK) return rc;
    const size_t pitch = (size_t)(T + 1 + kRowAlign - 1) / kRowAlign * kRowAlign;
    const size_t rows = (size_t)pr->n_instances * pr->n_stages;
    size_t off = 0;
    L->g_offset = off;    off = align_up(off + rows * pitch * sizeof(int32_t));
    L->garg_offset = off; off = align_up(off + rows * pitch * sizeof(uint16_t));
    L->a_offset = off;    off = align_up(off + rows * pitch * sizeof(uint16_t));
    L->f_offset = off;    off = align_up(off + (size_t)pr->n_instances * pitch * sizeof(int32_t));
    L->flag_offset = off; off = align_up(off + (size_t)pr->n_instances * sizeof(int32_t));
    // behind the tables: instances the sparse warp kernel hands to the block kernel (count, then ids)
    off = align_up(off + ((size_t)pr->n_instances + 1) * sizeof(int32_t));
    // candidate lists of the scoring kernels: per (profile, stage) a header and one uint4 per (cores, batch size)
    off = align_up(off + (size_t)pr->n_profiles * pr->n_stages * list_words_of(pr) * sizeof(uint32_t));
    // record of the bounds-checked build (four words)
    off = align_up(off + 4 * sizeof(int32_t));
    L->total_bytes = off;
    L->row_pitch = (int32_t)pitch;
    L->T = T;
    return THEMIS_OK;
}

int make_params(const themis_problem_t *pr, const SolveOpts &opts, void *ws, size_t ws_bytes, Params *P)
{
    const int vertical = opts.mode == kVertical;
    themis_workspace_layout_t L;
    int rc = layout_of(pr, vertical, &L);
    if (rc != THEMIS_OK) return rc;
    if (!ws || ((uintptr_t)ws & (kAlign - 1))) return THEMIS_E_INVALID_ARG;
    if (ws_bytes < L.total_bytes) return THEMIS_E_WORKSPACE_TOO_SMALL;
    memset(P, 0, sizeof(*P));
    P->prob = *pr;
    P->T = L.T;
    P->pitch = L.row_pitch;
    P->vertical = vertical ? 1 : 0;
    P->horizontal = opts.mode == kHorizontal ? 1 : 0;
    P->active = opts.active;
    char *base = static_cast<char *>(ws);
    P->G = reinterpret_cast<int32_t *>(base + L.g_offset);
    P->Garg = reinterpret_cast<uint16_t *>(base + L.garg_offset);
    P->A = reinterpret_cast<uint16_t *>(base + L.a_offset);
    P->F = reinterpret_cast<int32_t *>(base + L.f_offset);
    P->inst_flag = reinterpret_cast<int32_t *>(base + L.flag_offset);
    P->redo_count = reinterpret_cast<int32_t *>(base + align_up(L.flag_offset + (size_t)pr->n_instances * sizeof(int32_t)));
    P->redo_list = P->redo_count + 1;
    P->check = reinterpret_cast<int32_t *>(base + L.total_bytes - kAlign);
    P->lists = reinterpret_cast<uint32_t *>(base + L.total_bytes - kAlign -
                                            align_up((size_t)pr->n_profiles * pr->n_stages * list_words_of(pr) * sizeof(uint32_t)));
    return THEMIS_OK;
}

// Bounds-checked build: clears the violation record at the start of a solve.
cudaError_t reset_check(const Params &P, cudaStream_t st)
{
    return kBoundsChecked ? cudaMemsetAsync(P.check, 0, 4 * sizeof(int32_t), st) : cudaSuccess;
}

bool result_ok(const themis_result_t &o)
{
    return o.h && o.c && o.b && o.total_cost && o.latency_buckets && o.status;
}

int score_impl(const themis_problem_t *pr, const int32_t *lat, const int32_t *pid, const uint32_t *lam,
               const int32_t *rep, const SolveOpts &opts, void *ws, size_t ws_bytes, cudaStream_t st)
{
    const int vertical = opts.mode == kVertical;
    Params P;
    int rc = make_params(pr, opts, ws, ws_bytes, &P);
    if (rc != THEMIS_OK) return rc;
    if (!lat || !lam || (vertical && !rep)) return THEMIS_E_INVALID_ARG;
    P.lat_us = lat; P.profile_id = pid; P.lambda_mrps = lam; P.replicas = rep;
    cudaError_t e = reset_check(P, st);
    if (e == cudaSuccess) e = launch_score(P, st);
    return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
}

int minplus_impl(const themis_problem_t *pr, const int32_t *rep, const SolveOpts &opts, themis_result_t out,
                 void *ws, size_t ws_bytes, cudaStream_t st)
{
    const int vertical = opts.mode == kVertical;
    Params P;
    int rc = make_params(pr, opts, ws, ws_bytes, &P);
    if (rc != THEMIS_OK) return rc;
    if (!result_ok(out) || (vertical && !rep)) return THEMIS_E_INVALID_ARG;
    P.replicas = rep; P.out = out;
    cudaError_t e;
    const uint32_t kernel = kernel_of(pr);
    const int tile = tile_of(pr);
    if (kernel == THEMIS_KERNEL_WIDE32) {
        e = launch_minplus(P, tile, st);
    } else if (kernel >= THEMIS_KERNEL_PRUNED && kernel != THEMIS_KERNEL_PACKED16_BLOCK &&
               pruned_smem_bytes(P.pitch) <= kMaxDynamicSmem) {
        e = launch_minplus_pruned(P, st);
    } else {
        // short budgets: a warp per instance, unless the block kernel is asked for
        e = kernel != THEMIS_KERNEL_PACKED16_BLOCK && minplus16_warp_fits(P, tile) ? launch_minplus16_warp(P, tile, st)
                                                                                  : launch_minplus16(P, tile, st);
        // A total can only reach the 16-bit saturation value if the static bound allows it
        // (vertical: the bound depends on replicas[], which lives on the device).
        const bool may_saturate =
            vertical || (int64_t)pr->n_stages * pr->h_max * pr->c_max >= (int64_t)kInf16;
        if (e == cudaSuccess && may_saturate) {
            P.only_flagged = 1;
            e = launch_minplus(P, tile, st);
        }
    }
    return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
}

int solve_impl(const themis_problem_t *pr, const int32_t *lat, const int32_t *pid, const uint32_t *lam,
               const int32_t *rep, const SolveOpts &opts, themis_result_t out, void *ws, size_t ws_bytes,
               cudaStream_t st)
{
    const int vertical = opts.mode == kVertical;
    int32_t T, K;
    int rc = validate(pr, vertical, &T, &K);
    if (rc != THEMIS_OK) return rc;
    if (!result_ok(out)) return THEMIS_E_INVALID_ARG;
    const uint32_t kernel = kernel_of(pr);
    if (kernel == THEMIS_KERNEL_SPARSE || kernel == THEMIS_KERNEL_SPARSE_BLOCK) {
        // one kernel on undominated entries, when its shared memory fits
        Params P;
        rc = make_params(pr, opts, ws, ws_bytes, &P);
        if (rc != THEMIS_OK) return rc;
        if (!lat || !lam || (vertical && !rep)) return THEMIS_E_INVALID_ARG;
        P.lat_us = lat; P.profile_id = pid; P.lambda_mrps = lam; P.replicas = rep; P.out = out;
        const bool block_fits = sparse_smem_bytes(P) <= kMaxDynamicSmem;
        if (kernel == THEMIS_KERNEL_SPARSE && block_fits && front_kernel_fits(P)) {
            // one warp per instance on short sorted lists; what outgrows them is listed and
            // redone by the block kernel
            cudaError_t e = cudaMemsetAsync(P.redo_count, 0, sizeof(int32_t), st);
            if (e == cudaSuccess) e = reset_check(P, st);
            if (e == cudaSuccess) e = launch_solve_front(P, st);
            if (e == cudaSuccess) e = launch_solve_sparse(P, /*only_listed=*/true, st);
            return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
        }
        if (block_fits) {
            cudaError_t e = reset_check(P, st);
            if (e == cudaSuccess) e = launch_solve_sparse(P, /*only_listed=*/false, st);
            return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
        }
    }
    rc = score_impl(pr, lat, pid, lam, rep, opts, ws, ws_bytes, st);
    if (rc == THEMIS_OK) rc = minplus_impl(pr, rep, opts, out, ws, ws_bytes, st);
    return rc;
}

// Search state appended to the solver workspace by the fallback entry point (the result-shaped
// arrays behind it are reserved).
struct FallbackStage {
    size_t lo, hi, active, iter_active, trial_lambda, h, c, b, cost, latb, status, total;
};

void fallback_stage_of(const themis_problem_t *pr, size_t base, FallbackStage *F)
{
    const size_t N = pr->n_instances, S = pr->n_stages;
    size_t off = align_up(base);
    F->lo = off; off = align_up(off + N * 4);
    F->hi = off; off = align_up(off + N * 4);
    F->active = off; off = align_up(off + N * 4);
    F->iter_active = off; off = align_up(off + N * 4);
    F->trial_lambda = off; off = align_up(off + N * 4);
    F->h = off; off = align_up(off + N * S * 4);
    F->c = off; off = align_up(off + N * S * 4);
    F->b = off; off = align_up(off + N * S * 4);
    F->cost = off; off = align_up(off + N * 4);
    F->latb = off; off = align_up(off + N * 4);
    F->status = off; off = align_up(off + N * 4);
    F->total = off;
}

// Staging area appended to the solver workspace by the host-buffer variant.
struct HostStage {
    size_t lat, pid, lam, rep, h, c, b, cost, latb, status, total;
};

int host_stage_of(const themis_problem_t *pr, int vertical, size_t base, HostStage *H)
{
    const size_t N = pr->n_instances, S = pr->n_stages;
    size_t off = align_up(base);
    H->lat = off; off = align_up(off + (size_t)pr->n_profiles * S * pr->c_max * pr->n_batch * 4);
    H->pid = off; off = align_up(off + N * 4);
    H->lam = off; off = align_up(off + N * 4);
    H->rep = off; off = align_up(off + (vertical ? N * S * 4 : 0));
    H->h = off; off = align_up(off + N * S * 4);
    H->c = off; off = align_up(off + N * S * 4);
    H->b = off; off = align_up(off + N * S * 4);
    H->cost = off; off = align_up(off + N * 4);
    H->latb = off; off = align_up(off + N * 4);
    H->status = off; off = align_up(off + N * 4);
    H->total = off;
    return THEMIS_OK;
}

// Scratch of themis_solve_batch_static: lives in the library image, one copy per
// device that loads it.  In host code this name is only a handle for
// cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[THEMIS_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_ptr[kMaxDevices];   // device address of g_static_scratch, per device ordinal

// Device address of the static scratch on the current device; looked up on the
// first call per device.
int static_scratch_ptr(void **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(e);
    if (dev < 0 || dev >= kMaxDevices) return THEMIS_E_UNSUPPORTED_SIZE;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return fail_cuda(e);
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return THEMIS_OK;
}

}  // namespace
}  // namespace themis

using namespace themis;

extern "C" {

int themis_version(void) { return THEMIS_VERSION; }

const char *themis_strerror(int code)
{
    switch (code) {
        case THEMIS_OK: return "ok";
        case THEMIS_E_INVALID_ARG: return "invalid argument";
        case THEMIS_E_UNSUPPORTED_SIZE: return "problem size outside the supported limits";
        case THEMIS_E_WORKSPACE_TOO_SMALL: return "workspace too small";
        case THEMIS_E_STATIC_SCRATCH_EXCEEDED:
            return "problem needs more scratch than the library's built-in 32 MiB buffer; "
                   "split the batch or use the workspace entry points";
        case THEMIS_E_CUDA:
            snprintf(t_msg, sizeof(t_msg), "CUDA error: %s", cudaGetErrorString(t_last_cuda));
            return t_msg;
        default: return "unknown error code";
    }
}

int themis_workspace_layout(const themis_problem_t *problem, int vertical, themis_workspace_layout_t *out_layout)
{
    if (!out_layout) return THEMIS_E_INVALID_ARG;
    return layout_of(problem, vertical, out_layout);
}

int themis_workspace_bytes(const themis_problem_t *problem, int vertical, size_t *out_bytes)
{
    if (!out_bytes) return THEMIS_E_INVALID_ARG;
    themis_workspace_layout_t L;
    int rc = layout_of(problem, vertical, &L);
    if (rc == THEMIS_OK) *out_bytes = L.total_bytes;
    return rc;
}

int themis_solve_batch(const themis_problem_t *problem, const int32_t *d_lat_us, const int32_t *d_profile_id,
                       const uint32_t *d_lambda_mrps, themis_result_t out, void *d_workspace,
                       size_t workspace_bytes, void *cuda_stream)
{
    return solve_impl(problem, d_lat_us, d_profile_id, d_lambda_mrps, nullptr, SolveOpts{kJoint}, out, d_workspace,
                      workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int themis_solve_vertical_batch(const themis_problem_t *problem, const int32_t *d_lat_us,
                                const int32_t *d_profile_id, const uint32_t *d_lambda_mrps,
                                const int32_t *d_replicas, themis_result_t out, void *d_workspace,
                                size_t workspace_bytes, void *cuda_stream)
{
    if (!d_replicas) return THEMIS_E_INVALID_ARG;
    return solve_impl(problem, d_lat_us, d_profile_id, d_lambda_mrps, d_replicas, SolveOpts{kVertical}, out, d_workspace,
                      workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int themis_fallback_workspace_bytes(const themis_problem_t *problem, size_t *out_bytes)
{
    if (!out_bytes) return THEMIS_E_INVALID_ARG;
    themis_workspace_layout_t L;
    int rc = layout_of(problem, 1, &L);
    if (rc != THEMIS_OK) return rc;
    FallbackStage F;
    fallback_stage_of(problem, L.total_bytes, &F);
    *out_bytes = F.total;
    return THEMIS_OK;
}

int themis_vertical_fallback_batch(const themis_problem_t *problem, const int32_t *d_lat_us,
                                   const int32_t *d_profile_id, const uint32_t *d_lambda_mrps,
                                   const int32_t *d_replicas, uint32_t resolution_mrps,
                                   uint32_t lambda_max_mrps, themis_result_t out,
                                   uint32_t *d_lambda_vertical, int32_t *d_extra_replicas,
                                   void *d_workspace, size_t workspace_bytes, void *cuda_stream)
{
    themis_workspace_layout_t L;
    int rc = layout_of(problem, 1, &L);
    if (rc != THEMIS_OK) return rc;
    if (!d_replicas || !d_lambda_vertical || !d_extra_replicas || !result_ok(out) || !d_lat_us || !d_lambda_mrps ||
        resolution_mrps < 1 || lambda_max_mrps < 1)
        return THEMIS_E_INVALID_ARG;
    if (!d_workspace || ((uintptr_t)d_workspace & (kAlign - 1))) return THEMIS_E_INVALID_ARG;
    FallbackStage F;
    fallback_stage_of(problem, L.total_bytes, &F);
    if (workspace_bytes < F.total) return THEMIS_E_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char *base = static_cast<char *>(d_workspace);
    const int N = problem->n_instances;
    uint32_t *lo = reinterpret_cast<uint32_t *>(base + F.lo), *hi = reinterpret_cast<uint32_t *>(base + F.hi);
    int32_t *active = reinterpret_cast<int32_t *>(base + F.active);
    int32_t *iter_active = reinterpret_cast<int32_t *>(base + F.iter_active);
    uint32_t *trial_lambda = reinterpret_cast<uint32_t *>(base + F.trial_lambda);

    // 1. the whole load on the replicas in place
    rc = solve_impl(problem, d_lat_us, d_profile_id, d_lambda_mrps, d_replicas, SolveOpts{kVertical}, out, d_workspace,
                    L.total_bytes, st);
    if (rc != THEMIS_OK) return rc;
    cudaError_t e = launch_fb_init(N, resolution_mrps, out.status, d_lambda_mrps, lo, hi, active, st);
    if (e != cudaSuccess) return fail_cuda(e);
    // 2. bisection: enough rounds to close an interval of ceil(max / resolution) points
    const unsigned long long points = ((unsigned long long)lambda_max_mrps + resolution_mrps - 1) / resolution_mrps;
    int rounds = 0;
    while ((1ull << rounds) < points) ++rounds;
    Params P;
    rc = make_params(problem, SolveOpts{kVertical}, d_workspace, L.total_bytes, &P);
    if (rc != THEMIS_OK) return rc;
    P.lat_us = d_lat_us; P.profile_id = d_profile_id; P.lambda_mrps = d_lambda_mrps; P.replicas = d_replicas;
    P.out = out;
    e = launch_fb_bisect(P, rounds, resolution_mrps, active, lo, hi, st);
    if (e != cudaSuccess) return fail_cuda(e);
    // 3. the vertical part at the rate found, straight into the caller's arrays
    e = launch_fb_final_trial(N, resolution_mrps, lo, active, iter_active, trial_lambda, st);
    if (e != cudaSuccess) return fail_cuda(e);
    rc = solve_impl(problem, d_lat_us, d_profile_id, trial_lambda, d_replicas, SolveOpts{kVertical, iter_active},
                    out, d_workspace, L.total_bytes, st);
    if (rc != THEMIS_OK) return rc;
    // 4. the rest of the load on extra replicas
    e = launch_fb_finish(P, resolution_mrps, lo, hi, active, d_lambda_vertical, d_extra_replicas, st);
    return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
}

int themis_solve_horizontal_batch(const themis_problem_t *problem, const int32_t *d_lat_us,
                                  const int32_t *d_profile_id, const uint32_t *d_lambda_mrps,
                                  themis_result_t out, void *d_workspace, size_t workspace_bytes,
                                  void *cuda_stream)
{
    if (problem && problem->c_max != 1) return THEMIS_E_INVALID_ARG;
    return solve_impl(problem, d_lat_us, d_profile_id, d_lambda_mrps, nullptr, SolveOpts{kHorizontal}, out, d_workspace,
                      workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int themis_configs_equal_batch(int32_t n_instances, int32_t n_stages, themis_result_t current,
                               themis_result_t predicted, int32_t *d_stable, void *cuda_stream)
{
    if (n_instances < 1 || n_stages < 1 || !d_stable || !current.h || !current.c || !current.b || !current.status ||
        !predicted.h || !predicted.c || !predicted.b || !predicted.status)
        return THEMIS_E_INVALID_ARG;
    cudaError_t e = launch_configs_equal(n_instances, n_stages, current, predicted, d_stable,
                                         static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
}

int themis_score_batch(const themis_problem_t *problem, const int32_t *d_lat_us, const int32_t *d_profile_id,
                       const uint32_t *d_lambda_mrps, const int32_t *d_replicas, void *d_workspace,
                       size_t workspace_bytes, void *cuda_stream)
{
    return score_impl(problem, d_lat_us, d_profile_id, d_lambda_mrps, d_replicas,
                      SolveOpts{d_replicas ? kVertical : kJoint},
                      d_workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int themis_minplus_batch(const themis_problem_t *problem, const int32_t *d_replicas, themis_result_t out,
                         void *d_workspace, size_t workspace_bytes, void *cuda_stream)
{
    return minplus_impl(problem, d_replicas, SolveOpts{d_replicas ? kVertical : kJoint}, out, d_workspace, workspace_bytes,
                        static_cast<cudaStream_t>(cuda_stream));
}

int themis_host_workspace_bytes(const themis_problem_t *problem, int vertical, size_t *out_bytes)
{
    if (!out_bytes) return THEMIS_E_INVALID_ARG;
    themis_workspace_layout_t L;
    int rc = layout_of(problem, vertical, &L);
    if (rc != THEMIS_OK) return rc;
    HostStage H;
    host_stage_of(problem, vertical, L.total_bytes, &H);
    *out_bytes = H.total;
    return THEMIS_OK;
}

int themis_solve_batch_host(const themis_problem_t *problem, const int32_t *h_lat_us, const int32_t *h_profile_id,
                            const uint32_t *h_lambda_mrps, const int32_t *h_replicas, themis_result_t h_out,
                            void *d_workspace, size_t workspace_bytes, void *cuda_stream)
{
    const int vertical = h_replicas != nullptr;
    themis_workspace_layout_t L;
    int rc = layout_of(problem, vertical, &L);
    if (rc != THEMIS_OK) return rc;
    if (!h_lat_us || !h_lambda_mrps || !result_ok(h_out)) return THEMIS_E_INVALID_ARG;
    if (!d_workspace || ((uintptr_t)d_workspace & (kAlign - 1))) return THEMIS_E_INVALID_ARG;
    HostStage H;
    host_stage_of(problem, vertical, L.total_bytes, &H);
    if (workspace_bytes < H.total) return THEMIS_E_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char *base = static_cast<char *>(d_workspace);
    const size_t N = problem->n_instances, S = problem->n_stages;
    const size_t lat_bytes = (size_t)problem->n_profiles * S * problem->c_max * problem->n_batch * 4;
    cudaError_t e;
#define THEMIS_COPY(dst, src, bytes, kind)                                    \
    do {                                                                      \
        e = cudaMemcpyAsync((dst), (src), (bytes), (kind), st);               \
        if (e != cudaSuccess) return fail_cuda(e);                            \
    } while (0)
    THEMIS_COPY(base + H.lat, h_lat_us, lat_bytes, cudaMemcpyHostToDevice);
    if (h_profile_id) THEMIS_COPY(base + H.pid, h_profile_id, N * 4, cudaMemcpyHostToDevice);
    THEMIS_COPY(base + H.lam, h_lambda_mrps, N * 4, cudaMemcpyHostToDevice);
    if (vertical) THEMIS_COPY(base + H.rep, h_replicas, N * S * 4, cudaMemcpyHostToDevice);
    themis_result_t d_out;
    d_out.h = reinterpret_cast<int32_t *>(base + H.h);
    d_out.c = reinterpret_cast<int32_t *>(base + H.c);
    d_out.b = reinterpret_cast<int32_t *>(base + H.b);
    d_out.total_cost = reinterpret_cast<int32_t *>(base + H.cost);
    d_out.latency_buckets = reinterpret_cast<int32_t *>(base + H.latb);
    d_out.status = reinterpret_cast<int32_t *>(base + H.status);
    rc = solve_impl(problem, reinterpret_cast<const int32_t *>(base + H.lat),
                    h_profile_id ? reinterpret_cast<const int32_t *>(base + H.pid) : nullptr,
                    reinterpret_cast<const uint32_t *>(base + H.lam),
                    vertical ? reinterpret_cast<const int32_t *>(base + H.rep) : nullptr,
                    SolveOpts{vertical ? kVertical : kJoint}, d_out,
                    d_workspace, L.total_bytes, st);
    if (rc != THEMIS_OK) return rc;
    THEMIS_COPY(h_out.h, d_out.h, N * S * 4, cudaMemcpyDeviceToHost);
    THEMIS_COPY(h_out.c, d_out.c, N * S * 4, cudaMemcpyDeviceToHost);
    THEMIS_COPY(h_out.b, d_out.b, N * S * 4, cudaMemcpyDeviceToHost);
    THEMIS_COPY(h_out.total_cost, d_out.total_cost, N * 4, cudaMemcpyDeviceToHost);
    THEMIS_COPY(h_out.latency_buckets, d_out.latency_buckets, N * 4, cudaMemcpyDeviceToHost);
    THEMIS_COPY(h_out.status, d_out.status, N * 4, cudaMemcpyDeviceToHost);
#undef THEMIS_COPY
    e = cudaStreamSynchronize(st);
    return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
}

int themis_solve_batch_static(const themis_problem_t *problem, const int32_t *d_lat_us,
                              const int32_t *d_profile_id, const uint32_t *d_lambda_mrps,
                              const int32_t *d_replicas, themis_result_t out, void *cuda_stream)
{
    const int vertical = d_replicas != nullptr;
    themis_workspace_layout_t L;
    int rc = layout_of(problem, vertical, &L);
    if (rc != THEMIS_OK) return rc;
    if (L.total_bytes > (size_t)THEMIS_STATIC_SCRATCH_BYTES) return THEMIS_E_STATIC_SCRATCH_EXCEEDED;
    void *scratch = nullptr;
    rc = static_scratch_ptr(&scratch);
    if (rc != THEMIS_OK) return rc;
    return solve_impl(problem, d_lat_us, d_profile_id, d_lambda_mrps, d_replicas,
                      SolveOpts{vertical ? kVertical : kJoint}, out, scratch,
                      (size_t)THEMIS_STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(cuda_stream));
}

int themis_fit_profiles_batch(int32_t n_models, int32_t n_samples, const int32_t *d_sample_b,
                              const int32_t *d_sample_c, const double *d_latency_ms, int32_t c_max,
                              int32_t n_batch, const int32_t *d_batch_sizes, double *d_coeffs,
                              int32_t *d_lat_us, int32_t *d_status, void *cuda_stream)
{
    if (n_models < 1 || n_samples < 4 || c_max < 1 || n_batch < 1 || n_batch > THEMIS_MAX_BATCH_SIZES ||
        !d_sample_b || !d_sample_c || !d_latency_ms || !d_batch_sizes || !d_coeffs || !d_lat_us || !d_status)
        return THEMIS_E_INVALID_ARG;
    cudaError_t e = launch_fit_profiles(n_models, n_samples, d_sample_b, d_sample_c, d_latency_ms, c_max, n_batch,
                                        d_batch_sizes, d_coeffs, d_lat_us, d_status,
                                        static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
}

int themis_alu_probe(int mode, int blocks, int threads, int iters, uint32_t *d_sink, void *cuda_stream)
{
    if (mode < 0 || mode > 5 || (mode == 5 && threads != 256) || blocks < 1 || threads < 32 || threads > 1024 || iters < 1 || !d_sink)
        return THEMIS_E_INVALID_ARG;
    cudaError_t e = launch_alu_probe(mode, blocks, threads, iters, d_sink, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
}

int themis_bounds_check_report(const themis_problem_t *problem, int vertical, const void *d_workspace,
                               size_t workspace_bytes, int32_t *h_report, void *cuda_stream)
{
    themis_workspace_layout_t L;
    int rc = layout_of(problem, vertical, &L);
    if (rc != THEMIS_OK) return rc;
    if (!d_workspace || !h_report) return THEMIS_E_INVALID_ARG;
    if (workspace_bytes < L.total_bytes) return THEMIS_E_WORKSPACE_TOO_SMALL;
    h_report[0] = h_report[1] = h_report[2] = 0;
    h_report[3] = kBoundsChecked;
    if (!kBoundsChecked) return THEMIS_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaMemcpyAsync(h_report, static_cast<const char *>(d_workspace) + L.total_bytes - kAlign,
                                    3 * sizeof(int32_t), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
}

int themis_wait_probe(int32_t max_polls, const uint32_t *d_src16, uint32_t *d_dst16, int32_t *d_status,
                      void *cuda_stream)
{
    if (max_polls < 1 || max_polls > (1 << 20) || !d_src16 || !d_dst16 || !d_status ||
        ((uintptr_t)d_src16 & 15u))
        return THEMIS_E_INVALID_ARG;
    cudaError_t e = launch_wait_probe((uint32_t)max_polls, d_src16, d_dst16, d_status,
                                      static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? THEMIS_OK : fail_cuda(e);
}

}  // extern "C"

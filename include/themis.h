/*
 * libthemis: batched solver for the joint horizontal + vertical scaling problem
 * of multi-model inference pipelines (Themis, arXiv 2407.14843), for NVIDIA B200.
 *
 * One "instance" is one pipeline of S stages under one arrival rate lambda.  For
 * every stage the solver picks replicas h (the paper's n_s), cores per replica c
 * and batch size b, minimising  sum_s h_s * c_s  (Eq. 6) subject to
 *     sum_s  l_s(b_s, c_s) + q_s(b_s)  <=  SLO            (Eq. 5)
 *     lambda <= h_s * thr_s(b_s, c_s),  thr = b / l(b, c)   (Eq. 6)
 * where l is the profiled processing latency and q the queuing delay of Eq. 4,
 * q = (b - 1) / lambda.  Latencies are discretised to buckets of bucket_us:
 * a stage occupies ceil(l / w) + ceil(q / w) buckets out of T = floor(SLO / w).
 * Instances are independent and solved in one batch.
 *
 * Method (Algorithm 1, restructured): per stage the candidates are reduced to a
 * per-bucket minimum cost G_s[l]; stages are combined by the recurrence
 *     F_0 = G_0,   F_s[t] = min_{0<=l<=t} F_{s-1}[t-l] + G_s[l]
 * and the configuration is read back from the argmin tables.  Ties resolve to
 * the lowest index everywhere (lowest total latency, then lowest latency of the
 * last stage, ..., then lowest candidate index per stage), which is what
 * Algorithm 1's strict '<' in ascending loop order yields.
 *
 * Conventions for every entry point:
 *  - returns THEMIS_OK or a negative THEMIS_E_* code; never throws;
 *  - "d_" pointers are DEVICE memory, "h_" pointers are HOST memory; all are
 *    owned by the caller and must stay valid until the stream work completes;
 *  - nothing is allocated on the device; scratch comes from the caller's
 *    workspace (see themis_workspace_bytes);
 *  - work is enqueued on the given CUDA stream (a cudaStream_t passed as void*,
 *    NULL = default stream) and the call returns without synchronising, except
 *    themis_solve_batch_host, which synchronises the stream before returning;
 *  - scalar arguments are validated on the host before anything is launched;
 *    bad array contents (lambda = 0, latency <= 0, replicas < 1) are detected on
 *    the device and reported per instance in status[n];
 *  - an instance with no feasible configuration is not an error: status[n] = 1
 *    (Algorithm 1's "no solution" branch).
 */
#ifndef THEMIS_H_
#define THEMIS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define THEMIS_VERSION 100

/* problem limits */
#define THEMIS_MAX_BATCH_SIZES 16
#define THEMIS_MAX_STAGES 64
#define THEMIS_MAX_T 16383        /* budget in buckets (argmin tables are 14-bit) */
#define THEMIS_MAX_CANDIDATES 65535 /* per stage (candidate index is uint16) */
#define THEMIS_MAX_TOTAL_COST 131070 /* n_stages * h_max * c_max must not exceed it */

/* themis_problem_t.flags, bit 0: the queuing model */
#define THEMIS_QUEUE_PER_REPLICA 1u /* q = (b-1) * h / lambda: every replica fills
                                       its own batch.  Clear: q = (b-1)/lambda, Eq. 4 */

/* themis_problem_t.flags, bits 8..11: which kernels this call runs.  An implementation
 * choice per call (the paper has no counterpart): returned configurations, costs,
 * latencies and statuses never depend on it; what the rows of the workspace hold
 * does (see themis_workspace_layout_t).  The choice travels with the call, so calls
 * from different host threads on different streams may differ in it.
 *   THEMIS_KERNEL_DEFAULT      same as THEMIS_KERNEL_PACKED16.
 *   THEMIS_KERNEL_PACKED16     dense recurrence on packed 16-bit costs (two budget
 *      cells per register), on costs relative to every stage's cheapest entry; the A
 *      rows then hold the prefix tables themselves, uint16
 *          F_s[t] - sum_{k<=s} min_l G_k[l]     (0x7FFF: unreachable or >= 32767),
 *      computed only for budgets that can still be completed, t <= T - (sum over the later
 *      stages of their first non-empty bucket), and 0x7FFF above (such a state is part of
 *      no solution); the backtrack recovers the argmin along the optimal path only.  Instances
 *      whose optimum lies 32767 or more above the sum of the stages' cheapest entries
 *      are redone by the 32-bit kernel in a second launch.  Budgets of up to 1900 cells
 *      run with one warp per instance, longer ones with one thread block per instance.
 *   THEMIS_KERNEL_PACKED16_BLOCK  the same with one thread block per instance whatever
 *      the budget length (same tables, same results).
 *   THEMIS_KERNEL_WIDE32       dense recurrence on 32-bit keys; the A rows hold the
 *      argmin tables.  Budgets of up to 2800 cells run with one warp per instance, longer
 *      ones (and THEMIS_TILE_16) with one thread block per instance.
 *   THEMIS_KERNEL_PRUNED       dense scoring, then the recurrence restricted to the
 *      undominated entries of every G_s (an entry is dominated when a smaller l has
 *      a cost at most as high; such entries never occur in the returned solution);
 *      A and F are the tables of the restricted problem.  Budgets above about 11000
 *      buckets run THEMIS_KERNEL_PACKED16 instead.
 *   THEMIS_KERNEL_SPARSE       the solvers (themis_solve_*batch, host and static
 *      variants, the fallback) run one kernel, one warp per instance, that scores only
 *      the candidates that can matter (per cores and batch size the fewest replicas
 *      that sustain lambda) and keeps only undominated stage entries and undominated
 *      prefix states (budget, total) as short sorted lists; no dense table exists and
 *      its cost does not grow with the budget length T.  The G rows of the workspace
 *      then hold one backtrack record per prefix state.  Instances whose lists outgrow
 *      the kernel's fixed capacities are redone by THEMIS_KERNEL_SPARSE_BLOCK's kernel
 *      in a second launch.  The two-step entry points treat it as THEMIS_KERNEL_PRUNED.
 *   THEMIS_KERNEL_SPARSE_BLOCK the same restriction with one thread block per instance
 *      and dense shared-memory rows per budget cell (any list length); G, Garg and A
 *      rows hold the stage fronts and the argmin of the front cells.  Falls back to
 *      THEMIS_KERNEL_PRUNED when its shared memory (about 12 * row_pitch bytes plus
 *      tables) does not fit. */
#define THEMIS_KERNEL_DEFAULT      (0u << 8)
#define THEMIS_KERNEL_PACKED16     (1u << 8)
#define THEMIS_KERNEL_WIDE32       (2u << 8)
#define THEMIS_KERNEL_PRUNED       (3u << 8)
#define THEMIS_KERNEL_SPARSE       (4u << 8)
#define THEMIS_KERNEL_SPARSE_BLOCK (5u << 8)
#define THEMIS_KERNEL_PACKED16_BLOCK (6u << 8)
#define THEMIS_KERNEL_MASK         (15u << 8)

/* themis_problem_t.flags, bits 12..13: consecutive budget cells per thread of the
 * dense recurrence kernels (a tuning knob, no counterpart in the paper; the 32-bit
 * kernel treats 4 as its default).  Results do not depend on it. */
#define THEMIS_TILE_DEFAULT (0u << 12)
#define THEMIS_TILE_4       (1u << 12)
#define THEMIS_TILE_8       (2u << 12)
#define THEMIS_TILE_16      (3u << 12)
#define THEMIS_TILE_MASK    (3u << 12)

/* return codes */
#define THEMIS_OK 0
#define THEMIS_E_INVALID_ARG (-1)
#define THEMIS_E_UNSUPPORTED_SIZE (-2)
#define THEMIS_E_WORKSPACE_TOO_SMALL (-3)
#define THEMIS_E_CUDA (-4)
#define THEMIS_E_STATIC_SCRATCH_EXCEEDED (-5)

/* per-instance status */
#define THEMIS_STATUS_OK 0
#define THEMIS_STATUS_INFEASIBLE 1
#define THEMIS_STATUS_SPLIT 2          /* themis_vertical_fallback_batch: part of the load is served
                                          by the replicas in place, the rest needs extra replicas */
#define THEMIS_STATUS_BAD_INPUT (-1)   /* lambda = 0, a latency <= 0, replicas < 1, replicas * c_max > 65535,
                                          sum of replicas * c_max > THEMIS_MAX_TOTAL_COST, profile id out
                                          of range */
#define THEMIS_STATUS_TIMEOUT (-2)     /* a bounded on-device wait expired */

/* value of an empty bucket in the G table of the workspace */
#define THEMIS_G_INF INT32_MAX

typedef struct {
    int32_t n_instances;   /* N >= 1 */
    int32_t n_stages;      /* S in 1..THEMIS_MAX_STAGES */
    int32_t n_profiles;    /* P >= 1 distinct pipelines (sets of latency tables) */
    int32_t c_max;         /* cores per replica range over 1..c_max */
    int32_t n_batch;       /* number of batch sizes, 1..THEMIS_MAX_BATCH_SIZES */
    int32_t batch_sizes[THEMIS_MAX_BATCH_SIZES]; /* strictly increasing, 1..65536 */
    int32_t h_max;         /* joint: replicas range over 1..h_max; vertical: ignored */
    int32_t slo_us;        /* SLO in microseconds */
    int32_t bucket_us;     /* bucket width w; T = slo_us / bucket_us, 1 <= T <= THEMIS_MAX_T */
    uint32_t flags;        /* THEMIS_QUEUE_PER_REPLICA | THEMIS_KERNEL_* | THEMIS_TILE_* */
} themis_problem_t;

/* Result arrays, caller-owned and caller-sized.  Device pointers for the d_
 * entry points, host pointers for themis_solve_batch_host. */
typedef struct {
    int32_t *h;               /* [N][S] row-major; 0 where unsolved */
    int32_t *c;               /* [N][S] */
    int32_t *b;               /* [N][S] */
    int32_t *total_cost;      /* [N] sum_s h*c; -1 where unsolved */
    int32_t *latency_buckets; /* [N] sum of stage latencies in buckets (<= T); -1 where unsolved */
    int32_t *status;          /* [N] THEMIS_STATUS_* */
} themis_result_t;

/* Where the intermediate tables live inside a workspace (byte offsets from its
 * start; rows are row_pitch entries long, entries beyond T are padding).
 *   G    int32  [N][S][row_pitch]  per-bucket minimum cost, THEMIS_G_INF if empty
 *   Garg uint16 [N][S][row_pitch]  lowest candidate index attaining G (0 if empty)
 *   A    uint16 [N][S][row_pitch]  THEMIS_KERNEL_WIDE32: A[s][t] = lowest l attaining
 *                                  F_s[t] (row 0 unused, 0 where F_s[t] is unreachable);
 *                                  THEMIS_KERNEL_PACKED16: the prefix tables F_s[t]
 *                                  (see the THEMIS_KERNEL_* flags)
 *   F    int32  [N][row_pitch]     last prefix table F_{S-1}, THEMIS_G_INF if unreachable
 * Candidate index: idx = ((h-1)*c_max + (c-1))*n_batch + bi (joint),
 *                  idx = (c-1)*n_batch + bi (vertical). */
typedef struct {
    size_t g_offset, garg_offset, a_offset, f_offset, flag_offset;
    size_t total_bytes;
    int32_t row_pitch;
    int32_t T;
} themis_workspace_layout_t;

/* Device workspace needed by the d_ entry points for this problem
 * (8 * N * S * row_pitch bytes plus small terms, among them the scoring kernels'
 * candidate lists: about 24 * c_max * n_batch bytes per profile and stage, which is why
 * n_profiles enters the size).  vertical != 0 selects the h-fixed variant.  Fails with INVALID_ARG / UNSUPPORTED_SIZE like the solvers. */
int themis_workspace_bytes(const themis_problem_t *problem, int vertical, size_t *out_bytes);
int themis_workspace_layout(const themis_problem_t *problem, int vertical,
                            themis_workspace_layout_t *out_layout);

/*
 * Joint solver (Eq. 6 over h in 1..h_max, c in 1..c_max, b in batch_sizes).
 *   d_lat_us       [P][S][c_max][n_batch] int32, batch index fastest: profiled
 *                  latency of one batch in microseconds, >= 1
 *   d_profile_id   [N] int32 in 0..P-1, or NULL (every instance uses profile 0)
 *   d_lambda_mrps  [N] uint32 arrival rate in milli-requests per second, >= 1
 *   out            device result arrays
 *   d_workspace    device scratch, 256-byte aligned, >= themis_workspace_bytes
 * Runs the candidate-scoring kernels (candidate lists per profile and stage, then the
 * per-bucket minimum per instance), then the min-plus/backtrack kernel.
 */
int themis_solve_batch(const themis_problem_t *problem, const int32_t *d_lat_us,
                       const int32_t *d_profile_id, const uint32_t *d_lambda_mrps,
                       themis_result_t out, void *d_workspace, size_t workspace_bytes,
                       void *cuda_stream);

/*
 * In-place vertical-only variant (Algorithm 1): replicas are fixed,
 *   d_replicas     [N][S] int32, >= 1
 * candidates range over (c, b) only and a stage costs replicas * c.
 */
int themis_solve_vertical_batch(const themis_problem_t *problem, const int32_t *d_lat_us,
                                const int32_t *d_profile_id, const uint32_t *d_lambda_mrps,
                                const int32_t *d_replicas, themis_result_t out,
                                void *d_workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Vertical solver with Algorithm 1's last branch.  Instances for which the
 * replicas in place cannot serve lambda within the SLO at any core count are
 * split: a bisection on the arrival rate finds a rate lambda_vertical that
 * vertical scaling still serves, and the rest of the load is given to extra
 * replicas with the cores and batch size just chosen,
 *     extra[n][s] = ceil((lambda - lambda_vertical) / thr_s(b_s, c_s)).
 * Search points are multiples k * resolution_mrps: lo = 0, hi = ceil(lambda /
 * resolution); while hi - lo > 1: mid = (lo + hi) / 2, served at mid * resolution ?
 * lo = mid : hi = mid (the printed loop's midpoint and branch are garbled; this is
 * the reading taken).  Feasibility is not monotone in the rate in general, so, as
 * in the paper, the result is a served rate whose next search point is not served,
 * not necessarily the largest such rate.
 *   lambda_max_mrps      host-side upper bound on every d_lambda_mrps[n]; fixes the
 *                        number of bisection rounds, ceil(log2(ceil(max / resolution))),
 *                        without reading the device.  An instance above the bound
 *                        that needs the search gets THEMIS_STATUS_BAD_INPUT.
 *   d_lambda_vertical    [N] uint32 out: lambda where the instance is feasible as it
 *                        is, else the served rate found (0 if not even `resolution`
 *                        is served: status stays THEMIS_STATUS_INFEASIBLE)
 *   d_extra_replicas     [N][S] int32 out: 0 except for THEMIS_STATUS_SPLIT instances
 *   out                  the vertical part's configuration (for split instances: the
 *                        solve at lambda_vertical), status in {0, 1, 2, < 0}
 * A search point only has to be classified as served or not, and a rate is served
 * exactly when the fastest feasible candidates of all stages fit the budget
 * together, so the search of an instance runs inside one kernel without the
 * recurrence; the recurrence runs twice, at the full rate and at the rate found
 * (for the searching instances only).  Workspace: themis_fallback_workspace_bytes.
 */
int themis_fallback_workspace_bytes(const themis_problem_t *problem, size_t *out_bytes);
int themis_vertical_fallback_batch(const themis_problem_t *problem, const int32_t *d_lat_us,
                                   const int32_t *d_profile_id, const uint32_t *d_lambda_mrps,
                                   const int32_t *d_replicas, uint32_t resolution_mrps,
                                   uint32_t lambda_max_mrps, themis_result_t out,
                                   uint32_t *d_lambda_vertical, int32_t *d_extra_replicas,
                                   void *d_workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Horizontal-only variant (Algorithm 2): one-core replicas.  problem->c_max must
 * be 1 and d_lat_us is [P][S][1][n_batch].  For every stage and batch size the
 * replica count is not enumerated but computed, h = ceil(lambda / thr(b, 1)), the
 * fewest replicas with thr * h >= lambda (Algorithm 2 prints a floor, which would
 * break Eq. 6's throughput constraint); batch sizes that would need more than
 * problem->h_max replicas are dropped.  Cost of a stage is h.  Results equal those
 * of themis_solve_batch on the same problem (extra replicas only add cost and
 * queuing delay), at n_batch instead of h_max * n_batch candidates per stage.
 * In the workspace, Garg holds the batch index and G the replica count.
 * Solving the same pipelines at the current and at the predicted arrival rate
 * (two batches, or one batch of 2N instances) and comparing the returned
 * configurations is the paper's test for a stable workload (Section "Transition").
 */
int themis_solve_horizontal_batch(const themis_problem_t *problem, const int32_t *d_lat_us,
                                  const int32_t *d_profile_id, const uint32_t *d_lambda_mrps,
                                  themis_result_t out, void *d_workspace, size_t workspace_bytes,
                                  void *cuda_stream);

/*
 * Stability test of the transition policy (Section "Transition", vertical to
 * horizontal: when): the workload counts as stable when the horizontal solver
 * returns the same configuration for the current and for the predicted arrival
 * rate.  Given the results of two solves of the same N pipelines (device arrays),
 *   d_stable[n] = 1 iff both have status 0 and equal (h, c, b) at every stage, else 0.
 */
int themis_configs_equal_batch(int32_t n_instances, int32_t n_stages, themis_result_t current,
                               themis_result_t predicted, int32_t *d_stable, void *cuda_stream);

/*
 * The two halves of the solvers, for checking and timing each step on its own.
 * themis_score_batch fills G and Garg of the workspace (candidate scoring: the
 * inner loops of Algorithm 1 with Eq. 4 and the throughput test of Eq. 6);
 * themis_minplus_batch consumes them (recurrence, final scan, backtrack) and
 * fills A, F and the result arrays.  d_replicas = NULL selects the joint problem.
 * Calling them back to back on one stream equals the corresponding solver.
 */
int themis_score_batch(const themis_problem_t *problem, const int32_t *d_lat_us,
                       const int32_t *d_profile_id, const uint32_t *d_lambda_mrps,
                       const int32_t *d_replicas, void *d_workspace, size_t workspace_bytes,
                       void *cuda_stream);
int themis_minplus_batch(const themis_problem_t *problem, const int32_t *d_replicas,
                         themis_result_t out, void *d_workspace, size_t workspace_bytes,
                         void *cuda_stream);

/*
 * Host-buffer variant: inputs and results are HOST arrays (pinned memory makes
 * the copies asynchronous).  Copies the inputs into the workspace, solves, copies
 * the results back and synchronises the stream.  h_replicas = NULL selects the
 * joint problem.  The workspace must hold themis_host_workspace_bytes.
 */
int themis_host_workspace_bytes(const themis_problem_t *problem, int vertical, size_t *out_bytes);
int themis_solve_batch_host(const themis_problem_t *problem, const int32_t *h_lat_us,
                            const int32_t *h_profile_id, const uint32_t *h_lambda_mrps,
                            const int32_t *h_replicas, themis_result_t h_out,
                            void *d_workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Solver variant for callers that cannot allocate device memory.  (The paper has
 * no counterpart; this is a convenience of the library.)
 *
 * Some callers have no way to obtain a workspace: code running under a memory
 * pool that hands out no scratch, a plug-in that is only given its input and
 * output buffers, a service that must not call cudaMalloc on its request path
 * because that call synchronises the device.  For them this entry point runs
 * the same kernels as themis_solve_batch / themis_solve_vertical_batch (whichever
 * the problem's THEMIS_KERNEL_* flag selects; d_replicas = NULL selects the joint
 * problem) with the intermediate tables in
 * a fixed buffer of THEMIS_STATIC_SCRATCH_BYTES that is part of the library
 * image: every GPU that loads the library holds that much memory until the
 * process exits.  It calls no allocation or free routine of any kind.
 *
 *  - Limit: themis_workspace_bytes(problem) must not exceed
 *    THEMIS_STATIC_SCRATCH_BYTES; larger problems are refused with
 *    THEMIS_E_STATIC_SCRATCH_EXCEEDED before anything is launched (split the
 *    batch, or use the workspace entry points).
 *  - The first call on each device looks up the buffer's device address (with
 *    that device current).  Make that first call outside any stream capture.
 *  - All calls share the one buffer, which keeps whatever the last call left in
 *    it.  Nothing in it has to start at zero: every word a call reads it has
 *    written itself first, so no clearing is done.  Two calls whose kernels
 *    overlap on the GPU (different streams, or different host threads on
 *    different streams) race on the buffer and give wrong results: keep calls on
 *    one stream, or order them with events.
 */
#define THEMIS_STATIC_SCRATCH_BYTES (32u << 20)
int themis_solve_batch_static(const themis_problem_t *problem, const int32_t *d_lat_us,
                              const int32_t *d_profile_id, const uint32_t *d_lambda_mrps,
                              const int32_t *d_replicas, themis_result_t out, void *cuda_stream);

/*
 * Profile fit (Eq. 1): least-squares fit of
 *     l(b, c) = gamma * b / c + epsilon / c + delta * b + eta      [milliseconds]
 * to measured samples, one model (pipeline stage) at a time, and the latency table
 * the solvers take as input, evaluated from the fitted coefficients.
 *   d_sample_b, d_sample_c  [n_samples] int32: the (batch size, cores) grid the models
 *                           were run on (shared by all models), values >= 1
 *   d_latency_ms            [n_models][n_samples] double: measured latency per model
 *   d_batch_sizes           [n_batch] int32 (device): the table's batch sizes
 *   d_coeffs                [n_models][4] double out: gamma, epsilon, delta, eta
 *   d_lat_us                [n_models][c_max][n_batch] int32 out: ceil(1000 * l(b, c)),
 *                           at least 1; this is the layout of one profile's stages
 *                           in the solvers' d_lat_us when models are its stages
 *   d_status                [n_models] int32 out: 0, or THEMIS_STATUS_BAD_INPUT when the
 *                           samples do not determine the four coefficients (table = 0)
 * Double precision throughout (normal equations, Gaussian elimination with partial
 * pivoting).  n_samples >= 4.
 */
int themis_fit_profiles_batch(int32_t n_models, int32_t n_samples, const int32_t *d_sample_b,
                              const int32_t *d_sample_c, const double *d_latency_ms, int32_t c_max,
                              int32_t n_batch, const int32_t *d_batch_sizes, double *d_coeffs,
                              int32_t *d_lat_us, int32_t *d_status, void *cuda_stream);

/* Library housekeeping (no counterpart in the paper).  Text for a return code; for THEMIS_E_CUDA includes the last CUDA error seen by
 * the calling thread.  The pointer stays valid until the thread's next call. */
const char *themis_strerror(int code);
int themis_version(void);

#ifdef __cplusplus
}
#endif
#endif /* THEMIS_H_ */

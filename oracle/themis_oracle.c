/*
 * CPU oracle for the batched pipeline-scaling solver (Themis, arXiv 2407.14843).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, scalar restatement of
 * what the solver computes.  It shares no code with the CUDA library and must
 * never be called from the product path; only the tests, the smoke check and
 * the benchmark's CPU-baseline leg use it.
 *
 * What is computed, per independent instance (one pipeline, one arrival rate):
 *
 *   minimise   sum_s  h_s * c_s                               (Eq. 6, objective)
 *   subject to sum_s  l_s(b_s, c_s) + q_s(b_s)  <=  SLO       (Eq. 5 / Eq. 6)
 *              lambda <= thr_s(b_s, c_s) * h_s   for all s     (Eq. 6)
 *
 * with h = replicas (the paper's n_s), c = cores per replica, b = batch size,
 * thr(b, c) = b / l(b, c) the throughput of one replica, and the queuing delay
 * q(b) = (b - 1) / lambda of Eq. 4 (optionally (b - 1) * h / lambda when every
 * replica fills its own batch, flag ORACLE_QUEUE_PER_REPLICA).
 *
 * Latencies are discretised to buckets of width w: a stage costs
 * ceil(l / w) + ceil(q / w) buckets and the budget is T = floor(SLO / w).
 *
 * Three solvers are provided and pinned against each other by the tests:
 *   oracle_solve_batch      the stage-by-stage dynamic program of Algorithm 1,
 *                           with the candidate minimum hoisted out of the
 *                           budget loop (G_s) and a min-plus combine (F_s);
 *   oracle_alg1_scatter     the same optimum by forward relaxation over reachable
 *                           (stage, budget) states, extended option by option in
 *                           Algorithm 1's visiting order, with no per-bucket
 *                           minimum and no (min,+) combine;
 *   brute_force.c           Eq. 6 by exhaustive enumeration (separate file);
 * and, for the horizontal-only solver of Algorithm 2 (one-core replicas, replica
 * count computed as ceil(lambda / thr) per batch size):
 *   oracle_solve_horizontal_batch   the same program over batch sizes only;
 *   oracle_alg2_scatter             Algorithm 2's problem by the same forward relaxation.
 *
 * Readings of the paper taken here (each is pinned by a test):
 *   - a candidate is skipped iff its replicas cannot sustain lambda or it does
 *     not fit the remaining budget (the printed condition in Algorithm 1 is
 *     inverted; the prose under it states the intent);
 *   - throughput equality (thr * h == lambda) is feasible, as in Eq. 6;
 *   - the budget test is on i + l, the index actually written;
 *   - ties: strict '<' in ascending candidate order, so the lowest candidate
 *     index wins, the lowest stage latency wins in the combine, and the lowest
 *     total latency wins in the final scan (the paper's loops do the same);
 *   - cost of a stage is h * c (Eq. 6), which equals Algorithm 1's 'c' when
 *     every stage has one replica.
 *
 * Candidate index: idx = ((h - 1) * c_max + (c - 1)) * n_batch + bi for the
 * joint problem (h slowest, then c, batch fastest, the loop order of
 * Algorithm 1 with h added outside); idx = (c - 1) * n_batch + bi when h is
 * fixed.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_INF INT32_MAX
#define ORACLE_QUEUE_PER_REPLICA 1u

typedef struct {
    int32_t n_instances;
    int32_t n_stages;
    int32_t n_profiles;
    int32_t c_max;
    int32_t n_batch;
    int32_t batch_sizes[16];
    int32_t h_max;
    int32_t slo_us;
    int32_t bucket_us;
    uint32_t flags;
} oracle_problem;

static uint64_t ceil_div_u64(uint64_t a, uint64_t b) { return (a + b - 1) / b; }

/*
 * One candidate of one stage (the body of Algorithm 1's inner loops).
 * Returns 1 and sets *ell (latency in buckets) and *cost when the candidate
 * can sustain the arrival rate; returns 0 otherwise.  *ell may exceed T.
 *
 *   l   = profiled latency of a batch of b on c cores          [us]
 *   q   = (b - 1) / lambda  (times h with the per-replica flag) [us]  (Eq. 4)
 *   thr = b / l per replica; feasible iff h * thr >= lambda     (Eq. 6)
 *
 * lambda is given in milli-requests per second, so
 *   h * b / (l_us * 1e-6) >= lambda_m * 1e-3   <=>   h * b * 1e9 >= lambda_m * l_us
 *   q_us = (b - 1) * m * 1e9 / lambda_m.
 */
static int score_candidate(int32_t l_us, int32_t h, int32_t c, int32_t b, uint32_t lambda_m,
                           int32_t bucket_us, uint32_t flags, int64_t *ell, int32_t *cost)
{
    uint64_t supply = (uint64_t)h * (uint64_t)b * 1000000000ull;
    uint64_t demand = (uint64_t)lambda_m * (uint64_t)l_us;
    if (supply < demand) return 0;
    uint64_t m = (flags & ORACLE_QUEUE_PER_REPLICA) ? (uint64_t)h : 1ull;
    uint64_t q_buckets = ceil_div_u64((uint64_t)(b - 1) * m * 1000000000ull,
                                      (uint64_t)lambda_m * (uint64_t)bucket_us);
    uint64_t l_buckets = ceil_div_u64((uint64_t)l_us, (uint64_t)bucket_us);
    *ell = (int64_t)(l_buckets + q_buckets);
    *cost = h * c;
    return 1;
}

/*
 * Per-bucket minimum over the candidates of one stage:
 *   G[l]    = min cost over feasible candidates whose latency is exactly l buckets
 *   Garg[l] = lowest candidate index attaining it (0 where G[l] is INF)
 * lat_stage is [c_max][n_batch].  h_fixed > 0 selects the vertical variant.
 */
void oracle_score_stage(const oracle_problem *p, const int32_t *lat_stage, uint32_t lambda_m,
                        int32_t h_fixed, int32_t T, int32_t *G, uint16_t *Garg)
{
    for (int32_t l = 0; l <= T; ++l) { G[l] = ORACLE_INF; Garg[l] = 0; }
    int32_t h_lo = h_fixed > 0 ? h_fixed : 1;
    int32_t h_hi = h_fixed > 0 ? h_fixed : p->h_max;
    int32_t idx = 0;
    for (int32_t h = h_lo; h <= h_hi; ++h)
        for (int32_t c = 1; c <= p->c_max; ++c)
            for (int32_t bi = 0; bi < p->n_batch; ++bi, ++idx) {
                int64_t ell; int32_t cost;
                int32_t l_us = lat_stage[(c - 1) * p->n_batch + bi];
                if (!score_candidate(l_us, h, c, p->batch_sizes[bi], lambda_m, p->bucket_us,
                                     p->flags, &ell, &cost))
                    continue;
                if (ell > T) continue;
                if (cost < G[ell]) { G[ell] = cost; Garg[ell] = (uint16_t)idx; }
            }
}

/*
 * Horizontal scaling (Algorithm 2): one-core replicas only.  For every batch
 * size the replica count is computed, not enumerated: the fewest replicas whose
 * combined throughput sustains lambda, h = ceil(lambda / thr(b, 1)) (Algorithm 2
 * prints a floor, which would leave thr * h below lambda; Eq. 6 requires
 * thr * h >= lambda).  Candidates that would need more than h_max replicas are
 * dropped.  Cost is h (one core each); candidate index = batch index.
 * lat_stage is [1][n_batch].
 */
static int horizontal_candidate(const oracle_problem *p, int32_t l_us, int32_t b, uint32_t lambda_m,
                                int64_t *ell, int32_t *h_out)
{
    uint64_t per_replica = (uint64_t)b * 1000000000ull;              /* b / l, scaled */
    uint64_t demand = (uint64_t)lambda_m * (uint64_t)l_us;
    uint64_t h = ceil_div_u64(demand, per_replica);
    if (h < 1) h = 1;
    if (h > (uint64_t)p->h_max) return 0;
    int32_t cost;
    if (!score_candidate(l_us, (int32_t)h, 1, b, lambda_m, p->bucket_us, p->flags, ell, &cost)) return 0;
    *h_out = (int32_t)h;
    return 1;
}

void oracle_score_stage_horizontal(const oracle_problem *p, const int32_t *lat_stage, uint32_t lambda_m,
                                   int32_t T, int32_t *G, uint16_t *Garg)
{
    for (int32_t l = 0; l <= T; ++l) { G[l] = ORACLE_INF; Garg[l] = 0; }
    for (int32_t bi = 0; bi < p->n_batch; ++bi) {
        int64_t ell; int32_t h;
        if (!horizontal_candidate(p, lat_stage[bi], p->batch_sizes[bi], lambda_m, &ell, &h)) continue;
        if (ell > T) continue;
        if (h < G[ell]) { G[ell] = h; Garg[ell] = (uint16_t)bi; }
    }
}

/*
 * Min-plus combine of the prefix with one more stage:
 *   F[t] = min_{0 <= l <= t} Fprev[t - l] + G[l],  A[t] = lowest l attaining it
 * (A[t] = 0 where F[t] is INF).
 */
void oracle_minplus(int32_t T, const int32_t *Fprev, const int32_t *G, int32_t *F, uint16_t *A)
{
    for (int32_t t = 0; t <= T; ++t) {
        int32_t best = ORACLE_INF; int32_t arg = 0;
        for (int32_t l = 0; l <= t; ++l) {
            if (Fprev[t - l] == ORACLE_INF || G[l] == ORACLE_INF) continue;
            int32_t v = Fprev[t - l] + G[l];
            if (v < best) { best = v; arg = l; }
        }
        F[t] = best; A[t] = (uint16_t)arg;
    }
}

static void decode_idx(const oracle_problem *p, int32_t idx, int32_t h_fixed,
                       int32_t *h, int32_t *c, int32_t *b)
{
    int32_t bi = idx % p->n_batch;
    int32_t r = idx / p->n_batch;
    *b = p->batch_sizes[bi];
    *c = r % p->c_max + 1;
    *h = h_fixed > 0 ? h_fixed : r / p->c_max + 1;
}

/*
 * One instance, dynamic program.  Work arrays hold S rows of T+1 entries:
 *   Gs, Gargs  per-stage candidate minima;  Fs  prefix tables;  As  argmin.
 * Returns 0 (solved) or 1 (infeasible).
 */
static int solve_instance(const oracle_problem *p, const int32_t *lat_pipeline /* [S][C][B] */,
                          uint32_t lambda_m, const int32_t *replicas /* [S] or NULL */, int horizontal,
                          int32_t *h_out, int32_t *c_out, int32_t *b_out,
                          int32_t *cost_out, int32_t *lat_out,
                          int32_t *Gs, uint16_t *Gargs, int32_t *Fs, uint16_t *As)
{
    const int32_t S = p->n_stages, T = p->slo_us / p->bucket_us, W = T + 1;
    const int32_t stage_words = p->c_max * p->n_batch;
    for (int32_t s = 0; s < S; ++s) {
        if (horizontal)
            oracle_score_stage_horizontal(p, lat_pipeline + (size_t)s * stage_words, lambda_m, T,
                                          Gs + (size_t)s * W, Gargs + (size_t)s * W);
        else
            oracle_score_stage(p, lat_pipeline + (size_t)s * stage_words, lambda_m,
                               replicas ? replicas[s] : 0, T, Gs + (size_t)s * W, Gargs + (size_t)s * W);
    }
    /* first stage: the whole budget spent so far belongs to it */
    memcpy(Fs, Gs, sizeof(int32_t) * (size_t)W);
    memset(As, 0, sizeof(uint16_t) * (size_t)W);
    for (int32_t s = 1; s < S; ++s)
        oracle_minplus(T, Fs + (size_t)(s - 1) * W, Gs + (size_t)s * W,
                       Fs + (size_t)s * W, As + (size_t)s * W);
    /* final scan: cheapest total, lowest total latency among equals */
    const int32_t *Fl = Fs + (size_t)(S - 1) * W;
    int32_t best = ORACLE_INF, tstar = -1;
    for (int32_t t = 0; t <= T; ++t)
        if (Fl[t] < best) { best = Fl[t]; tstar = t; }
    if (tstar < 0) {
        for (int32_t s = 0; s < S; ++s) { h_out[s] = 0; c_out[s] = 0; b_out[s] = 0; }
        *cost_out = -1; *lat_out = -1;
        return 1;
    }
    /* walk the argmin tables back from the last stage */
    int32_t t = tstar;
    for (int32_t s = S - 1; s >= 0; --s) {
        int32_t ell = s > 0 ? (int32_t)As[(size_t)s * W + t] : t;
        int32_t idx = Gargs[(size_t)s * W + ell];
        if (horizontal) {      /* the stage's cost is its replica count */
            h_out[s] = Gs[(size_t)s * W + ell]; c_out[s] = 1; b_out[s] = p->batch_sizes[idx];
        } else {
            decode_idx(p, idx, replicas ? replicas[s] : 0, &h_out[s], &c_out[s], &b_out[s]);
        }
        t -= ell;
    }
    *cost_out = best; *lat_out = tstar;
    return 0;
}

/*
 * Batch driver.  All pointers are host memory.
 *   lat_us      [P][S][c_max][n_batch]
 *   profile_id  [N] or NULL (all 0)
 *   lambda_mrps [N]
 *   replicas    [N][S] (vertical variant) or NULL (joint)
 *   h, c, b     [N][S];  total_cost, latency_buckets, status  [N]
 * Optional dumps (NULL to skip), row-major with rows of T+1 entries:
 *   dump_G int32 [N][S][T+1], dump_Garg uint16 [N][S][T+1],
 *   dump_F int32 [N][S][T+1], dump_A uint16 [N][S][T+1]  (A row 0 is zero).
 * n_threads <= 0 uses every core OpenMP sees.  Returns the thread count used,
 * or -1 on allocation failure.
 */
static int solve_batch_mode(const oracle_problem *p, const int32_t *lat_us, const int32_t *profile_id,
                            const uint32_t *lambda_mrps, const int32_t *replicas, int horizontal,
                            int32_t *h, int32_t *c, int32_t *b,
                            int32_t *total_cost, int32_t *latency_buckets, int32_t *status,
                            int32_t *dump_G, uint16_t *dump_Garg, int32_t *dump_F, uint16_t *dump_A,
                            int n_threads)
{
    const int32_t N = p->n_instances, S = p->n_stages;
    const size_t W = (size_t)(p->slo_us / p->bucket_us) + 1;
    const size_t rows = (size_t)S * W;
    const size_t pipeline_words = (size_t)S * p->c_max * p->n_batch;
    int used = 1, failed = 0;
#ifdef _OPENMP
    if (n_threads <= 0) n_threads = omp_get_max_threads();
    used = n_threads;
#pragma omp parallel num_threads(n_threads)
#endif
    {
        int32_t *Gs = (int32_t *)malloc(sizeof(int32_t) * rows);
        int32_t *Fs = (int32_t *)malloc(sizeof(int32_t) * rows);
        uint16_t *Gargs = (uint16_t *)malloc(sizeof(uint16_t) * rows);
        uint16_t *As = (uint16_t *)malloc(sizeof(uint16_t) * rows);
        if (!Gs || !Fs || !Gargs || !As) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            failed = 1;
        } else {
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
            for (int32_t n = 0; n < N; ++n) {
                int32_t pid = profile_id ? profile_id[n] : 0;
                status[n] = solve_instance(p, lat_us + (size_t)pid * pipeline_words, lambda_mrps[n],
                                           replicas ? replicas + (size_t)n * S : NULL, horizontal,
                                           h + (size_t)n * S, c + (size_t)n * S, b + (size_t)n * S,
                                           &total_cost[n], &latency_buckets[n], Gs, Gargs, Fs, As);
                if (dump_G) memcpy(dump_G + (size_t)n * rows, Gs, sizeof(int32_t) * rows);
                if (dump_F) memcpy(dump_F + (size_t)n * rows, Fs, sizeof(int32_t) * rows);
                if (dump_Garg) memcpy(dump_Garg + (size_t)n * rows, Gargs, sizeof(uint16_t) * rows);
                if (dump_A) memcpy(dump_A + (size_t)n * rows, As, sizeof(uint16_t) * rows);
            }
        }
        free(Gs); free(Fs); free(Gargs); free(As);
    }
    return failed ? -1 : used;
}

int oracle_solve_batch(const oracle_problem *p, const int32_t *lat_us, const int32_t *profile_id,
                       const uint32_t *lambda_mrps, const int32_t *replicas,
                       int32_t *h, int32_t *c, int32_t *b,
                       int32_t *total_cost, int32_t *latency_buckets, int32_t *status,
                       int32_t *dump_G, uint16_t *dump_Garg, int32_t *dump_F, uint16_t *dump_A,
                       int n_threads)
{
    return solve_batch_mode(p, lat_us, profile_id, lambda_mrps, replicas, 0, h, c, b, total_cost,
                            latency_buckets, status, dump_G, dump_Garg, dump_F, dump_A, n_threads);
}

/* Horizontal-only variant (Algorithm 2): c_max must be 1, lat_us is [P][S][1][n_batch]. */
int oracle_solve_horizontal_batch(const oracle_problem *p, const int32_t *lat_us, const int32_t *profile_id,
                                  const uint32_t *lambda_mrps,
                                  int32_t *h, int32_t *c, int32_t *b,
                                  int32_t *total_cost, int32_t *latency_buckets, int32_t *status,
                                  int32_t *dump_G, uint16_t *dump_Garg, int32_t *dump_F, uint16_t *dump_A,
                                  int n_threads)
{
    if (p->c_max != 1) return -1;
    return solve_batch_mode(p, lat_us, profile_id, lambda_mrps, NULL, 1, h, c, b, total_cost,
                            latency_buckets, status, dump_G, dump_Garg, dump_F, dump_A, n_threads);
}

/*
 * Algorithm 1's last branch, batch form.  When the replicas in place cannot serve
 * lambda within the SLO at any core count, the paper bisects on the workload for
 * the largest rate that vertical scaling still serves and brings up extra replicas,
 * with the cores and batch size just chosen, for the rest.  Reading taken of the
 * printed loop (whose midpoint and branch sense are garbled): search points are
 * multiples k * resolution; lo = 0 (nothing served), hi = ceil(lambda / resolution)
 * (known not to be served); while hi - lo > 1: mid = (lo + hi) / 2, served at
 * mid * resolution ? lo = mid : hi = mid.  Feasibility is not monotone in the rate
 * in general (queuing delay shrinks as the rate grows), so this is the paper's
 * heuristic, not a maximum: the result is a rate that is served whose successor
 * search point is not.
 *   lambda_vertical[n] = lo * resolution (lambda itself if the instance is feasible;
 *                        0 if no search point is served: status stays 1)
 *   extra[n][s]        = ceil((lambda - lambda_vertical) / thr_s(b_s, c_s)) replicas
 *   status             = 0 feasible as is, 2 split into vertical + extra replicas,
 *                        1 not even the lowest search point is served
 * h, c, b, total_cost, latency_buckets describe the vertical part.
 */
int oracle_vertical_fallback_batch(const oracle_problem *p, const int32_t *lat_us, const int32_t *profile_id,
                                   const uint32_t *lambda_mrps, const int32_t *replicas, uint32_t resolution,
                                   int32_t *h, int32_t *c, int32_t *b,
                                   int32_t *total_cost, int32_t *latency_buckets, int32_t *status,
                                   uint32_t *lambda_vertical, int32_t *extra, int n_threads)
{
    const int32_t N = p->n_instances, S = p->n_stages;
    const size_t W = (size_t)(p->slo_us / p->bucket_us) + 1;
    const size_t rows = (size_t)S * W;
    const size_t pipeline_words = (size_t)S * p->c_max * p->n_batch;
    int used = 1, failed = 0;
    if (resolution < 1 || !replicas) return -1;
#ifdef _OPENMP
    if (n_threads <= 0) n_threads = omp_get_max_threads();
    used = n_threads;
#pragma omp parallel num_threads(n_threads)
#endif
    {
        int32_t *Gs = (int32_t *)malloc(sizeof(int32_t) * rows);
        int32_t *Fs = (int32_t *)malloc(sizeof(int32_t) * rows);
        uint16_t *Gargs = (uint16_t *)malloc(sizeof(uint16_t) * rows);
        uint16_t *As = (uint16_t *)malloc(sizeof(uint16_t) * rows);
        if (!Gs || !Fs || !Gargs || !As) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            failed = 1;
        } else {
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
            for (int32_t n = 0; n < N; ++n) {
                const int32_t *lat = lat_us + (size_t)(profile_id ? profile_id[n] : 0) * pipeline_words;
                const int32_t *rep = replicas + (size_t)n * S;
                int32_t *hn = h + (size_t)n * S, *cn = c + (size_t)n * S, *bn = b + (size_t)n * S;
                int32_t *en = extra + (size_t)n * S;
                const uint32_t lam = lambda_mrps[n];
                for (int32_t s = 0; s < S; ++s) en[s] = 0;
                int st = solve_instance(p, lat, lam, rep, 0, hn, cn, bn, &total_cost[n], &latency_buckets[n],
                                        Gs, Gargs, Fs, As);
                lambda_vertical[n] = lam;
                status[n] = st;
                if (st == 0) continue;
                uint64_t lo = 0, hi = ((uint64_t)lam + resolution - 1) / resolution;
                while (hi - lo > 1) {
                    uint64_t mid = (lo + hi) / 2;
                    int served = solve_instance(p, lat, (uint32_t)(mid * resolution), rep, 0, hn, cn, bn,
                                                &total_cost[n], &latency_buckets[n], Gs, Gargs, Fs, As) == 0;
                    if (served) lo = mid; else hi = mid;
                }
                lambda_vertical[n] = (uint32_t)(lo * resolution);
                if (lo == 0) {       /* leave the "no configuration" result of the last trial */
                    solve_instance(p, lat, lam, rep, 0, hn, cn, bn, &total_cost[n], &latency_buckets[n],
                                   Gs, Gargs, Fs, As);
                    continue;
                }
                solve_instance(p, lat, lambda_vertical[n], rep, 0, hn, cn, bn, &total_cost[n],
                               &latency_buckets[n], Gs, Gargs, Fs, As);
                status[n] = 2;
                const uint64_t rest = (uint64_t)lam - lambda_vertical[n];
                for (int32_t s = 0; s < S; ++s) {
                    int32_t bi = 0;
                    while (p->batch_sizes[bi] != bn[s]) ++bi;
                    uint64_t l_us = (uint64_t)lat[((size_t)s * p->c_max + (cn[s] - 1)) * p->n_batch + bi];
                    en[s] = (int32_t)ceil_div_u64(rest * l_us, (uint64_t)bn[s] * 1000000000ull);
                }
            }
        }
        free(Gs); free(Fs); free(Gargs); free(As);
    }
    return failed ? -1 : used;
}

/*
 * Cross-check of the hoisted solver: the same optimum by forward relaxation over
 * reachable states, without per-bucket minima and without a (min,+) combine.
 *
 * A state is "the first s+1 stages take exactly t buckets"; it remembers the
 * cheapest total found so far, the state of the previous stage it was reached
 * from and the option that led there.  The options of a stage (feasible
 * candidates with their latency, cost and index) are listed once, in index
 * order; then every reachable state of the previous stage, the one with the
 * largest budget first, is extended by every option that still fits, and a
 * state is replaced only by a strictly cheaper total.  Visiting order and the
 * strict comparison are what Algorithm 1 / Algorithm 2 do (budget loop downwards,
 * candidate loops upwards, '<'), so ties resolve as there: for a given state the
 * extension with the shortest stage latency, and among those the lowest option
 * index, is kept.  The final choice is the cheapest state of the last stage, the
 * smallest budget among equals.
 */
typedef struct { int32_t ell, cost, idx, h; } relax_option;
typedef struct { int32_t total, from, option; } relax_state;    /* total < 0: not reached */

static int relax_pipeline(int32_t S, int32_t T, relax_option *const *options, const int32_t *n_options,
                          int32_t *opt_of_stage /* [S] out: chosen option per stage */,
                          int32_t *cost_out, int32_t *lat_out)
{
    const int32_t W = T + 1;
    relax_state *st = (relax_state *)malloc(sizeof(relax_state) * (size_t)S * W);
    if (!st) return -1;
    for (size_t k = 0; k < (size_t)S * W; ++k) st[k].total = -1;
    for (int32_t s = 0; s < S; ++s) {
        relax_state *here = st + (size_t)s * W;
        const relax_state *before = s ? st + (size_t)(s - 1) * W : NULL;
        for (int32_t spent = s ? T : 0; spent >= 0; --spent) {
            int32_t base_total = 0;
            if (before) {
                if (before[spent].total < 0) continue;
                base_total = before[spent].total;
            }
            for (int32_t o = 0; o < n_options[s]; ++o) {
                const relax_option *opt = &options[s][o];
                if ((int64_t)spent + opt->ell > T) continue;
                relax_state *dst = &here[spent + opt->ell];
                int32_t total = base_total + opt->cost;
                if (dst->total < 0 || total < dst->total) {
                    dst->total = total; dst->from = spent; dst->option = o;
                }
            }
        }
    }
    int32_t end = -1;
    const relax_state *last = st + (size_t)(S - 1) * W;
    for (int32_t t = 0; t <= T; ++t)
        if (last[t].total >= 0 && (end < 0 || last[t].total < last[end].total)) end = t;
    int rc = 1;
    *cost_out = -1; *lat_out = -1;
    if (end >= 0) {
        *cost_out = last[end].total; *lat_out = end;
        int32_t t = end;
        for (int32_t s = S - 1; s >= 0; --s) {
            const relax_state *x = &st[(size_t)s * W + t];
            opt_of_stage[s] = x->option;
            t = x->from;
        }
        rc = 0;
    }
    free(st);
    return rc;
}

/* Runs relax_pipeline on the options produced by fill(stage, list) and decodes the result. */
static int relax_and_decode(const oracle_problem *p, const int32_t *lat_pipeline, uint32_t lambda_m,
                            const int32_t *replicas, int horizontal, int32_t *h_out, int32_t *c_out,
                            int32_t *b_out, int32_t *cost_out, int32_t *lat_out)
{
    const int32_t S = p->n_stages, T = p->slo_us / p->bucket_us;
    const int32_t per_stage_max = horizontal ? p->n_batch : (replicas ? 1 : p->h_max) * p->c_max * p->n_batch;
    relax_option **options = (relax_option **)calloc((size_t)S, sizeof(relax_option *));
    int32_t *n_options = (int32_t *)calloc((size_t)S, sizeof(int32_t));
    int32_t *chosen = (int32_t *)calloc((size_t)S, sizeof(int32_t));
    int rc = -1;
    if (!options || !n_options || !chosen) goto done;
    for (int32_t s = 0; s < S; ++s) {
        options[s] = (relax_option *)malloc(sizeof(relax_option) * (size_t)per_stage_max);
        if (!options[s]) goto done;
        relax_option *list = options[s];
        int32_t n = 0;
        if (horizontal) {
            const int32_t *lat_stage = lat_pipeline + (size_t)s * p->n_batch;
            for (int32_t bi = 0; bi < p->n_batch; ++bi) {
                int64_t ell; int32_t h;
                if (!horizontal_candidate(p, lat_stage[bi], p->batch_sizes[bi], lambda_m, &ell, &h)) continue;
                if (ell > T) continue;
                list[n].ell = (int32_t)ell; list[n].cost = h; list[n].idx = bi; list[n].h = h;
                ++n;
            }
        } else {
            const int32_t *lat_stage = lat_pipeline + (size_t)s * p->c_max * p->n_batch;
            const int32_t h_first = replicas ? replicas[s] : 1, h_last = replicas ? replicas[s] : p->h_max;
            int32_t idx = 0;
            for (int32_t h = h_first; h <= h_last; ++h)
                for (int32_t c = 1; c <= p->c_max; ++c)
                    for (int32_t bi = 0; bi < p->n_batch; ++bi, ++idx) {
                        int64_t ell; int32_t cost;
                        if (!score_candidate(lat_stage[(c - 1) * p->n_batch + bi], h, c, p->batch_sizes[bi],
                                             lambda_m, p->bucket_us, p->flags, &ell, &cost))
                            continue;
                        if (ell > T) continue;
                        list[n].ell = (int32_t)ell; list[n].cost = cost; list[n].idx = idx; list[n].h = h;
                        ++n;
                    }
        }
        n_options[s] = n;
    }
    rc = relax_pipeline(S, T, options, n_options, chosen, cost_out, lat_out);
    if (rc >= 0) {
        for (int32_t s = 0; s < S; ++s) {
            if (rc != 0) { h_out[s] = 0; c_out[s] = 0; b_out[s] = 0; continue; }
            const relax_option *opt = &options[s][chosen[s]];
            if (horizontal) { h_out[s] = opt->h; c_out[s] = 1; b_out[s] = p->batch_sizes[opt->idx]; }
            else decode_idx(p, opt->idx, replicas ? replicas[s] : 0, &h_out[s], &c_out[s], &b_out[s]);
        }
    }
done:
    if (options) for (int32_t s = 0; s < S; ++s) free(options[s]);
    free(options); free(n_options); free(chosen);
    return rc;
}

/* Algorithm 2's problem (one-core replicas, replica count computed per batch size) by
 * forward relaxation; lat_pipeline is [S][1][n_batch].  Returns 0 (solved) or 1 (infeasible). */
int oracle_alg2_scatter(const oracle_problem *p, const int32_t *lat_pipeline, uint32_t lambda_m,
                        const int32_t *unused, int32_t *h_out, int32_t *c_out, int32_t *b_out,
                        int32_t *cost_out, int32_t *lat_out)
{
    (void)unused;
    return relax_and_decode(p, lat_pipeline, lambda_m, NULL, 1, h_out, c_out, b_out, cost_out, lat_out);
}

/* Algorithm 1's problem (replicas given) or the joint problem (replicas == NULL) by forward
 * relaxation; lat_pipeline is [S][c_max][n_batch].  Returns 0 (solved) or 1 (infeasible);
 * outputs as in oracle_solve_batch. */
int oracle_alg1_scatter(const oracle_problem *p, const int32_t *lat_pipeline, uint32_t lambda_m,
                        const int32_t *replicas, int32_t *h_out, int32_t *c_out, int32_t *b_out,
                        int32_t *cost_out, int32_t *lat_out)
{
    return relax_and_decode(p, lat_pipeline, lambda_m, replicas, 0, h_out, c_out, b_out, cost_out, lat_out);
}

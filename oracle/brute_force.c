/*
 * Exhaustive solver for the scaling integer program (Themis, arXiv 2407.14843,
 * Eq. 6): every tuple of per-stage configurations is visited.
 *
 * TEST INFRASTRUCTURE ONLY: it pins the dynamic-programming oracle on
 * instances small enough to enumerate (K^S tuples).  It shares no code with
 * the CUDA library, and none with themis_oracle.c either: the candidate test
 * below is restated in 128-bit arithmetic straight from the inequalities
 *
 *     n_s * thr_s(b, c) >= lambda,   thr = b / l(b, c)          (Eq. 6)
 *     sum_s ceil(l_s / w) + ceil(q_s / w) <= T,  q = (b-1)/lambda  (Eq. 4, 5)
 *
 * Among all feasible tuples the winner minimises, in lexicographic order,
 *   ( total cost, total latency, latency of the last stage, of the one before,
 *     ..., of the second stage, candidate index of stage 0, 1, ..., S-1 ),
 * which is the solution a stage-by-stage program with strict '<' comparisons
 * in ascending order reaches.
 */
#include <stdint.h>
#include <stdlib.h>

typedef struct {
    int32_t n_instances, n_stages, n_profiles, c_max, n_batch;
    int32_t batch_sizes[16];
    int32_t h_max, slo_us, bucket_us;
    uint32_t flags;
} bf_problem;

typedef struct { int32_t idx, h, c, b, cost; int64_t ell; } bf_cand;

typedef unsigned __int128 u128;

#define BF_MAX_STAGES 8

typedef struct {
    int32_t S, T;
    const bf_cand *cands[BF_MAX_STAGES];
    int32_t n_cands[BF_MAX_STAGES];
    int32_t pick[BF_MAX_STAGES];
    int have_best;
    int64_t best_cost, best_lat;
    int32_t best_pick[BF_MAX_STAGES];
} bf_state;

/* is tuple 'a' (picks) strictly better than the stored best under the key? */
static int better(const bf_state *st, int64_t cost, int64_t lat)
{
    if (!st->have_best) return 1;
    if (cost != st->best_cost) return cost < st->best_cost;
    if (lat != st->best_lat) return lat < st->best_lat;
    for (int32_t s = st->S - 1; s >= 1; --s) {
        int64_t a = st->cands[s][st->pick[s]].ell, b = st->cands[s][st->best_pick[s]].ell;
        if (a != b) return a < b;
    }
    for (int32_t s = 0; s < st->S; ++s) {
        int32_t a = st->cands[s][st->pick[s]].idx, b = st->cands[s][st->best_pick[s]].idx;
        if (a != b) return a < b;
    }
    return 0;
}

static void enumerate(bf_state *st, int32_t s, int64_t cost, int64_t lat)
{
    if (s == st->S) {
        if (better(st, cost, lat)) {
            st->have_best = 1; st->best_cost = cost; st->best_lat = lat;
            for (int32_t k = 0; k < st->S; ++k) st->best_pick[k] = st->pick[k];
        }
        return;
    }
    for (int32_t k = 0; k < st->n_cands[s]; ++k) {
        const bf_cand *cd = &st->cands[s][k];
        if (lat + cd->ell > st->T) continue;       /* Eq. 5: the sum only grows */
        st->pick[s] = k;
        enumerate(st, s + 1, cost + cd->cost, lat + cd->ell);
    }
}

/*
 * One instance.  lat_pipeline is [S][c_max][n_batch] in microseconds, lambda
 * in milli-requests/s, replicas [S] (h fixed per stage) or NULL (h in 1..h_max).
 * Outputs h, c, b [S], total cost, total latency in buckets.
 * Returns 0 solved, 1 infeasible, -1 unsupported (S > 8 or no memory).
 */
int brute_force_instance(const bf_problem *p, const int32_t *lat_pipeline, uint32_t lambda_m,
                         const int32_t *replicas, int32_t *h_out, int32_t *c_out, int32_t *b_out,
                         int32_t *cost_out, int32_t *lat_out)
{
    const int32_t S = p->n_stages;
    if (S > BF_MAX_STAGES) return -1;
    bf_state st;
    st.S = S; st.T = p->slo_us / p->bucket_us; st.have_best = 0;
    bf_cand *store[BF_MAX_STAGES] = {0};
    int rc = 0;
    for (int32_t s = 0; s < S && rc == 0; ++s) {
        int32_t h_lo = replicas ? replicas[s] : 1, h_hi = replicas ? replicas[s] : p->h_max;
        int32_t K = (h_hi - h_lo + 1) * p->c_max * p->n_batch;
        store[s] = (bf_cand *)malloc(sizeof(bf_cand) * (size_t)K);
        if (!store[s]) { rc = -1; break; }
        int32_t n = 0, idx = 0;
        for (int32_t h = h_lo; h <= h_hi; ++h)
            for (int32_t c = 1; c <= p->c_max; ++c)
                for (int32_t bi = 0; bi < p->n_batch; ++bi, ++idx) {
                    int32_t b = p->batch_sizes[bi];
                    u128 l_us = (u128)lat_pipeline[((size_t)s * p->c_max + (c - 1)) * p->n_batch + bi];
                    /* h * (b / l) >= lambda, cleared of fractions */
                    if ((u128)h * b * 1000000000u < (u128)lambda_m * l_us) continue;
                    u128 m = (p->flags & 1u) ? (u128)h : (u128)1;
                    u128 q_num = (u128)(b - 1) * m * 1000000000u;   /* q in us times lambda_m */
                    u128 q_den = (u128)lambda_m * (u128)p->bucket_us;
                    u128 q_b = q_num / q_den + (q_num % q_den != 0);
                    u128 l_b = l_us / (u128)p->bucket_us + (l_us % (u128)p->bucket_us != 0);
                    bf_cand cd = { idx, h, c, b, h * c, (int64_t)(q_b + l_b) };
                    store[s][n++] = cd;
                }
        st.cands[s] = store[s]; st.n_cands[s] = n;
    }
    if (rc == 0) {
        enumerate(&st, 0, 0, 0);
        if (!st.have_best) {
            for (int32_t s = 0; s < S; ++s) { h_out[s] = 0; c_out[s] = 0; b_out[s] = 0; }
            *cost_out = -1; *lat_out = -1; rc = 1;
        } else {
            for (int32_t s = 0; s < S; ++s) {
                const bf_cand *cd = &st.cands[s][st.best_pick[s]];
                h_out[s] = cd->h; c_out[s] = cd->c; b_out[s] = cd->b;
            }
            *cost_out = (int32_t)st.best_cost; *lat_out = (int32_t)st.best_lat;
        }
    }
    for (int32_t s = 0; s < S; ++s) free(store[s]);
    return rc;
}

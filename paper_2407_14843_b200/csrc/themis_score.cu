// Candidate scoring: reduces every stage's candidate configurations to the
// per-bucket minimum-cost vector G_s and its argmin Garg_s (the inner loops of
// Algorithm 1, with the queuing delay of Eq. 4 and the throughput constraint of
// Eq. 6), one thread block per instance.
//
// Everything that needs 64-bit arithmetic is hoisted out of the candidate loop
// into two small shared-memory tables indexed by (batch size, replicas):
//   Q[bi][h]    = ceil((b-1) * m * 1e9 / (lambda_m * w_us)),  m = h or 1   (Eq. 4 in buckets)
//   Lmax[bi][h] = floor(h * b * 1e9 / lambda_m)     largest latency [us] that still
//                 satisfies  h * b / l >= lambda                           (Eq. 6)
// (joint problem: one table for all stages; vertical variant: one row pair per
// stage, for that stage's fixed replica count), all filled before the first stage.
// A candidate then costs a compare, an add, a multiply-add and a shared-memory
// atomic min on the packed word (cost << 16 | candidate index), whose ordering
// gives "cheapest, then lowest index" directly.
//
// Work is dealt to warps as (one batch size) x (32 consecutive core counts), so
// all lanes of a warp read the same table rows (no bank conflicts) and walk the
// replica count upward from the fewest replicas that sustain lambda.  Two key
// rows alternate between stages, so a stage costs one block barrier.
#include "themis_internal.h"

namespace themis {
namespace {

constexpr uint32_t kEmptyKey = 0xFFFFFFFFu;
constexpr int kScoreThreads = 256;

__device__ __forceinline__ uint32_t sat_u32(unsigned long long v, uint32_t cap)
{
    return v > (unsigned long long)cap ? cap : (uint32_t)v;
}

__global__ void __launch_bounds__(kScoreThreads)
score_kernel(const Params p)
{
    extern __shared__ __align__(16) uint32_t smem[];
    const int n = blockIdx.x;
    if (p.active && !p.active[n]) return;
    const int tid = threadIdx.x;
    const int T = p.T, pitch = p.pitch;
    const int S = p.prob.n_stages, C = p.prob.c_max, NB = p.prob.n_batch;
    const int CB = C * NB;
    const int HN = p.vertical ? 1 : p.prob.h_max;   // replica values per table row
    const int SV = p.vertical ? S : 1;              // table sets: one per stage when h is per stage
    const uint32_t w_us = (uint32_t)p.prob.bucket_us;

    uint32_t *keys0 = smem;                     // [pitch]
    uint32_t *keys1 = keys0 + pitch;            // [pitch]
    uint32_t *Q = keys1 + pitch;                // [SV][NB][HN]
    uint32_t *Lmax = Q + SV * NB * HN;          // [SV][NB][HN]
    __shared__ int s_bad;

    const uint32_t lambda_m = p.lambda_mrps[n];
    const int pid = p.profile_id ? p.profile_id[n] : 0;
    const int32_t *lat = p.lat_us + (size_t)pid * S * CB;
    const int32_t *rep = p.vertical ? p.replicas + (size_t)n * S : nullptr;

    if (tid == 0) {
        int bad = (lambda_m == 0) || pid < 0 || pid >= p.prob.n_profiles;
        if (rep) {
            long long total = 0;
            for (int s = 0; s < S; ++s) {
                if (rep[s] < 1 || (long long)rep[s] * C > 65535) bad = 1;   // cost field is 16 bits
                total += (long long)rep[s] * C;
            }
            if (total > THEMIS_MAX_TOTAL_COST) bad = 1;
        }
        s_bad = bad;
    }
    for (int l = tid; l < 2 * pitch; l += kScoreThreads) keys0[l] = kEmptyKey;
    __syncthreads();
    const bool skip_all = s_bad != 0;

    if (!skip_all) {
        const unsigned long long q_den = (unsigned long long)lambda_m * w_us;
        for (int e = tid; e < SV * NB * HN; e += kScoreThreads) {
            const int sv = e / (NB * HN);
            const int bi = (e - sv * NB * HN) / HN;
            const int k = e - (sv * NB + bi) * HN;
            const unsigned long long h = (unsigned long long)((p.vertical ? rep[sv] : 1) + k);
            const unsigned long long b = (unsigned long long)p.prob.batch_sizes[bi];
            const unsigned long long m = (p.prob.flags & THEMIS_QUEUE_PER_REPLICA) ? h : 1ull;
            const unsigned long long q_num = (b - 1ull) * m * 1000000000ull;
            Q[e] = sat_u32((q_num + q_den - 1ull) / q_den, (uint32_t)T + 1u);
            Lmax[e] = sat_u32(h * b * 1000000000ull / lambda_m, 0x7FFFFFFFu);
        }
    }
    __syncthreads();                            // tables ready, both key rows empty

    const bool q_grows_with_h = (p.prob.flags & THEMIS_QUEUE_PER_REPLICA) != 0;
    int saw_bad_latency = 0;
    const int lane = tid & 31, warp = tid >> 5;
    const int c_chunks = (C + 31) / 32;
    const int n_tasks = NB * c_chunks;
    const uint32_t w_magic = 0xFFFFFFFFu / w_us;            // floor((2^32 - 1) / w)

    for (int s = 0; s < S; ++s) {
        uint32_t *keys = (s & 1) ? keys1 : keys0;
        if (!skip_all) {
            const int h_lo = p.vertical ? rep[s] : 1;
            const int32_t *lat_s = lat + (size_t)s * CB;
            const uint32_t *Q_s = Q + (p.vertical ? s * NB : 0);
            const uint32_t *Lmax_s = Lmax + (p.vertical ? s * NB : 0);
            for (int task = warp; task < n_tasks; task += kScoreThreads / 32) {
                const int bi = task / c_chunks;
                const int c = (task - bi * c_chunks) * 32 + lane + 1;
                if (c > C) continue;
                const int pair = (c - 1) * NB + bi;
                const int32_t l_us = lat_s[pair];
                if (l_us <= 0) { saw_bad_latency = 1; continue; }
                // Same latency with one core fewer: that candidate reaches the same buckets with
                // the same replica counts at a lower cost, so this one can never be a minimum
                // (latency tables are flat over long runs of core counts).
                if (c > 1 && lat_s[pair - NB] == l_us) continue;
                // l_b = ceil(l_us / w): quotient estimate by the precomputed reciprocal, then fix up
                uint32_t l_q = __umulhi((uint32_t)l_us, w_magic);
                uint32_t l_r = (uint32_t)l_us - l_q * w_us;
                while (l_r >= w_us) { l_r -= w_us; ++l_q; }
                const uint32_t l_b = l_q + (l_r != 0u);
                if (l_b > (uint32_t)T) continue;
                const int b = p.prob.batch_sizes[bi];
                // Stop at the fewest replicas when more of them cannot reach another bucket
                // more cheaply (q does not depend on h), or when only that count is a candidate.
                const bool q_const = !q_grows_with_h || b == 1 || p.horizontal;
                const uint32_t *q_row = Q_s + bi * HN;
                const uint32_t *lmax_row = Lmax_s + bi * HN;
                // Fewest replicas that sustain lambda: feasibility is monotone in h.  Start
                // from a floating-point estimate of lambda * l / b and settle it on the exact
                // integer table; if the estimate is not provably below the answer, scan from 0.
                const float need = (float)l_us * ((float)lambda_m / ((float)b * 1.0e9f)) - (float)h_lo;
                int k = (int)fminf(fmaxf(need, 0.0f), (float)HN) - 1;      // one or two below the answer
                k = max(k, 0);
                if (k > 0 && (uint32_t)l_us <= lmax_row[k - 1]) k = 0;     // estimate not below: scan from 0
                while (k < HN && (uint32_t)l_us > lmax_row[k]) ++k;        // cannot sustain lambda
                uint32_t cost = (uint32_t)(h_lo + k) * (uint32_t)c;
                uint32_t idx = (uint32_t)((p.horizontal ? 0 : k * CB) + pair);
                for (; k < HN; ++k, cost += (uint32_t)c, idx += (uint32_t)CB) {
                    const uint32_t ell = l_b + q_row[k];
                    if (ell > (uint32_t)T) break;                  // q never shrinks with h
                    atomicMin(&keys[ell], (cost << 16) | idx);
                    if (q_const) break;   // more replicas only cost more in this bucket
                }
            }
        }
        __syncthreads();
        // Unpack to G (int32) and Garg (uint16), four buckets per thread, and leave the
        // key row empty for the stage after next (the next stage uses the other row).
        int32_t *G_row = p.G + ((size_t)n * S + s) * pitch;
        uint16_t *Garg_row = p.Garg + ((size_t)n * S + s) * pitch;
        for (int l4 = tid * 4; l4 < pitch; l4 += kScoreThreads * 4) {
            const uint4 k4 = *reinterpret_cast<const uint4 *>(keys + l4);
            *reinterpret_cast<uint4 *>(keys + l4) = make_uint4(kEmptyKey, kEmptyKey, kEmptyKey, kEmptyKey);
            const uint32_t kk[4] = {k4.x, k4.y, k4.z, k4.w};
            int4 g;
            int32_t *gv = reinterpret_cast<int32_t *>(&g);
            uint32_t a[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const bool empty = kk[i] == kEmptyKey;
                gv[i] = empty ? THEMIS_G_INF : (int32_t)(kk[i] >> 16);
                a[i] = empty ? 0u : (kk[i] & 0xFFFFu);
            }
            *reinterpret_cast<int4 *>(G_row + l4) = g;
            *reinterpret_cast<uint2 *>(Garg_row + l4) = make_uint2(a[0] | (a[1] << 16), a[2] | (a[3] << 16));
        }
    }
    const int any_bad = __syncthreads_or(saw_bad_latency);
    if (tid == 0) p.inst_flag[n] = (skip_all || any_bad) ? kFlagBadInput : 0;
}

}  // namespace

cudaError_t launch_score(const Params &p, cudaStream_t stream)
{
    const size_t table = p.vertical ? (size_t)p.prob.n_stages * p.prob.n_batch
                                    : (size_t)p.prob.n_batch * p.prob.h_max;
    const size_t smem = sizeof(uint32_t) * (2u * (size_t)p.pitch + 2u * table);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess) return e;
    }
    score_kernel<<<p.prob.n_instances, kScoreThreads, smem, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace themis

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
// so one candidate costs a compare, an add, a multiply and a shared-memory
// atomic min on the packed word (cost << 16 | candidate index), whose ordering
// gives "cheapest, then lowest index" directly.
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
    const int tid = threadIdx.x;
    const int T = p.T, pitch = p.pitch;
    const int S = p.prob.n_stages, C = p.prob.c_max, NB = p.prob.n_batch;
    const int CB = C * NB;
    const int HN = p.vertical ? 1 : p.prob.h_max;   // replica values per table row
    const uint32_t w_us = (uint32_t)p.prob.bucket_us;

    uint32_t *keys = smem;                      // [pitch]
    uint32_t *Q = keys + pitch;                 // [NB][HN]
    uint32_t *Lmax = Q + NB * HN;               // [NB][HN]
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
                if (rep[s] < 1) bad = 1;
                total += (long long)rep[s] * C;
            }
            if (total > THEMIS_MAX_TOTAL_COST) bad = 1;
        }
        s_bad = bad;
    }
    for (int l = tid; l < pitch; l += kScoreThreads) keys[l] = kEmptyKey;
    __syncthreads();
    const bool skip_all = s_bad != 0;

    // Fills Q and Lmax for replicas h_lo .. h_lo + HN - 1.
    auto fill_tables = [&](int h_lo) {
        const unsigned long long q_den = (unsigned long long)lambda_m * w_us;
        for (int e = tid; e < NB * HN; e += kScoreThreads) {
            const int bi = e / HN;
            const unsigned long long h = (unsigned long long)(h_lo + e % HN);
            const unsigned long long b = (unsigned long long)p.prob.batch_sizes[bi];
            const unsigned long long m = (p.prob.flags & THEMIS_QUEUE_PER_REPLICA) ? h : 1ull;
            const unsigned long long q_num = (b - 1ull) * m * 1000000000ull;
            Q[e] = sat_u32((q_num + q_den - 1ull) / q_den, (uint32_t)T + 1u);
            Lmax[e] = sat_u32(h * b * 1000000000ull / lambda_m, 0x7FFFFFFFu);
        }
    };
    if (!skip_all && !p.vertical) fill_tables(1);

    const bool q_grows_with_h = (p.prob.flags & THEMIS_QUEUE_PER_REPLICA) != 0;
    int saw_bad_latency = 0;

    for (int s = 0; s < S; ++s) {
        const int h_lo = p.vertical ? (skip_all ? 1 : rep[s]) : 1;
        if (!skip_all && p.vertical) fill_tables(h_lo);
        __syncthreads();                       // tables ready, keys are all empty
        if (!skip_all) {
            const int32_t *lat_s = lat + (size_t)s * CB;
            for (int pair = tid; pair < CB; pair += kScoreThreads) {
                const int bi = pair % NB;
                const int c = pair / NB + 1;
                const int32_t l_us = lat_s[pair];
                if (l_us <= 0) { saw_bad_latency = 1; continue; }
                const uint32_t l_b = ((uint32_t)l_us + w_us - 1u) / w_us;
                if (l_b > (uint32_t)T) continue;
                const bool q_const = !q_grows_with_h || p.prob.batch_sizes[bi] == 1;
                const uint32_t *q_row = Q + bi * HN;
                const uint32_t *lmax_row = Lmax + bi * HN;
                for (int k = 0; k < HN; ++k) {
                    if ((uint32_t)l_us > lmax_row[k]) continue;    // cannot sustain lambda
                    const uint32_t ell = l_b + q_row[k];
                    if (ell > (uint32_t)T) break;                  // q never shrinks with h
                    const uint32_t cost = (uint32_t)(h_lo + k) * (uint32_t)c;
                    const uint32_t idx = (uint32_t)(k * CB + pair);
                    atomicMin(&keys[ell], (cost << 16) | idx);
                    if (q_const) break;   // more replicas only cost more in this bucket
                }
            }
        }
        __syncthreads();
        // Unpack to G (int32) and Garg (uint16), four buckets per thread, and
        // leave the key row empty for the next stage.
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
        // the barrier at the top of the next stage orders these key writes
    }
    const int any_bad = __syncthreads_or(saw_bad_latency);
    if (tid == 0) p.inst_flag[n] = (skip_all || any_bad) ? 1 : 0;
}

}  // namespace

cudaError_t launch_score(const Params &p, cudaStream_t stream)
{
    const int HN = p.vertical ? 1 : p.prob.h_max;
    const size_t smem = sizeof(uint32_t) * ((size_t)p.pitch + 2u * (size_t)p.prob.n_batch * HN);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess) return e;
    }
    score_kernel<<<p.prob.n_instances, kScoreThreads, smem, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace themis

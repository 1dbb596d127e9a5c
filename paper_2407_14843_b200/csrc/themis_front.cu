// Whole solver on short sorted lists, one warp per instance: candidate scoring, the
// undominated entries ("front") of every stage and of every prefix of stages, and the
// stage recurrence, with work that does not grow with the budget length T.
//
// The recurrence F_s[t] = min_l F_{s-1}[t-l] + G_s[l] (Algorithm 1's budget loop with the
// candidate minimum hoisted) only ever returns undominated entries: a stage entry (l, cost)
// with a smaller l' at cost' <= cost, or a prefix state (t, total) with a smaller t' at
// total' <= total, can be swapped for its dominator without raising the cost and with a
// lower total latency, so the solution the solver returns (cheapest, then lowest total
// latency, then lowest stage latencies from the last stage down, then lowest candidate
// indices) contains neither.  Hence per (cores, batch size) only the fewest replicas that
// sustain lambda are scored (Eq. 6's throughput constraint; more replicas cost more and
// never shorten the latency), and only fronts are combined.
//
// A front is a list sorted by latency with strictly falling cost, one packed word per
// entry: cost << 14 | latency (a stage) or total << 14 | budget (a prefix).  Two kernels,
// one warp per instance in each, so that each keeps only its own lists in shared memory
// and more instances share an SM:
//
// stage_fronts_kernel: per stage, scores the candidates, drops those that a candidate in
//   a coarser-grained lower latency bin already beats (64 bins, a warp-wide prefix minimum),
//   and builds the front from the survivors by repeated minimum, cheapest entry first: a
//   step takes the smallest word among survivors below the previous entry's latency (one
//   warp reduction, a second one for the lowest candidate index among equals).  The front
//   goes to the workspace (G row: words, Garg row: candidate indices, A row word 0: count).
//   The next stage's latency table is fetched (cp.async) meanwhile.
//
// prefix_fronts_kernel: the recurrence.  Lane k owns the list "front(F_{s-1}) shifted by
//   entry k of front(G_s)", itself sorted with falling cost, so its best entry below a budget
//   bound is the last one below it.  Its position is the number of prefix budgets up to
//   (bound - 1 - l_k), read from a bitmap of the prefix's budgets with running counts per
//   word (two loads and a population count, no search).  A step is one warp reduction over
//   the lanes' current words, cheapest entry first; the lowest k among equals wins (lowest
//   stage latency).  Every step yields one entry.  The workspace receives one record per
//   entry, (position of its predecessor << 16 | candidate index), in the order found (they
//   overwrite the stage front in the G row, which is in registers by then); the backtrack
//   starts at record 0 of the last stage.
//
// Capacities are fixed per launch (stage front: 128 entries, up to four lists per lane; survivors
// of the bin test: 512; prefix front: `cap` entries of shared memory).  An instance that
// outgrows them is appended to the redo list and solved by the block-per-instance kernel
// afterwards.
#include "themis_async.cuh"
#include "themis_internal.h"

namespace themis {
namespace {

constexpr int kFrontWarps = 4;          // instances per block; warps never wait for each other
constexpr int kMaxStageFront = 128;     // entries of a stage's front: four lists per lane at most
constexpr int kBins = 256;              // latency bins of the dominance pre-test: eight per lane
constexpr int kMaxSurvivors = 512;      // candidates that may pass the pre-test
constexpr uint32_t kNone = 0xFFFFFFFFu;
constexpr uint32_t kLowMask = kIdxMask; // latency / budget field of a packed entry

__device__ __forceinline__ uint32_t sat_u32(unsigned long long v, uint32_t cap)
{
    return v > (unsigned long long)cap ? cap : (uint32_t)v;
}

__device__ __forceinline__ uint32_t warp_min(uint32_t v) { return __reduce_min_sync(0xFFFFFFFFu, v); }

// Asynchronous copy of n words from global to this warp's shared memory (one commit group);
// dst is 16-byte aligned, 16-byte pieces are used when src is too and n is a multiple of 4.
__device__ __forceinline__ void prefetch_words(uint32_t *dst, const int32_t *src, int n, int lane)
{
    if (((n & 3) | (int)(reinterpret_cast<uintptr_t>(src) & 15u)) == 0) {
        for (int i = 4 * lane; i < n; i += 128)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst + i)), "l"(src + i) : "memory");
    } else {
        for (int i = lane; i < n; i += 32)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_addr(dst + i)), "l"(src + i) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// Warps per block that let most warps share an SM's shared memory (227 KB, 1 KB reserved per
// block, at most 32 blocks), the larger block among equals; 0 if one warp does not fit.
int warps_per_block(size_t warp_bytes)
{
    int warps = 0, best = 0;
    for (int w = 1; w <= kFrontWarps; ++w) {
        if (w * warp_bytes > kMaxDynamicSmem) break;
        size_t blocks = (227u * 1024u) / (w * warp_bytes + 1024u);
        if (blocks > 32) blocks = 32;
        if ((int)(blocks * w) >= best) { best = (int)(blocks * w); warps = w; }
    }
    return warps;
}

// ------------------------------------------------------------------ stage fronts

// Shared memory of one warp of stage_fronts_kernel, in words.
struct StageLayout {
    int tab;        // entries of Q and of Lmax
    int cb;         // c_max * n_batch rounded up to a multiple of 32
    int words;      // total, a multiple of 4
};

__host__ __device__ inline StageLayout stage_layout(int C, int NB, int HN, int SV)
{
    StageLayout L;
    L.tab = SV * NB * HN;
    L.cb = (C * NB + 31) & ~31;
    // latency table | candidate words | candidate indices (16 bit) | bins | survivors: words,
    // indices (16 bit) | stage front: words, indices | rates | Q | Lmax
    L.words = (2 * L.cb + L.cb / 2 + kBins + kMaxSurvivors + kMaxSurvivors / 2 + 2 * kMaxStageFront +
               THEMIS_MAX_BATCH_SIZES + 2 * L.tab + 3) & ~3;
    return L;
}

__global__ void __launch_bounds__(kFrontWarps * 32)
stage_fronts_kernel(const Params p)
{
    extern __shared__ __align__(16) uint32_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = blockIdx.x * (blockDim.x >> 5) + warp;
    if (n >= p.prob.n_instances) return;
    if (p.active && !p.active[n]) return;
    const int T = p.T, pitch = p.pitch;
    const int S = p.prob.n_stages, C = p.prob.c_max, NB = p.prob.n_batch;
    const int CB = C * NB;
    const int HN = p.vertical ? 1 : p.prob.h_max;
    const int SV = p.vertical ? S : 1;
    const uint32_t w_us = (uint32_t)p.prob.bucket_us;
    const StageLayout L = stage_layout(C, NB, HN, SV);

    uint32_t *latb = smem + (size_t)warp * L.words;       // [cb] latency table of the stage being scored
    uint32_t *ckey = latb + L.cb;                          // [cb] candidates: cost << 14 | latency, kNone = none
    uint16_t *cidx = reinterpret_cast<uint16_t *>(ckey + L.cb);        // [cb] ... and their candidate index
    uint32_t *bins = ckey + L.cb + L.cb / 2;               // [256] cheapest word per latency bin, 16-byte aligned
    uint32_t *skey = bins + kBins;                         // [512] survivors of the bin test
    uint16_t *sidx = reinterpret_cast<uint16_t *>(skey + kMaxSurvivors);
    uint32_t *gf = skey + kMaxSurvivors + kMaxSurvivors / 2;   // [128] stage front, filled from the last slot down
    uint32_t *gidx = gf + kMaxStageFront;                  // [64]
    float *rate_b = reinterpret_cast<float *>(gidx + kMaxStageFront);   // [16] lambda / (b * 1e9)
    uint32_t *Q = reinterpret_cast<uint32_t *>(rate_b) + THEMIS_MAX_BATCH_SIZES;   // [SV][NB][HN]
    uint32_t *Lmax = Q + L.tab;                            // [SV][NB][HN]

    const uint32_t lambda_m = p.lambda_mrps[n];
    const int pid = p.profile_id ? p.profile_id[n] : 0;
    const int32_t *rep = p.vertical ? p.replicas + (size_t)n * S : nullptr;
    auto write_bad_input = [&]() {
        int32_t *h_o = p.out.h + (size_t)n * S, *c_o = p.out.c + (size_t)n * S, *b_o = p.out.b + (size_t)n * S;
        for (int s = lane; s < S; s += 32) { h_o[s] = 0; c_o[s] = 0; b_o[s] = 0; }
        if (lane == 0) {
            p.out.total_cost[n] = -1;
            p.out.latency_buckets[n] = -1;
            p.out.status[n] = THEMIS_STATUS_BAD_INPUT;
            p.inst_flag[n] = kFlagBadInput;
        }
    };

    {
        int bad = (lambda_m == 0) || pid < 0 || pid >= p.prob.n_profiles;
        if (rep) {
            int total = 0;                                 // at most 64 stages x 65535
            for (int s = lane; s < S; s += 32) {
                const int r = rep[s];
                if (r < 1 || (long long)r * C > 65535) bad = 1; else total += r * C;
            }
            total = __reduce_add_sync(0xFFFFFFFFu, total);
            if (total > THEMIS_MAX_TOTAL_COST) bad = 1;
        }
        if (__any_sync(0xFFFFFFFFu, bad)) { write_bad_input(); return; }
    }
    const int32_t *lat = p.lat_us + (size_t)pid * S * CB;
    prefetch_words(latb, lat, CB, lane);                   // stage 0's table, behind the divisions below
    {
        const unsigned long long q_den = (unsigned long long)lambda_m * w_us;
        for (int e = lane; e < L.tab; e += 32) {
            const int sv = e / (NB * HN);
            const int bi = (e - sv * NB * HN) / HN;
            const int k = e - (sv * NB + bi) * HN;
            const unsigned long long h = (unsigned long long)((p.vertical ? rep[sv] : 1) + k);
            const unsigned long long b = (unsigned long long)p.prob.batch_sizes[bi];
            const unsigned long long m = (p.prob.flags & THEMIS_QUEUE_PER_REPLICA) ? h : 1ull;
            const unsigned long long q_num = (b - 1ull) * m * 1000000000ull;
            Q[TH_IDX(601, e, L.tab)] = sat_u32((q_num + q_den - 1ull) / q_den, (uint32_t)T + 1u);
            Lmax[TH_IDX(602, e, L.tab)] = sat_u32(h * b * 1000000000ull / lambda_m, 0x7FFFFFFFu);
        }
        if (lane < NB) rate_b[lane] = (float)lambda_m / ((float)p.prob.batch_sizes[lane] * 1.0e9f);
    }

    const uint32_t w_magic = 0xFFFFFFFFu / w_us;
    const uint32_t nb_magic = NB > 1 ? 0xFFFFFFFFu / (uint32_t)NB + 1u : 0u;   // e / NB for e < 2^16
    // latency bin of l (0 .. T): floor(l * 64 / (T + 1)), monotone, so a lower bin means a lower latency
    const uint32_t bin_scale = (uint32_t)(((unsigned long long)kBins << 16) / (unsigned)(T + 1));
    const uint32_t lanemask_lt = (1u << lane) - 1u;
    int saw_bad_latency = 0;
    bool redo = false;

    for (int s = 0; s < S && !redo; ++s) {
        for (int b = lane; b < kBins; b += 32) bins[b] = kNone;
        asm volatile("cp.async.wait_all;" ::: "memory");
        __syncwarp();                                      // this stage's latencies (and the tables) are in place
        // 1. candidates of stage s: per (cores, batch size) the fewest replicas that sustain
        //    lambda; those that fit the budget go to ckey/cidx, compacted, and into the bins
        const int h_lo = p.vertical ? rep[s] : 1;
        const uint32_t *Q_s = Q + (p.vertical ? s * NB : 0);
        const uint32_t *Lmax_s = Lmax + (p.vertical ? s * NB : 0);
        int n_live = 0;
        for (int e = lane; e < L.cb; e += 32) {            // e = (c - 1) * NB + bi
            uint32_t key = kNone, idx = 0u;
            if (e < CB) {
                const int c1 = NB > 1 ? (int)__umulhi((uint32_t)e, nb_magic) : e;
                const int bi = e - c1 * NB;
                const int32_t l_us = (int32_t)latb[TH_IDX(603, e, L.cb)];
                const int32_t l_prev = e >= NB ? (int32_t)latb[TH_IDX(604, e - NB, L.cb)] : 0;   // one core fewer
                if (l_us <= 0) saw_bad_latency = 1;
                // ceil(l / w): the reciprocal's quotient is the true one or one below it
                // (l < 2^31, so the error of l * floor((2^32 - 1) / w) / 2^32 stays below 1/2)
                uint32_t l_q = __umulhi((uint32_t)l_us, w_magic);
                uint32_t l_r = (uint32_t)l_us - l_q * w_us;
                if (l_r >= w_us) { l_r -= w_us; ++l_q; }
                const uint32_t l_b = l_q + (l_r != 0u);
                // same latency with one core fewer: same buckets at a lower cost
                if (l_us > 0 && l_us != l_prev && l_b <= (uint32_t)T) {
                    const uint32_t *lmax_row = Lmax_s + bi * HN;
                    int k = 0;
                    if (HN > 1) {
                        // fewest replicas: about l * lambda / (b * 1e9); the estimate is taken one
                        // low and settled on the exact table, two steps up at most as a rule
                        const float need = (float)l_us * rate_b[TH_IDX(605, bi, THEMIS_MAX_BATCH_SIZES)] - (float)h_lo;
                        k = min(max(__float2int_rz(need) - 1, 0), HN - 1);   // the conversion saturates
                        k += (uint32_t)l_us > lmax_row[TH_IDX(606, k, HN)];
                        k = min(k, HN - 1);
                        k += (uint32_t)l_us > lmax_row[TH_IDX(607, k, HN)];
                        if (k > 0 && k < HN && (uint32_t)l_us <= lmax_row[TH_IDX(608, k - 1, HN)]) k = 0;   // estimate too high
                    }
                    while (k < HN && (uint32_t)l_us > lmax_row[TH_IDX(609, k, HN)]) ++k;
                    if (k < HN) {                          // else no replica count sustains lambda
                        const uint32_t ell = l_b + Q_s[TH_IDX(610, bi * HN + k, NB * HN)];
                        if (ell <= (uint32_t)T) {
                            key = (((uint32_t)(h_lo + k) * (uint32_t)(c1 + 1)) << kIdxBits) | ell;
                            idx = (uint32_t)(k * CB + e);
                            atomicMin(&bins[TH_IDX(611, (ell * bin_scale) >> 16, kBins)], key);
                        }
                    }
                }
            }
            const unsigned live = __ballot_sync(0xFFFFFFFFu, key != kNone);
            if (key != kNone) {
                const int at = n_live + __popc(live & lanemask_lt);
                ckey[TH_IDX(612, at, L.cb)] = key;
                cidx[TH_IDX(613, at, L.cb)] = (uint16_t)idx;
            }
            n_live += __popc(live);
        }
        __syncwarp();
        if (s + 1 < S) prefetch_words(latb, lat + (size_t)(s + 1) * CB, CB, lane);

        // 2. bins -> cheapest word over all lower bins (lane owns kBins / 32 consecutive bins)
        {
            constexpr int kOwn = kBins / 32;
            uint32_t own[kOwn];
#pragma unroll
            for (int v = 0; v < kOwn / 4; ++v) {
                const uint4 x = *reinterpret_cast<const uint4 *>(bins + kOwn * lane + 4 * v);
                own[4 * v] = x.x; own[4 * v + 1] = x.y; own[4 * v + 2] = x.z; own[4 * v + 3] = x.w;
            }
            uint32_t inc = own[0];
#pragma unroll
            for (int i = 1; i < kOwn; ++i) inc = min(inc, own[i]);
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (lane >= d) inc = min(inc, o);
            }
            uint32_t below = __shfl_up_sync(0xFFFFFFFFu, inc, 1);
            if (lane == 0) below = kNone;
            // exclusive running minimum within the lane's own bins
#pragma unroll
            for (int i = 0; i < kOwn; ++i) {
                const uint32_t mine = own[i];
                own[i] = below;
                below = min(below, mine);
            }
#pragma unroll
            for (int v = 0; v < kOwn / 4; ++v)
                *reinterpret_cast<uint4 *>(bins + kOwn * lane + 4 * v) =
                    make_uint4(own[4 * v], own[4 * v + 1], own[4 * v + 2], own[4 * v + 3]);
        }
        __syncwarp();

        // 3. survivors: candidates no cheaper-or-equal candidate of a lower bin beats
        int n_sv = 0;
        for (int i0 = 0; i0 < n_live; i0 += 32) {
            const int i = i0 + lane;
            const uint32_t key = i < n_live ? ckey[TH_IDX(615, i, L.cb)] : kNone;
            const bool keep = key != kNone &&
                              (key >> kIdxBits) < (bins[TH_IDX(614, ((key & kLowMask) * bin_scale) >> 16, kBins)] >> kIdxBits);
            const unsigned kept = __ballot_sync(0xFFFFFFFFu, keep);
            const int at = n_sv + __popc(kept & lanemask_lt);
            if (keep && at < kMaxSurvivors) {
                skey[TH_IDX(616, at, kMaxSurvivors)] = key;
                sidx[TH_IDX(617, at, kMaxSurvivors)] = cidx[TH_IDX(618, i, L.cb)];
            }
            n_sv += __popc(kept);
        }
        if (n_sv > kMaxSurvivors) { redo = true; break; }
        __syncwarp();

        // 4. front of G_s from the survivors by repeated minimum, cheapest entry first (written
        //    from the last slot down): a step takes the smallest word among survivors below the
        //    previous entry's latency, then the lowest candidate index among equals
        int n_g = 0;
        if (n_sv <= 64) {                                  // the survivors fit two registers per lane
            const uint32_t k0 = lane < n_sv ? skey[lane] : kNone, k1 = lane + 32 < n_sv ? skey[lane + 32] : kNone;
            const uint32_t i0 = lane < n_sv ? (uint32_t)sidx[lane] : kNone;
            const uint32_t i1 = lane + 32 < n_sv ? (uint32_t)sidx[lane + 32] : kNone;
            uint32_t bound = (uint32_t)T + 1u;
            for (;;) {
                const uint32_t m = warp_min(min((k0 & kLowMask) < bound ? k0 : kNone,
                                                (k1 & kLowMask) < bound ? k1 : kNone));
                if (m == kNone) break;
                const uint32_t idx = warp_min(min(k0 == m ? i0 : kNone, k1 == m ? i1 : kNone));
                ++n_g;                                     // at most 64 survivors: the front fits its slots
                if (lane == 0) {
                    gf[TH_IDX(619, kMaxStageFront - n_g, kMaxStageFront)] = m;
                    gidx[TH_IDX(620, kMaxStageFront - n_g, kMaxStageFront)] = idx;
                }
                bound = m & kLowMask;
            }
        } else {
            uint32_t bound = (uint32_t)T + 1u;
            for (;;) {
                uint32_t mine = kNone;
                for (int i = lane; i < n_sv; i += 32) {
                    const uint32_t key = skey[TH_IDX(621, i, kMaxSurvivors)];
                    if ((key & kLowMask) < bound) mine = min(mine, key);
                }
                const uint32_t m = warp_min(mine);
                if (m == kNone) break;
                if (n_g == kMaxStageFront) { redo = true; break; }
                uint32_t idx = kNone;
                for (int i = lane; i < n_sv; i += 32)
                    if (skey[i] == m) idx = min(idx, (uint32_t)sidx[i]);
                idx = warp_min(idx);
                ++n_g;
                if (lane == 0) {
                    gf[TH_IDX(622, kMaxStageFront - n_g, kMaxStageFront)] = m;
                    gidx[TH_IDX(623, kMaxStageFront - n_g, kMaxStageFront)] = idx;
                }
                bound = m & kLowMask;
            }
        }
        if (redo) break;
        __syncwarp();
        // 5. to the workspace, ascending latency
        const size_t row = ((size_t)n * S + s) * pitch;
        for (int k = lane; k < n_g; k += 32) {
            reinterpret_cast<uint32_t *>(p.G)[TH_IDX(624, row + k, (size_t)p.prob.n_instances * S * pitch)] =
                gf[TH_IDX(625, kMaxStageFront - n_g + k, kMaxStageFront)];
            p.Garg[TH_IDX(626, row + k, (size_t)p.prob.n_instances * S * pitch)] = (uint16_t)gidx[kMaxStageFront - n_g + k];
        }
        if (lane == 0) p.A[TH_IDX(627, row, (size_t)p.prob.n_instances * S * pitch)] = (uint16_t)n_g;
        __syncwarp();
    }
    asm volatile("cp.async.wait_all;" ::: "memory");       // nothing of ours in flight when the warp leaves

    if (redo) {                                            // lists outgrown: the block kernel solves it
        if (lane == 0) {
            p.inst_flag[n] = kFlagRedo;
            p.redo_list[TH_IDX(628, atomicAdd(p.redo_count, 1), p.prob.n_instances)] = n;
        }
        return;
    }
    if (__any_sync(0xFFFFFFFFu, saw_bad_latency)) { write_bad_input(); return; }
    if (lane == 0) p.inst_flag[n] = 0;
}

// ------------------------------------------------------------------ prefix fronts

constexpr uint32_t kAbsent = 0xC0000000u;   // word of "no entry": above every real word even
                                            // after a stage entry (< 2^31) is added to it
constexpr int kBoundSearchSteps = 14;       // bisection steps of the upper-bound search

// Shared memory of one warp of prefix_fronts_kernel, in words.
struct PrefixLayout {
    int cap;        // entries of a prefix front
    int wb;         // words of the budget bitmap
    int words;      // total, a multiple of 4
};

__host__ __device__ inline PrefixLayout prefix_layout(int T, int S)
{
    PrefixLayout L;
    const int want = min(T + 1, 48 * S);
    L.cap = 64;
    while (L.cap < want && L.cap < 4096) L.cap <<= 1;
    L.wb = (T + 32) / 32;
    // two prefix fronts, an "absent" word in front of each | bitmap with running counts, an
    // empty pair in front | per stage: entry count, later stages' cheapest total, candidate
    // index, offset of the stage front in the bound search
    L.words = (2 * (L.cap + 1) + 2 * (L.wb + 1) + 4 * THEMIS_MAX_STAGES + 3) & ~3;
    return L;
}

// One (bitmap word, set bits before it) pair per 32 budgets of a prefix front; pair -1 is
// empty, so budgets below zero need no test.
struct BudgetRank {
    const uint2 *pairs;     // points at pair 0
    int wb;                 // pairs 0 .. wb - 1 (and pair -1)
    int32_t *check;         // violation record of the bounds-checked build
    // number of front entries with budget <= x, for any x >= -32
    __device__ __forceinline__ int upto(int x) const
    {
#ifdef THEMIS_CHECK_BOUNDS
        const uint2 pr = pairs[th_checked_index(701, (long long)(x >> 5) + 1, (long long)wb + 1, check) - 1];
#else
        const uint2 pr = pairs[x >> 5];
#endif
        return (int)pr.y + __popc(pr.x & (0xFFFFFFFFu >> (31 - (x & 31))));
    }
};

// Prefix front of stage s from front(F_{s-1}) (Fprev[0 .. n_prev), ascending budget, with
// Fprev[-1] = kAbsent; `rank` built on its budgets) and front(G_s) (g_row/gidx_row[0 .. n_g)
// in the workspace, ascending latency): the entries with budget below `bound` and word below
// `stop`, cheapest first, at most `limit` (<= cap) of them.  Entries are written from
// Ftop[-1] down and their records, (number of prefix entries up to the predecessor << 16 |
// candidate index), to rec (= g_row) from 0 up.  Returns the number of entries; *more is
// set when the limit cut the front short.
template <int NL>
__device__ __forceinline__ int merge_fronts(const Params &p, const uint32_t *Fprev, int n_prev, const BudgetRank &rank,
                                            uint32_t *g_row, const uint16_t *gidx_row, int n_g, uint32_t *Ftop,
                                            int bound, uint32_t stop, int limit, int lane, bool *more)
{
    (void)p; (void)n_prev;
    uint32_t gk[NL], gix[NL], cur[NL];
    int lk[NL], pp[NL];                      // list q: its latency + 1; prefix entries it may still use
#pragma unroll
    for (int q = 0; q < NL; ++q) {
        const int k = lane + 32 * q;
        const bool valid = k < n_g;
        gk[q] = valid ? g_row[TH_IDX(702, k, p.pitch)] : 0u;
        gix[q] = valid ? (uint32_t)gidx_row[TH_IDX(703, k, p.pitch)] : 0u;
        lk[q] = valid ? (int)(gk[q] & kLowMask) + 1 : 0x20000000;   // no budget reaches an absent list
    }
    __syncwarp();                            // the stage front is in registers: its row may take records
    uint32_t *rec = g_row;
    const uint32_t lanemask_lt = (1u << lane) - 1u;
    // Points list q at its last entry below the bound.  The test is made on the prefix's own
    // budget, so the sum of the two low fields never carries; a list with nothing below the
    // bound reads the absent word in front of the prefix front.
    auto settle = [&](int q, int below) {
        pp[q] = rank.upto(max(below - lk[q], -1));
        cur[q] = Fprev[TH_IDX(704, pp[q], n_prev + 1) - 1] + gk[q];
    };
#pragma unroll
    for (int q = 0; q < NL; ++q) settle(q, bound);
    int count = 0;
    uint32_t m;
    for (;;) {
        uint32_t mine = cur[0];
#pragma unroll
        for (int q = 1; q < NL; ++q) mine = min(mine, cur[q]);
        m = warp_min(mine);
        if (m >= stop || count == limit) break;
        // lowest k among the lists that offer m (list q of lane i is entry i + 32 q) writes
        bool found = false;
#pragma unroll
        for (int q = 0; q < NL; ++q) {
            const bool offer = cur[q] == m;
            const unsigned offers = __ballot_sync(0xFFFFFFFFu, offer);
            if (!found && offer && (offers & lanemask_lt) == 0u) {
                Ftop[-1 - TH_IDX(705, count, limit)] = m;
                rec[TH_IDX(706, count, p.pitch)] = ((uint32_t)pp[q] << 16) | gix[q];
            }
            found = found || offers != 0u;
        }
        ++count;
        const int below = (int)(m & kLowMask);
#pragma unroll
        for (int q = 0; q < NL; ++q) settle(q, below);
    }
    *more = m < stop;
    return count;
}

// Upper bound on the optimal total from the stage fronts alone (Lagrangian search): for a
// price mu per bucket every stage takes the entry minimising cost + mu * latency; the total
// latency falls as mu grows, and every mu whose choice fits the budget T gives a feasible
// configuration, hence an upper bound.  Bisection on log2(mu).  sf holds the stage fronts as
// (latency, cost) float pairs, stage s at off[s] .. off[s] + n_of[s]; lane i serves stages i
// and i + 32.  All stages must be non-empty and the fastest entries must fit T.
__device__ __forceinline__ uint32_t bound_from_stage_fronts(const float2 *sf, const uint32_t *off,
                                                            const uint32_t *n_of, int S, int T, int lane)
{
    auto choose = [&](float mu, int *lat_sum, int *cost_sum) {
        int lat = 0, cost = 0;
        for (int s = lane; s < S; s += 32) {
            const float2 *f = sf + off[s];
            const int n = (int)n_of[s];
            float best = 3.0e38f;
            int at = 0;
            for (int j = 0; j < n; ++j) {
                const float2 e = f[j];
                const float v = fmaf(mu, e.x, e.y);
                if (v < best) { best = v; at = j; }
            }
            lat += (int)f[at].x;
            cost += (int)f[at].y;
        }
        *lat_sum = __reduce_add_sync(0xFFFFFFFFu, lat);
        *cost_sum = __reduce_add_sync(0xFFFFFFFFu, cost);
    };
    int lat, cost;
    choose(0.0f, &lat, &cost);               // the cheapest entries: if they fit, they are optimal
    if (lat <= T) return (uint32_t)cost;
    choose(1.0e9f, &lat, &cost);             // the fastest entries (they fit)
    uint32_t best = (uint32_t)cost;
    float lo = -14.0f, hi = 18.0f;           // log2(mu): 2^18 exceeds every cost difference
    for (int it = 0; it < kBoundSearchSteps; ++it) {
        const float mid = 0.5f * (lo + hi);
        choose(exp2f(mid), &lat, &cost);
        if (lat <= T) { hi = mid; best = min(best, (uint32_t)cost); }
        else lo = mid;
    }
    return best;
}

__global__ void __launch_bounds__(kFrontWarps * 32)
prefix_fronts_kernel(const Params p)
{
    extern __shared__ __align__(16) uint32_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = blockIdx.x * (blockDim.x >> 5) + warp;
    if (n >= p.prob.n_instances) return;
    if (p.active && !p.active[n]) return;
    if (p.inst_flag[n] != 0) return;         // bad input (already reported) or handed to the block kernel
    const int T = p.T, pitch = p.pitch;
    const int S = p.prob.n_stages, C = p.prob.c_max, NB = p.prob.n_batch;
    const PrefixLayout L = prefix_layout(T, S);
    const int cap = L.cap;

    uint32_t *Fa = smem + (size_t)warp * L.words + 1;      // [-1 .. cap) prefix front, right-aligned
    uint32_t *Fb = Fa + cap + 1;                           // [-1 .. cap)
    uint2 *pairs = reinterpret_cast<uint2 *>(Fb + cap) + 1;   // [-1 .. wb) bitmap word, set bits before it
    uint32_t *n_of = reinterpret_cast<uint32_t *>(pairs + L.wb);       // [64] entries of the stage front, then of the prefix front
    uint32_t *later_cost = n_of + THEMIS_MAX_STAGES;       // [64] sum of the later stages' cheapest entries
    uint32_t *idx_of = later_cost + THEMIS_MAX_STAGES;     // [64] candidate index of the chosen entry per stage
    uint32_t *off = idx_of + THEMIS_MAX_STAGES;            // [64] bound search: where a stage front starts

    uint32_t *rec_inst = reinterpret_cast<uint32_t *>(p.G + (size_t)n * S * pitch);
    const uint16_t *gidx_inst = p.Garg + (size_t)n * S * pitch;
    const uint16_t *count_inst = p.A + (size_t)n * S * pitch;
    const BudgetRank rank{pairs, L.wb, p.check};
    int32_t *h_o = p.out.h + (size_t)n * S, *c_o = p.out.c + (size_t)n * S, *b_o = p.out.b + (size_t)n * S;
    auto write_infeasible = [&]() {
        for (int s = lane; s < S; s += 32) { h_o[s] = 0; c_o[s] = 0; b_o[s] = 0; }
        if (lane == 0) {
            p.out.total_cost[n] = -1;
            p.out.latency_buckets[n] = -1;
            p.out.status[n] = THEMIS_STATUS_INFEASIBLE;
        }
    };

    // Per stage: size of its front, its fastest and its cheapest entry (fronts ascend in
    // latency and fall in cost: entries 0 and n - 1).
    int later_min = 0, total_entries = 0;    // sum of the fastest latencies; entries of all fronts
    {
        int lmin_sum = 0, any_empty = 0;
        uint32_t cheapest[2] = {0u, 0u};
        int count[2] = {0, 0};
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int s = lane + 32 * q;
            if (s < S) {
                count[q] = (int)count_inst[(size_t)s * pitch];
                if (count[q] == 0) any_empty = 1;
                else {
                    lmin_sum += (int)(rec_inst[(size_t)s * pitch] & kLowMask);
                    cheapest[q] = rec_inst[TH_IDX(707, (size_t)s * pitch + count[q] - 1, (size_t)S * pitch)] >> kIdxBits;
                }
                n_of[s] = (uint32_t)count[q];
            }
        }
        later_min = __reduce_add_sync(0xFFFFFFFFu, lmin_sum);
        if (__any_sync(0xFFFFFFFFu, any_empty) || later_min > T) { write_infeasible(); return; }
        // exclusive prefix sums over the stages: front offsets; suffix sums: later stages' cheapest
        int inc0 = count[0], inc1 = count[1];
        uint32_t c0 = cheapest[0], c1 = cheapest[1];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int a0 = __shfl_up_sync(0xFFFFFFFFu, inc0, d), a1 = __shfl_up_sync(0xFFFFFFFFu, inc1, d);
            const uint32_t b0 = __shfl_down_sync(0xFFFFFFFFu, c0, d), b1 = __shfl_down_sync(0xFFFFFFFFu, c1, d);
            if (lane >= d) { inc0 += a0; inc1 += a1; }
            if (lane + d < 32) { c0 += b0; c1 += b1; }
        }
        const int first32 = __shfl_sync(0xFFFFFFFFu, inc0, 31);
        const uint32_t upper32 = __shfl_sync(0xFFFFFFFFu, c1, 0);        // cheapest of stages 32..63
        total_entries = first32 + __shfl_sync(0xFFFFFFFFu, inc1, 31);
        if (lane < S) { off[lane] = (uint32_t)(inc0 - count[0]); later_cost[lane] = c0 - cheapest[0] + upper32; }
        if (lane + 32 < S) { off[lane + 32] = (uint32_t)(first32 + inc1 - count[1]); later_cost[lane + 32] = c1 - cheapest[1]; }
    }
    __syncwarp();
    later_min -= (int)(rec_inst[0] & kLowMask);            // now the sum over the stages after stage 0

    // Upper bound on the optimal total (when the stage fronts fit the scratch: both prefix
    // front buffers are free now).  A state of stages 0..s whose total plus the later stages'
    // cheapest entries exceeds it cannot be part of an optimal configuration.
    uint32_t upper = 0x7FFFFFFFu >> kIdxBits;
    if (S > 1 && 2 * total_entries <= 2 * (cap + 1)) {
        float2 *sf = reinterpret_cast<float2 *>(Fa - 1);
        for (int s = 0; s < S; ++s) {
            const uint32_t *g_row = rec_inst + (size_t)s * pitch;
            for (int k = lane; k < (int)n_of[s]; k += 32) {
                const uint32_t w = g_row[k];
                sf[TH_IDX(708, off[s] + k, cap + 1)] = make_float2((float)(w & kLowMask), (float)(w >> kIdxBits));
            }
        }
        __syncwarp();
        upper = bound_from_stage_fronts(sf, off, n_of, S, T, lane);
        __syncwarp();
    }

    bool redo = false;
    int n_prev = 0;
    uint32_t *Fprev = Fa, *Fcur = Fb;
    for (int s = 0; s < S; ++s) {
        uint32_t *g_row = rec_inst + (size_t)s * pitch;
        const uint16_t *gidx_row = gidx_inst + (size_t)s * pitch;
        const int n_g = (int)n_of[s];
        if (s > 0) later_min -= (int)(g_row[0] & kLowMask);   // now the sum over the stages after s
        // Budgets that can still be completed lie below `bound`: the fastest entries of the later
        // stages must fit.  Words that can still be optimal lie below `stop`.
        const int bound = T + 1 - later_min;
        const uint32_t spare = upper - min(upper, later_cost[s]);
        const uint32_t stop = min(0x80000000u, (spare + 1u) << kIdxBits);
        int n_cur = 0;
        bool more = false;
        __syncwarp();
        if (s == 0) {
            // the first stage's front is the first prefix front: its entries below bound and stop
            constexpr int kLists = kMaxStageFront / 32;
            uint32_t gk[kLists], gix[kLists];
            int n_fit = 0, first = 0;
#pragma unroll
            for (int q = 0; q < kLists; ++q) {
                const int k = lane + 32 * q;
                gk[q] = k < n_g ? g_row[k] : kNone;
                gix[q] = k < n_g ? (uint32_t)gidx_row[k] : 0u;
                const unsigned fit =
                    __ballot_sync(0xFFFFFFFFu, k < n_g && (int)(gk[q] & kLowMask) < bound && gk[q] < stop);
                // the front ascends in latency and falls in cost: the fitting entries are contiguous
                if (n_fit == 0 && fit != 0u) first = 32 * q + __ffs((int)fit) - 1;
                n_fit += __popc(fit);
            }
            __syncwarp();
#pragma unroll
            for (int q = 0; q < kLists; ++q) {
                const int k = lane + 32 * q - first;
                if (k >= 0 && k < n_fit) {
                    Fcur[TH_IDX(709, cap - n_fit + k, cap)] = gk[q];
                    g_row[TH_IDX(710, n_fit - 1 - k, pitch)] = gix[q];
                }
            }
            n_cur = n_fit;
        } else {
            // the last stage only has to yield its cheapest entry: the answer
            const int limit = s == S - 1 ? 1 : cap;
            uint32_t *Ftop = Fcur + cap;
            const uint32_t *Fp = Fprev + (cap - n_prev);
            n_cur = n_g <= 32 ? merge_fronts<1>(p, Fp, n_prev, rank, g_row, gidx_row, n_g, Ftop, bound, stop, limit, lane, &more)
                  : n_g <= 64 ? merge_fronts<2>(p, Fp, n_prev, rank, g_row, gidx_row, n_g, Ftop, bound, stop, limit, lane, &more)
                              : merge_fronts<kMaxStageFront / 32>(p, Fp, n_prev, rank, g_row, gidx_row, n_g, Ftop, bound, stop,
                                                                  limit, lane, &more);
            if (more && s < S - 1) { redo = true; break; }
        }
        __syncwarp();
        if (lane == 0) n_of[s] = (uint32_t)n_cur;         // from here on: entries of the prefix front
        uint32_t *tmp = Fprev; Fprev = Fcur; Fcur = tmp;
        n_prev = n_cur;
        if (n_prev == 0) break;              // cannot happen while the bound is an upper bound

        // bitmap of the new front's budgets and the running counts, for the next stage
        if (s + 1 < S) {
            if (lane == 0) { Fprev[TH_IDX(711, cap - n_prev, cap + 1) - 1] = kAbsent; pairs[-1] = make_uint2(0u, 0u); }
            for (int w = lane; w < L.wb; w += 32) pairs[w].x = 0u;
            __syncwarp();
            for (int i = lane; i < n_prev; i += 32) {
                const uint32_t t = Fprev[TH_IDX(712, cap - n_prev + i, cap)] & kLowMask;
                atomicOr(&pairs[TH_IDX(713, t >> 5, L.wb)].x, 1u << (t & 31));
            }
            __syncwarp();
            uint32_t carry = 0;
            for (int w0 = 0; w0 < L.wb; w0 += 32) {
                const int w = w0 + lane;
                const uint32_t c = w < L.wb ? (uint32_t)__popc(pairs[w].x) : 0u;
                uint32_t inc = c;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                    if (lane >= d) inc += o;
                }
                if (w < L.wb) pairs[w].y = carry + inc - c;
                carry += __shfl_sync(0xFFFFFFFFu, inc, 31);
            }
            __syncwarp();
        }
    }

    if (redo) {                                            // front outgrown: the block kernel solves it
        if (lane == 0) {
            p.inst_flag[n] = kFlagRedo;
            p.redo_list[TH_IDX(716, atomicAdd(p.redo_count, 1), p.prob.n_instances)] = n;
        }
        return;
    }
    if (n_prev == 0) { write_infeasible(); return; }
    // The last entry is the cheapest total at the lowest budget that reaches it; its
    // record is number 0 of the last stage.  Lane 0 walks the records (a record names its
    // predecessor by the number of entries up to it, counted from the lowest budget; records
    // are stored from the highest budget down), then the lanes turn candidate indices into
    // configurations.
    const uint32_t best = Fprev[cap - 1];
    if (lane == 0) {
        uint32_t q = 0;
        for (int s = S - 1; s >= 0; --s) {
            const uint32_t r = rec_inst[TH_IDX(714, (size_t)s * pitch + q, (size_t)S * pitch)];
            idx_of[TH_IDX(715, s, THEMIS_MAX_STAGES)] = r & 0xFFFFu;
            if (s > 0) q = n_of[s - 1] - (r >> 16);
        }
        p.out.total_cost[n] = (int32_t)(best >> kIdxBits);
        p.out.latency_buckets[n] = (int32_t)(best & kLowMask);
        p.out.status[n] = THEMIS_STATUS_OK;
    }
    __syncwarp();
    for (int s = lane; s < S; s += 32) {
        const int idx = (int)idx_of[s];
        const int bi = idx % NB, rest = idx / NB;
        b_o[s] = p.prob.batch_sizes[bi];
        c_o[s] = rest % C + 1;
        h_o[s] = p.vertical ? p.replicas[(size_t)n * S + s] : rest / C + 1;
    }
}

StageLayout stage_layout_of(const Params &p)
{
    return stage_layout(p.prob.c_max, p.prob.n_batch, p.vertical ? 1 : p.prob.h_max,
                        p.vertical ? p.prob.n_stages : 1);
}

}  // namespace

bool front_kernel_fits(const Params &p)
{
    return warps_per_block(sizeof(uint32_t) * (size_t)stage_layout_of(p).words) > 0 &&
           warps_per_block(sizeof(uint32_t) * (size_t)prefix_layout(p.T, p.prob.n_stages).words) > 0;
}

cudaError_t launch_solve_front(const Params &p, cudaStream_t stream)
{
    static std::atomic<uint64_t> stage_ready{0}, prefix_ready{0};
    const int N = p.prob.n_instances;
    {
        const size_t warp_bytes = sizeof(uint32_t) * (size_t)stage_layout_of(p).words;
        const int warps = warps_per_block(warp_bytes);
        cudaError_t e = allow_max_smem(reinterpret_cast<const void *>(stage_fronts_kernel), stage_ready);
        if (e != cudaSuccess) return e;
        stage_fronts_kernel<<<(N + warps - 1) / warps, warps * 32, warp_bytes * warps, stream>>>(p);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    const size_t warp_bytes = sizeof(uint32_t) * (size_t)prefix_layout(p.T, p.prob.n_stages).words;
    const int warps = warps_per_block(warp_bytes);
    cudaError_t e = allow_max_smem(reinterpret_cast<const void *>(prefix_fronts_kernel), prefix_ready);
    if (e != cudaSuccess) return e;
    prefix_fronts_kernel<<<(N + warps - 1) / warps, warps * 32, warp_bytes * warps, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace themis

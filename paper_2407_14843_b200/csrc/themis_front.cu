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
// entry: cost << 14 | latency (a stage) or total << 14 | budget (a prefix).  Both steps of
// a stage build their front from its cheapest entry down by repeated minimum:
//  * stage front: every lane keeps its candidates in registers; a step takes the smallest
//    word among candidates below the previous entry's latency (one warp reduction, a
//    second one for the lowest candidate index among equals);
//  * prefix front: lane k owns the list "front(F_{s-1}) shifted by entry k of front(G_s)",
//    itself sorted with falling cost, so its best entry below a budget bound is the last
//    one below it: a pointer that only moves down.  A step is one warp reduction over the
//    lanes' current words, the lowest k among equals wins (lowest stage latency), and the
//    pointers of the lists that reach the new bound move on.
// Every step yields one entry, so a stage costs about |front(G_s)| + |front(F_s)| steps of a
// few instructions.  The workspace receives one record per prefix entry,
// (position of its predecessor << 16 | candidate index), in the order found, i.e. from the
// cheapest entry down; the backtrack starts at record 0 of the last stage.
//
// Capacities are fixed per launch (stage front: 64 entries, two lists per lane; prefix
// front: `cap` entries of shared memory).  An instance that outgrows them is appended to
// the redo list and solved by the block-per-instance kernel afterwards.
#include "themis_internal.h"

namespace themis {
namespace {

constexpr int kFrontWarps = 4;          // instances per block; warps never wait for each other
constexpr int kMaxStageFront = 64;      // entries of a stage's front: two lists per lane
constexpr int kMaxSlots = 32;           // candidate slots per lane: c_max * n_batch <= 1024
constexpr uint32_t kNone = 0xFFFFFFFFu;
constexpr uint32_t kLowMask = kIdxMask; // latency / budget field of a packed entry

__device__ __forceinline__ uint32_t sat_u32(unsigned long long v, uint32_t cap)
{
    return v > (unsigned long long)cap ? cap : (uint32_t)v;
}

__device__ __forceinline__ uint32_t warp_min(uint32_t v) { return __reduce_min_sync(0xFFFFFFFFu, v); }

// Shared memory of one warp, in words.
struct FrontLayout {
    int cap;        // entries of a prefix front
    int tab;        // entries of Q and of Lmax
    int words;      // total, a multiple of 4
};

__host__ __device__ inline FrontLayout front_layout(int T, int S, int NB, int HN, int SV)
{
    FrontLayout L;
    const int want = min(T + 1, 128 * S);
    L.cap = 64;
    while (L.cap < want && L.cap < 2048) L.cap <<= 1;
    L.tab = SV * NB * HN;
    L.words = (2 * L.cap + 2 * kMaxStageFront + THEMIS_MAX_BATCH_SIZES + 2 * L.tab + 3) & ~3;
    return L;
}

// Prefix front of stage s from front(F_{s-1}) (Fprev[base .. base + n_prev), ascending
// budget) and front(G_s) (gf/gidx[0 .. n_g), ascending latency).  Entries are written to
// Fcur from position cap - 1 down and their records to rec from 0 up.  Returns the number
// of entries, or -1 when more than cap would be needed.
template <int NL>
__device__ __forceinline__ int merge_fronts(const uint32_t *Fprev, int base, int n_prev, const uint32_t *gf,
                                            const uint32_t *gidx, int n_g, uint32_t *Fcur, int cap,
                                            uint32_t *rec, int T, int lane)
{
    uint32_t gk[NL], gix[NL], cur[NL];
    int pp[NL];                              // entries of list q still below the bound
#pragma unroll
    for (int q = 0; q < NL; ++q) {
        const int k = lane + 32 * q;
        const bool valid = k < n_g;
        gk[q] = valid ? gf[k] : 0u;
        gix[q] = valid ? gidx[k] : 0u;
        pp[q] = valid ? n_prev : 0;
        cur[q] = kNone;
    }
    uint32_t bound = (uint32_t)T + 1u;       // budgets of the entries still to come lie below it
    // Moves list q's pointer to its last entry below the bound.  The comparison is made on
    // the prefix's own budget so that the sum of the two low fields never carries.
    auto settle = [&](int q) {
        const int lim = (int)bound - 1 - (int)(gk[q] & kLowMask);
        while (pp[q] > 0 && (int)(Fprev[base + pp[q] - 1] & kLowMask) > lim) --pp[q];
        cur[q] = pp[q] > 0 ? Fprev[base + pp[q] - 1] + gk[q] : kNone;
    };
#pragma unroll
    for (int q = 0; q < NL; ++q)
        if (pp[q] > 0) settle(q);
    int pos = cap;
    for (;;) {
        uint32_t mine = cur[0];
#pragma unroll
        for (int q = 1; q < NL; ++q) mine = min(mine, cur[q]);
        const uint32_t m = warp_min(mine);
        if (m == kNone) break;
        if (pos == 0) return -1;
        --pos;
        // lowest k among the lists that offer m: list q of lane i is entry i + 32 q
        int q_win = 0;
        unsigned winners = __ballot_sync(0xFFFFFFFFu, cur[0] == m);
#pragma unroll
        for (int q = 1; q < NL; ++q)
            if (winners == 0u) {             // warp-uniform
                winners = __ballot_sync(0xFFFFFFFFu, cur[q] == m);
                q_win = q;
            }
        if (lane == __ffs((int)winners) - 1) {
#pragma unroll
            for (int q = 0; q < NL; ++q)
                if (q == q_win) {
                    Fcur[pos] = m;
                    rec[cap - 1 - pos] = ((uint32_t)(n_prev - pp[q]) << 16) | gix[q];
                }
        }
        bound = m & kLowMask;
#pragma unroll
        for (int q = 0; q < NL; ++q)
            if (pp[q] > 0 && (cur[q] & kLowMask) >= bound) settle(q);
    }
    return cap - pos;
}

// J: candidate slots per lane (c_max * n_batch <= 32 * J).
template <int J>
__global__ void __launch_bounds__(kFrontWarps * 32)
solve_front_kernel(const Params p)
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
    const FrontLayout L = front_layout(T, S, NB, HN, SV);
    const int cap = L.cap;

    uint32_t *Fprev = smem + (size_t)warp * L.words;      // [cap] prefix front, right-aligned
    uint32_t *Fcur = Fprev + cap;                          // [cap]
    uint32_t *gf = Fcur + cap;                             // [64] stage front: cost << 14 | latency
    uint32_t *gidx = gf + kMaxStageFront;                  // [64] ... and candidate index
    float *rate_b = reinterpret_cast<float *>(gidx + kMaxStageFront);   // [16] lambda / (b * 1e9)
    uint32_t *Q = reinterpret_cast<uint32_t *>(rate_b) + THEMIS_MAX_BATCH_SIZES;   // [SV][NB][HN]
    uint32_t *Lmax = Q + L.tab;                            // [SV][NB][HN]

    const uint32_t lambda_m = p.lambda_mrps[n];
    const int pid = p.profile_id ? p.profile_id[n] : 0;
    const int32_t *rep = p.vertical ? p.replicas + (size_t)n * S : nullptr;
    int32_t *h_o = p.out.h + (size_t)n * S, *c_o = p.out.c + (size_t)n * S, *b_o = p.out.b + (size_t)n * S;
    auto write_unsolved = [&](int status) {
        for (int s = lane; s < S; s += 32) { h_o[s] = 0; c_o[s] = 0; b_o[s] = 0; }
        if (lane == 0) {
            p.out.total_cost[n] = -1;
            p.out.latency_buckets[n] = -1;
            p.out.status[n] = status;
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
        if (__any_sync(0xFFFFFFFFu, bad)) {
            write_unsolved(THEMIS_STATUS_BAD_INPUT);
            if (lane == 0) p.inst_flag[n] = kFlagBadInput;
            return;
        }
    }
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
            Q[e] = sat_u32((q_num + q_den - 1ull) / q_den, (uint32_t)T + 1u);
            Lmax[e] = sat_u32(h * b * 1000000000ull / lambda_m, 0x7FFFFFFFu);
        }
        if (lane < NB) rate_b[lane] = (float)lambda_m / ((float)p.prob.batch_sizes[lane] * 1.0e9f);
    }
    __syncwarp();

    const int32_t *lat = p.lat_us + (size_t)pid * S * CB;
    const uint32_t w_magic = 0xFFFFFFFFu / w_us;
    const uint32_t nb_magic = NB > 1 ? 0xFFFFFFFFu / (uint32_t)NB + 1u : 0u;   // e / NB for e < 2^16
    uint32_t *rec_inst = reinterpret_cast<uint32_t *>(p.G + (size_t)n * S * pitch);
    int saw_bad_latency = 0;
    bool redo = false;
    int n_prev = 0;

    for (int s = 0; s < S; ++s) {
        // 1. candidates of stage s: per (cores, batch size) the fewest replicas that sustain lambda
        const int h_lo = p.vertical ? rep[s] : 1;
        const int32_t *lat_s = lat + (size_t)s * CB;
        const uint32_t *Q_s = Q + (p.vertical ? s * NB : 0);
        const uint32_t *Lmax_s = Lmax + (p.vertical ? s * NB : 0);
        uint32_t ck[J], ci[J];
#pragma unroll
        for (int j = 0; j < J; ++j) {
            const int e = lane + 32 * j;                   // (c - 1) * NB + bi
            ck[j] = kNone;
            ci[j] = 0u;
            if (e >= CB) continue;
            const int c1 = NB > 1 ? (int)__umulhi((uint32_t)e, nb_magic) : e;
            const int bi = e - c1 * NB;
            const int32_t l_us = lat_s[e];
            if (l_us <= 0) { saw_bad_latency = 1; continue; }
            if (c1 > 0 && lat_s[e - NB] == l_us) continue;   // same buckets, cheaper, one core fewer
            uint32_t l_q = __umulhi((uint32_t)l_us, w_magic);
            uint32_t l_r = (uint32_t)l_us - l_q * w_us;
            while (l_r >= w_us) { l_r -= w_us; ++l_q; }
            const uint32_t l_b = l_q + (l_r != 0u);
            if (l_b > (uint32_t)T) continue;
            const uint32_t *lmax_row = Lmax_s + bi * HN;
            int k = 0;
            if (HN > 1) {
                const float need = (float)l_us * rate_b[bi] - (float)h_lo;
                k = max((int)fminf(fmaxf(need, 0.0f), (float)HN) - 1, 0);
                if (k > 0 && (uint32_t)l_us <= lmax_row[k - 1]) k = 0;
            }
            while (k < HN && (uint32_t)l_us > lmax_row[k]) ++k;
            if (k >= HN) continue;                         // no replica count sustains lambda
            const uint32_t ell = l_b + Q_s[bi * HN + k];
            if (ell > (uint32_t)T) continue;
            ck[j] = (((uint32_t)(h_lo + k) * (uint32_t)(c1 + 1)) << kIdxBits) | ell;
            ci[j] = (uint32_t)(k * CB + e);
        }

        // 2. front of G_s, cheapest entry first, written from slot 63 down
        int n_g = 0;
        {
            uint32_t bound = (uint32_t)T + 1u;
            for (;;) {
                uint32_t mine = kNone;
#pragma unroll
                for (int j = 0; j < J; ++j)
                    if ((ck[j] & kLowMask) < bound) mine = min(mine, ck[j]);
                const uint32_t m = warp_min(mine);
                if (m == kNone) break;
                if (n_g == kMaxStageFront) { redo = true; break; }
                uint32_t idx = kNone;
#pragma unroll
                for (int j = 0; j < J; ++j)
                    if (ck[j] == m) idx = min(idx, ci[j]);
                idx = warp_min(idx);
                ++n_g;
                if (lane == 0) {
                    gf[kMaxStageFront - n_g] = m;
                    gidx[kMaxStageFront - n_g] = idx;
                }
                bound = m & kLowMask;
            }
        }
        if (redo) break;
        __syncwarp();

        // 3. front of F_s
        uint32_t *rec = rec_inst + (size_t)s * pitch;
        const uint32_t *gf_s = gf + (kMaxStageFront - n_g), *gidx_s = gidx + (kMaxStageFront - n_g);
        int n_cur;
        if (s == 0) {
            for (int k = lane; k < n_g; k += 32) {
                Fcur[cap - n_g + k] = gf_s[k];
                rec[n_g - 1 - k] = gidx_s[k];
            }
            n_cur = n_g;
        } else if (n_g <= 32) {
            n_cur = merge_fronts<1>(Fprev, cap - n_prev, n_prev, gf_s, gidx_s, n_g, Fcur, cap, rec, T, lane);
        } else {
            n_cur = merge_fronts<2>(Fprev, cap - n_prev, n_prev, gf_s, gidx_s, n_g, Fcur, cap, rec, T, lane);
        }
        if (n_cur < 0) { redo = true; break; }
        __syncwarp();
        uint32_t *tmp = Fprev; Fprev = Fcur; Fcur = tmp;
        n_prev = n_cur;
    }

    if (redo) {                                            // lists outgrown: the block kernel solves it
        if (lane == 0) p.redo_list[atomicAdd(p.redo_count, 1)] = n;
        return;
    }
    if (__any_sync(0xFFFFFFFFu, saw_bad_latency)) {
        write_unsolved(THEMIS_STATUS_BAD_INPUT);
        if (lane == 0) p.inst_flag[n] = kFlagBadInput;
        return;
    }
    if (lane == 0) p.inst_flag[n] = 0;
    if (n_prev == 0) { write_unsolved(THEMIS_STATUS_INFEASIBLE); return; }

    // The last entry is the cheapest total at the lowest budget that reaches it; its
    // record is number 0 of the last stage.  Lane 0 walks the records, then the lanes
    // turn candidate indices into configurations.
    const uint32_t best = Fprev[cap - 1];
    if (lane == 0) {
        uint32_t q = 0;
        for (int s = S - 1; s >= 0; --s) {
            const uint32_t r = rec_inst[(size_t)s * pitch + q];
            gidx[s] = r & 0xFFFFu;
            q = r >> 16;
        }
        p.out.total_cost[n] = (int32_t)(best >> kIdxBits);
        p.out.latency_buckets[n] = (int32_t)(best & kLowMask);
        p.out.status[n] = THEMIS_STATUS_OK;
    }
    __syncwarp();
    for (int s = lane; s < S; s += 32) {
        const int idx = (int)gidx[s];
        const int bi = idx % NB, rest = idx / NB;
        b_o[s] = p.prob.batch_sizes[bi];
        c_o[s] = rest % C + 1;
        h_o[s] = p.vertical ? rep[s] : rest / C + 1;
    }
}

template <int J>
cudaError_t launch_front_variant(const Params &p, int warps, size_t smem, cudaStream_t stream)
{
    static std::atomic<uint64_t> ready{0};
    cudaError_t e = allow_max_smem(reinterpret_cast<const void *>(solve_front_kernel<J>), ready);
    if (e != cudaSuccess) return e;
    const int blocks = (p.prob.n_instances + warps - 1) / warps;
    solve_front_kernel<J><<<blocks, warps * 32, smem, stream>>>(p);
    return cudaGetLastError();
}

FrontLayout layout_of_params(const Params &p)
{
    const int HN = p.vertical ? 1 : p.prob.h_max;
    const int SV = p.vertical ? p.prob.n_stages : 1;
    return front_layout(p.T, p.prob.n_stages, p.prob.n_batch, HN, SV);
}

}  // namespace

bool front_kernel_fits(const Params &p)
{
    if (p.prob.c_max * p.prob.n_batch > 32 * kMaxSlots) return false;
    return sizeof(uint32_t) * (size_t)layout_of_params(p).words <= kMaxDynamicSmem;
}

cudaError_t launch_solve_front(const Params &p, cudaStream_t stream)
{
    const FrontLayout L = layout_of_params(p);
    const size_t warp_bytes = sizeof(uint32_t) * (size_t)L.words;
    // warps per block: the count that lets most warps share an SM's shared memory (227 KB,
    // 1 KB reserved per block, at most 32 blocks), the larger block among equals
    int warps = 1, best = 0;
    for (int w = 1; w <= kFrontWarps; ++w) {
        if (w * warp_bytes > kMaxDynamicSmem) break;
        size_t blocks = (227u * 1024u) / (w * warp_bytes + 1024u);
        if (blocks > 32) blocks = 32;
        if ((int)(blocks * w) >= best) { best = (int)(blocks * w); warps = w; }
    }
    const size_t smem = warp_bytes * warps;
    const int slots = (p.prob.c_max * p.prob.n_batch + 31) / 32;
    if (slots <= 2) return launch_front_variant<2>(p, warps, smem, stream);
    if (slots <= 4) return launch_front_variant<4>(p, warps, smem, stream);
    if (slots <= 8) return launch_front_variant<8>(p, warps, smem, stream);
    if (slots <= 16) return launch_front_variant<16>(p, warps, smem, stream);
    return launch_front_variant<32>(p, warps, smem, stream);
}

}  // namespace themis

// Whole solver in one kernel on undominated entries only: candidate scoring, per-stage
// fronts and the stage recurrence, with no dense table leaving the SM.
//
// Two exchange arguments (costs are non-negative, budgets only shrink):
//  * a stage entry (l, cost) is dominated when a smaller l' has cost' <= cost;
//  * a prefix state (t, total) of stages 0..s is dominated when a smaller t' has total' <= total.
// Swapping a dominated entry or prefix for its dominator lowers the total latency
// without raising the cost, so the solution the solver returns (cheapest, then
// lowest total latency, then lowest stage latencies from the last stage down, then
// lowest candidate indices) contains neither.  Hence
//  * per (cores, batch size) only the fewest replicas that sustain lambda can matter
//    (more replicas cost more and never shorten the latency): K / h_max candidates;
//  * the recurrence F_s[t] = min_l F_{s-1}[t-l] + G_s[l] (Algorithm 1's budget loop)
//    only has to combine the front of F_{s-1} with the front of G_s: a few thousand
//    pairs per stage instead of (T+1)(T+2)/2 cells.
// Returned configurations, costs, latencies and statuses equal those of the dense
// kernels; the workspace holds the fronts instead of the dense tables:
//   G    rows: entry k of stage s's front as (l << 16 | candidate index)
//   Garg rows: its cost;   A rows: A[s][t] = k for every front cell t of F_s.
//
// One block per instance.  Per stage: candidates -> shared-memory atomic min on
// (cost << 16 | idx) per bucket; block scan -> front of G_s; front(F_{s-1}) x front(G_s)
// -> atomic min on (total << 14 | k) per budget cell; block scan -> front of F_s.
#include "themis_internal.h"

namespace themis {
namespace {

constexpr uint32_t kEmpty = 0xFFFFFFFFu;

__device__ __forceinline__ uint32_t sat_u32(unsigned long long v, uint32_t cap)
{
    return v > (unsigned long long)cap ? cap : (uint32_t)v;
}

// Exclusive prefix over the block in thread order (min or add).  Two barriers.
template <bool IS_MIN>
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t identity, uint32_t *warp_tot, int tid)
{
    const int lane = tid & 31, warp = tid >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc = IS_MIN ? min(inc, o) : inc + o;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    uint32_t before = identity;
    for (int w = 0; w < warp; ++w) before = IS_MIN ? min(before, warp_tot[w]) : before + warp_tot[w];
    uint32_t exc = __shfl_up_sync(0xFFFFFFFFu, inc, 1);
    if (lane == 0) exc = identity;
    __syncthreads();
    return IS_MIN ? min(before, exc) : before + exc;
}

// Front of a row of packed keys (cost in the bits above SHIFT, kEmpty = no entry):
// the entries whose cost is below every cost at a smaller index.  emit(pos, index, key)
// is called for each, pos counting from 0 in ascending index order; the row is left
// empty.  Returns the number of front entries.
template <int SHIFT, int kThreads, class Emit>
__device__ __forceinline__ int front_of_row(const Params &p, uint32_t *row, int n_entries, int seg,
                                            uint32_t *warp_tot, uint32_t *s_total, int tid, Emit emit)
{
    (void)p;
    constexpr uint32_t kBig = 0xFFFFFFFFu;
    const int l0 = tid * seg, l1 = min(l0 + seg, n_entries);
    uint32_t local_min = kBig;
    for (int l = l0; l < l1; ++l) {
        const uint32_t key = row[l];
        if (key != kEmpty) local_min = min(local_min, key >> SHIFT);
    }
    const uint32_t before = block_exclusive_scan<true>(local_min, kBig, warp_tot, tid);
    uint32_t running = before, count = 0;
    for (int l = l0; l < l1; ++l) {
        const uint32_t key = row[l];
        if (key != kEmpty && (key >> SHIFT) < running) { running = key >> SHIFT; ++count; }
    }
    uint32_t pos = block_exclusive_scan<false>(count, 0u, warp_tot, tid);
    running = before;
    for (int l = l0; l < l1; ++l) {
        const uint32_t key = row[TH_IDX(501, l, p.pitch)];
        row[l] = kEmpty;
        if (key != kEmpty && (key >> SHIFT) < running) { running = key >> SHIFT; emit((int)pos++, l, key); }
    }
    if (tid == kThreads - 1) *s_total = pos;
    __syncthreads();
    return (int)*s_total;
}

// One instance, solved by the whole block.
template <int kThreads>
__device__ __forceinline__ void solve_instance_sparse(const Params &p, const int n, uint32_t *smem)
{
    constexpr int kWarps = kThreads / 32;
    if (p.active && !p.active[n]) return;
    const int tid = threadIdx.x;
    const int T = p.T, pitch = p.pitch;
    const int S = p.prob.n_stages, C = p.prob.c_max, NB = p.prob.n_batch;
    const int CB = C * NB;
    const int HN = p.vertical ? 1 : p.prob.h_max;
    const int SV = p.vertical ? S : 1;
    const uint32_t w_us = (uint32_t)p.prob.bucket_us;
    const int seg = ((pitch + kThreads - 1) / kThreads) | 1;   // odd: segments start in distinct banks
    const int cap_g = min(pitch, CB);                          // one candidate per (c, b) at most

    // One key row serves both reductions in turn (each scan leaves it empty):
    // cost << 16 | idx per bucket while scoring, total << 14 | k per budget cell while pairing.
    uint32_t *keys_g = smem;                    // [pitch]
    uint32_t *keys_f = keys_g;
    uint32_t *ff_t = keys_g + pitch;            // [pitch]  front of the prefix: budget ...
    uint32_t *ff_c = ff_t + pitch;              // [pitch]  ... and total cost
    uint32_t *gf_l = ff_c + pitch;              // [cap_g]  front of the stage: latency ...
    uint32_t *gf_c = gf_l + cap_g;              // [cap_g]  ... and cost
    uint32_t *Q = gf_c + cap_g;                 // [SV][NB][HN]
    uint32_t *Lmax = Q + SV * NB * HN;          // [SV][NB][HN]
    uint32_t *warp_tot = Lmax + SV * NB * HN;   // [32]
    __shared__ uint32_t s_total;
    __shared__ int s_bad;

    const uint32_t lambda_m = p.lambda_mrps[TH_IDX(502, n, p.prob.n_instances)];
    const int pid = p.profile_id ? p.profile_id[n] : 0;
    const int32_t *lat = p.lat_us + (size_t)pid * S * CB;
    const int tab = SV * NB * HN;
    (void)tab;
    const int32_t *rep = p.vertical ? p.replicas + (size_t)n * S : nullptr;
    int32_t *h_o = p.out.h + (size_t)n * S, *c_o = p.out.c + (size_t)n * S, *b_o = p.out.b + (size_t)n * S;
    auto write_unsolved = [&](int status) {
        for (int s = 0; s < S; ++s) { h_o[s] = 0; c_o[s] = 0; b_o[s] = 0; }
        p.out.total_cost[n] = -1;
        p.out.latency_buckets[n] = -1;
        p.out.status[n] = status;
    };

    if (tid == 0) {
        int bad = (lambda_m == 0) || pid < 0 || pid >= p.prob.n_profiles;
        if (rep) {
            long long total = 0;
            for (int s = 0; s < S; ++s) {
                if (rep[s] < 1 || (long long)rep[s] * C > 65535) bad = 1;
                total += (long long)rep[s] * C;
            }
            if (total > THEMIS_MAX_TOTAL_COST) bad = 1;
        }
        s_bad = bad;
    }
    for (int l = tid; l < pitch; l += kThreads) keys_g[l] = kEmpty;
    __syncthreads();
    if (s_bad) {
        if (tid == 0) { write_unsolved(THEMIS_STATUS_BAD_INPUT); p.inst_flag[n] = kFlagBadInput; }
        return;
    }
    {
        const unsigned long long q_den = (unsigned long long)lambda_m * w_us;
        for (int e = tid; e < SV * NB * HN; e += kThreads) {
            const int sv = e / (NB * HN);
            const int bi = (e - sv * NB * HN) / HN;
            const int k = e - (sv * NB + bi) * HN;
            const unsigned long long h = (unsigned long long)((p.vertical ? rep[sv] : 1) + k);
            const unsigned long long b = (unsigned long long)p.prob.batch_sizes[bi];
            const unsigned long long m = (p.prob.flags & THEMIS_QUEUE_PER_REPLICA) ? h : 1ull;
            const unsigned long long q_num = (b - 1ull) * m * 1000000000ull;
            Q[TH_IDX(503, e, tab)] = sat_u32((q_num + q_den - 1ull) / q_den, (uint32_t)T + 1u);
            Lmax[TH_IDX(504, e, tab)] = sat_u32(h * b * 1000000000ull / lambda_m, 0x7FFFFFFFu);
        }
    }
    __syncthreads();

    const int lane = tid & 31, warp = tid >> 5;
    const int c_chunks = (C + 31) / 32;
    const int n_tasks = NB * c_chunks;
    const uint32_t w_magic = 0xFFFFFFFFu / w_us;
    int saw_bad_latency = 0;
    int n_f = 0;                                  // entries in the prefix front

    for (int s = 0; s < S; ++s) {
        // 1. candidates of stage s: per (cores, batch size) the fewest replicas that sustain lambda
        const int h_lo = p.vertical ? rep[s] : 1;
        const int32_t *lat_s = lat + (size_t)s * CB;
        const uint32_t *Q_s = Q + (p.vertical ? s * NB : 0);
        const uint32_t *Lmax_s = Lmax + (p.vertical ? s * NB : 0);
        for (int task = warp; task < n_tasks; task += kWarps) {
            const int bi = task / c_chunks;
            const int c = (task - bi * c_chunks) * 32 + lane + 1;
            if (c > C) continue;
            const int pair = (c - 1) * NB + bi;
            const int32_t l_us = lat_s[TH_IDX(505, pair, CB)];
            if (l_us <= 0) { saw_bad_latency = 1; continue; }
            if (c > 1 && lat_s[TH_IDX(506, pair - NB, CB)] == l_us) continue;   // same buckets, cheaper, one core fewer
            uint32_t l_q = __umulhi((uint32_t)l_us, w_magic);
            uint32_t l_r = (uint32_t)l_us - l_q * w_us;
            while (l_r >= w_us) { l_r -= w_us; ++l_q; }
            const uint32_t l_b = l_q + (l_r != 0u);
            if (l_b > (uint32_t)T) continue;
            const int b = p.prob.batch_sizes[bi];
            const uint32_t *lmax_row = Lmax_s + bi * HN;
            const float need = (float)l_us * ((float)lambda_m / ((float)b * 1.0e9f)) - (float)h_lo;
            int k = (int)fminf(fmaxf(need, 0.0f), (float)HN) - 1;
            k = max(k, 0);
            if (k > 0 && (uint32_t)l_us <= lmax_row[TH_IDX(507, k - 1, HN)]) k = 0;
            while (k < HN && (uint32_t)l_us > lmax_row[TH_IDX(508, k, HN)]) ++k;
            if (k >= HN) continue;                                   // no replica count sustains lambda
            const uint32_t ell = l_b + Q_s[TH_IDX(509, bi * HN + k, NB * HN)];
            if (ell > (uint32_t)T) continue;
            const uint32_t cost = (uint32_t)(h_lo + k) * (uint32_t)c;
            const uint32_t idx = (uint32_t)((p.horizontal ? 0 : k * CB) + pair);
            atomicMin(&keys_g[TH_IDX(510, ell, pitch)], (cost << 16) | idx);
        }
        __syncthreads();

        // 2. front of G_s, kept in shared memory for the pairing and in the workspace for the backtrack
        uint32_t *G_row = reinterpret_cast<uint32_t *>(p.G + ((size_t)n * S + s) * pitch);
        uint16_t *Gc_row = p.Garg + ((size_t)n * S + s) * pitch;
        uint16_t *A_row = p.A + ((size_t)n * S + s) * pitch;
        const int n_g = front_of_row<16, kThreads>(p, keys_g, T + 1, seg, warp_tot, &s_total, tid,
            [&](int pos, int l, uint32_t key) {
                gf_l[TH_IDX(511, pos, cap_g)] = (uint32_t)l;
                gf_c[TH_IDX(512, pos, cap_g)] = key >> 16;
                G_row[TH_IDX(513, pos, pitch)] = ((uint32_t)l << 16) | (key & 0xFFFFu);
                Gc_row[TH_IDX(514, pos, pitch)] = (uint16_t)(key >> 16);
                if (s == 0) {                      // the first stage's front is the first prefix front
                    ff_t[TH_IDX(515, pos, pitch)] = (uint32_t)l;
                    ff_c[TH_IDX(516, pos, pitch)] = key >> 16;
                    A_row[TH_IDX(517, l, pitch)] = (uint16_t)pos;
                }
            });
        if (s == 0) { n_f = n_g; continue; }

        // 3. front(F_{s-1}) x front(G_s): each warp takes prefix entries, lanes take stage entries
        for (int i = warp; i < n_f; i += kWarps) {
            const uint32_t t_i = ff_t[TH_IDX(518, i, pitch)], c_i = ff_c[TH_IDX(519, i, pitch)];
            for (int k = lane; k < n_g; k += 32) {
                const uint32_t t = t_i + gf_l[TH_IDX(520, k, cap_g)];
                if (t > (uint32_t)T) break;           // ascending l: the rest does not fit either
                atomicMin(&keys_f[TH_IDX(521, t, pitch)], ((c_i + gf_c[TH_IDX(522, k, cap_g)]) << kIdxBits) | (uint32_t)k);
            }
        }
        __syncthreads();

        // 4. front of F_s; the argmin k of every front cell goes to the workspace
        n_f = front_of_row<kIdxBits, kThreads>(p, keys_f, T + 1, seg, warp_tot, &s_total, tid,
            [&](int pos, int t, uint32_t key) {
                ff_t[TH_IDX(523, pos, pitch)] = (uint32_t)t;
                ff_c[TH_IDX(524, pos, pitch)] = key >> kIdxBits;
                A_row[TH_IDX(525, t, pitch)] = (uint16_t)(key & kIdxMask);
            });
    }
    const int any_bad = __syncthreads_or(saw_bad_latency);    // also orders this block's global stores
    if (tid != 0) return;
    p.inst_flag[n] = any_bad ? kFlagBadInput : 0;
    if (any_bad) { write_unsolved(THEMIS_STATUS_BAD_INPUT); return; }
    if (n_f == 0) { write_unsolved(THEMIS_STATUS_INFEASIBLE); return; }
    // Costs fall strictly along the front, so its last entry is the cheapest total at
    // the lowest budget that reaches it.
    const int tstar = (int)ff_t[TH_IDX(526, n_f - 1, pitch)];
    int t = tstar;
    for (int s = S - 1; s >= 0; --s) {
        const size_t row = ((size_t)n * S + s) * pitch;
        const int k = (int)p.A[TH_IDX(527, row + t, (size_t)p.prob.n_instances * S * pitch)];
        const uint32_t e = reinterpret_cast<const uint32_t *>(p.G)[TH_IDX(528, row + k, (size_t)p.prob.n_instances * S * pitch)];
        const int ell = (int)(e >> 16), idx = (int)(e & 0xFFFFu);
        const int bi = idx % NB, rest = idx / NB;
        b_o[s] = p.prob.batch_sizes[bi];
        c_o[s] = rest % C + 1;
        h_o[s] = p.vertical ? rep[s] : p.horizontal ? (int)p.Garg[row + k] : rest / C + 1;
        t -= ell;
    }
    p.out.total_cost[n] = (int32_t)ff_c[n_f - 1];
    p.out.latency_buckets[n] = tstar;
    p.out.status[n] = THEMIS_STATUS_OK;
}

// kThreads: 128 for short budgets (fewer, cheaper barriers per stage), else 256.
// LISTED: the grid works through the instances in redo_list (those the warp kernel handed
// over) instead of taking one instance per block.
template <int kThreads, bool LISTED>
__global__ void __launch_bounds__(kThreads)
solve_sparse_kernel(const Params p)
{
    extern __shared__ __align__(16) uint32_t smem[];
    if (!LISTED) {
        solve_instance_sparse<kThreads>(p, blockIdx.x, smem);
        return;
    }
    const int count = min(*p.redo_count, p.prob.n_instances);
    for (int i = blockIdx.x; i < count; i += gridDim.x) {
        solve_instance_sparse<kThreads>(p, TH_IDX(529, p.redo_list[TH_IDX(530, i, p.prob.n_instances)], p.prob.n_instances), smem);
        __syncthreads();                 // the last reader of this instance's shared memory is done
    }
}

}  // namespace

size_t sparse_smem_bytes(const Params &p)
{
    const size_t table = p.vertical ? (size_t)p.prob.n_stages * p.prob.n_batch
                                    : (size_t)p.prob.n_batch * p.prob.h_max;
    const size_t cap_g = (size_t)(p.pitch < p.prob.c_max * p.prob.n_batch ? p.pitch : p.prob.c_max * p.prob.n_batch);
    return sizeof(uint32_t) * (3u * (size_t)p.pitch + 2u * cap_g + 2u * table + 32u);
}

// (internal linkage: its `ready` word must belong to this copy of the library alone)
template <int kThreads, bool LISTED>
static cudaError_t launch_sparse_variant(const Params &p, size_t smem, cudaStream_t stream)
{
    static std::atomic<uint64_t> ready{0};
    cudaError_t e = allow_max_smem(reinterpret_cast<const void *>(solve_sparse_kernel<kThreads, LISTED>), ready);
    if (e != cudaSuccess) return e;
    // listed: a fixed grid of a few blocks per SM; an empty list costs one short launch
    const int blocks = LISTED ? min(p.prob.n_instances, 4 * 148) : p.prob.n_instances;
    solve_sparse_kernel<kThreads, LISTED><<<blocks, kThreads, smem, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_solve_sparse(const Params &p, bool only_listed, cudaStream_t stream)
{
    const size_t smem = sparse_smem_bytes(p);
    if (p.pitch <= 1024)
        return only_listed ? launch_sparse_variant<128, true>(p, smem, stream)
                           : launch_sparse_variant<128, false>(p, smem, stream);
    return only_listed ? launch_sparse_variant<256, true>(p, smem, stream)
                       : launch_sparse_variant<256, false>(p, smem, stream);
}

}  // namespace themis

// Min-plus stage recurrence over the undominated entries of G_s only.
//
// An entry (l, G_s[l]) is dominated when a smaller l' has G_s[l'] <= G_s[l]:
// swapping it for (l', G_s[l']) in any complete configuration lowers the total
// latency without raising the cost, so the solution the solver returns (cheapest,
// then lowest total latency, then lowest stage latencies from the last stage down)
// never contains a dominated entry.  Restricting every stage to its front
//   P_s = { l : G_s[l] < min_{l' < l} G_s[l'] }        (cost strictly falling in l)
// therefore leaves the returned configuration, cost and latency unchanged, while
//   F_s[t] = min_{l in P_s, l <= t} F_{s-1}[t - l] + G_s[l]
// needs |P_s| instead of t + 1 terms per cell (tens instead of thousands on the
// benchmark workloads).  The intermediate tables are those of the restricted
// problem, not the dense ones.  Same recurrence, tie-breaking and backtrack as
// Algorithm 1's budget loop; arithmetic on packed keys (cost << 14 | l) as in the
// 32-bit dense kernel, so one fused add-min per term carries the argmin.
//
// One block per instance.  Per stage: bulk-async copy of the G row (double
// buffered, bounded waits), block-wide front extraction (prefix minimum, flag,
// compaction), then every thread updates its cells against the front list.
#include "themis_async.cuh"
#include "themis_internal.h"

namespace themis {
namespace {

constexpr int kPrunedThreads = 256;
constexpr int kPrunedWarps = kPrunedThreads / 32;
constexpr int kCellsInFlight = 4;

// Exclusive prefix over the block in thread order; op is min or add.
template <bool IS_MIN>
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t identity, uint32_t *warp_tot,
                                                         int tid)
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
    __syncthreads();                                  // warp_tot may be reused
    return IS_MIN ? min(before, exc) : before + exc;
}

// Front of one raw G row (int32 costs, THEMIS_G_INF = empty) as packed keys
// (cost << 14 | l) in ascending l; returns the entry count.  seg = entries per thread.
__device__ __forceinline__ int extract_front(const Params &p, const uint32_t *g_row, int n_entries, int seg,
                                             uint32_t *front, uint32_t *warp_tot, int tid)
{
    (void)p;
    const int l0 = tid * seg, l1 = min(l0 + seg, n_entries);
    uint32_t local_min = 0xFFFFFFFFu;
    for (int l = l0; l < l1; ++l) local_min = min(local_min, g_row[l]);
    const uint32_t before = block_exclusive_scan<true>(local_min, 0xFFFFFFFFu, warp_tot, tid);
    uint32_t running = min(before, kInfCost);          // empty buckets and costs >= "unreachable" never enter
    uint32_t count = 0;
    for (int l = l0; l < l1; ++l)
        if (g_row[l] < running) { running = g_row[l]; ++count; }
    uint32_t pos = block_exclusive_scan<false>(count, 0u, warp_tot, tid);
    running = min(before, kInfCost);
    for (int l = l0; l < l1; ++l)
        if (g_row[TH_IDX(401, l, p.pitch)] < running) {
            running = g_row[l];
            front[TH_IDX(402, pos, p.pitch)] = (running << kIdxBits) | (uint32_t)l;
            ++pos;
        }
    // total = exclusive prefix of the last thread + its count
    __shared__ uint32_t s_total;
    if (tid == kPrunedThreads - 1) s_total = pos;
    __syncthreads();
    return (int)s_total;
}

__global__ void __launch_bounds__(kPrunedThreads)
minplus_pruned_kernel(const Params p)
{
    extern __shared__ __align__(128) uint32_t smem[];
    const int n = blockIdx.x;
    if (p.active && !p.active[n]) return;
    const int tid = threadIdx.x;
    const int T = p.T, pitch = p.pitch, S = p.prob.n_stages;
    // entries per thread in the front extraction; odd, so that the lanes' segments start in distinct banks
    const int seg = ((pitch + kPrunedThreads - 1) / kPrunedThreads) | 1;

    uint32_t *Fa = smem;                       // [pitch] prefix table, packed keys (cost << 14)
    uint32_t *Fb = Fa + pitch;                 // [pitch]
    uint32_t *Gbuf0 = Fb + pitch;              // [pitch] raw G rows
    uint32_t *Gbuf1 = Gbuf0 + pitch;
    uint32_t *front = Gbuf1 + pitch;           // [pitch] front entries of the current stage
    uint64_t *mbar = reinterpret_cast<uint64_t *>(front + pitch);
    uint32_t *red = reinterpret_cast<uint32_t *>(mbar + 2);   // 32 words

    const uint32_t row_bytes = (uint32_t)pitch * 4u;
    const int32_t *G_inst = p.G + (size_t)n * S * pitch;

    int32_t *h_o = p.out.h + (size_t)n * S, *c_o = p.out.c + (size_t)n * S, *b_o = p.out.b + (size_t)n * S;
    auto write_unsolved = [&](int status) {
        for (int s = 0; s < S; ++s) { h_o[s] = 0; c_o[s] = 0; b_o[s] = 0; }
        p.out.total_cost[n] = -1;
        p.out.latency_buckets[n] = -1;
        p.out.status[n] = status;
    };
    if (p.inst_flag[TH_IDX(411, n, p.prob.n_instances)] == kFlagBadInput) {     // bad input seen while scoring
        if (tid == 0) write_unsolved(THEMIS_STATUS_BAD_INPUT);
        return;
    }
    if (tid == 0) {
        mbar_init(&mbar[0], 1);
        mbar_init(&mbar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_expect_tx(&mbar[0], row_bytes);
        bulk_load(Gbuf0, G_inst, row_bytes, &mbar[0]);
        if (S > 1) {
            mbar_expect_tx(&mbar[1], row_bytes);
            bulk_load(Gbuf1, G_inst + pitch, row_bytes, &mbar[1]);
        }
    }
    int failed = 0;
    int pend0 = 0, pend1 = S > 1 ? 0 : -1;     // phase parity of a copy in flight, or -1
    // Row r goes into buffer r & 1 once that buffer's previous row has been consumed.
    auto refill = [&](int r) {
        if (r >= S) return;
        if (tid == 0) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_expect_tx(&mbar[r & 1], row_bytes);
            bulk_load((r & 1) ? Gbuf1 : Gbuf0, G_inst + (size_t)r * pitch, row_bytes, &mbar[r & 1]);
        }
        if (r & 1) pend1 = (r >> 1) & 1; else pend0 = (r >> 1) & 1;
    };

    // stage 0: the front of G_0 is the whole prefix table
    if (!mbar_wait(&mbar[0], 0)) failed = 1; else pend0 = -1;
    failed = __syncthreads_or(failed);
    uint32_t *Fprev = Fa, *Fnew = Fb;
    if (!failed) {
        for (int t = tid; t < pitch; t += kPrunedThreads) Fprev[t] = kInfKey;
        const int P = extract_front(p, Gbuf0, T + 1, seg, front, red, tid);   // barriers inside order the fill
        for (int k = tid; k < P; k += kPrunedThreads) {
            const uint32_t e = front[k];
            Fprev[TH_IDX(403, e & kIdxMask, pitch)] = e & ~kIdxMask;
        }
    }
    __syncthreads();
    if (!failed) refill(2);

    for (int s = 1; s < S && !failed; ++s) {
        const int cur = s & 1;
        uint32_t *Graw = cur ? Gbuf1 : Gbuf0;
        if (!mbar_wait(&mbar[cur], (uint32_t)((s >> 1) & 1))) failed = 1;
        else if (cur) pend1 = -1; else pend0 = -1;
        failed = __syncthreads_or(failed);
        if (failed) break;
        const int P = extract_front(p, Graw, T + 1, seg, front, red, tid);
        uint16_t *A_row = p.A + ((size_t)n * S + s) * pitch;
        // kCellsInFlight cells per thread at a time (independent chains hide the
        // shared-memory latency); cells of one thread are kPrunedThreads apart, so the
        // loads of a warp stay on consecutive words.
        for (int t0 = tid; t0 < pitch; t0 += kPrunedThreads * kCellsInFlight) {
            uint32_t acc[kCellsInFlight];
#pragma unroll
            for (int j = 0; j < kCellsInFlight; ++j) acc[j] = 0xFFFFFFFFu;
            const int t_hi = t0 + kPrunedThreads * (kCellsInFlight - 1);
            for (int k = 0; k < P; ++k) {
                const uint32_t e = front[TH_IDX(404, k, pitch)];
                const int l = (int)(e & kIdxMask);
                if (l > t_hi) break;            // ascending l: nothing further fits any of these cells
#pragma unroll
                for (int j = 0; j < kCellsInFlight; ++j) {
                    const int i = t0 + kPrunedThreads * j - l;
                    const uint32_t f = i >= 0 && i < pitch ? Fprev[TH_IDX(405, i, pitch)] : kInfKey;
                    acc[j] = __viaddmin_u32(f, e, acc[j]);
                }
            }
#pragma unroll
            for (int j = 0; j < kCellsInFlight; ++j) {
                const int t = t0 + kPrunedThreads * j;
                if (t < pitch) {
                    const bool inf = acc[j] >= kInfKey;
                    Fnew[TH_IDX(406, t, pitch)] = inf ? kInfKey : (acc[j] & ~kIdxMask);
                    A_row[TH_IDX(407, t, pitch)] = inf ? (uint16_t)0 : (uint16_t)(acc[j] & kIdxMask);
                }
            }
        }
        __syncthreads();                        // F_s complete; front and this G buffer free
        refill(s + 2);                          // row s+2 goes where row s was
        uint32_t *tmp = Fprev; Fprev = Fnew; Fnew = tmp;
    }
    failed = __syncthreads_or(failed);
    if (failed) {
        if (pend0 >= 0) mbar_wait(&mbar[0], (uint32_t)pend0);
        if (pend1 >= 0) mbar_wait(&mbar[1], (uint32_t)pend1);
        if (tid == 0) write_unsolved(THEMIS_STATUS_TIMEOUT);
        return;
    }

    // final scan: cheapest total, lowest total latency among equals
    uint32_t best = 0xFFFFFFFFu;
    int32_t *F_row = p.F + (size_t)n * pitch;
    for (int t = tid; t < pitch; t += kPrunedThreads) {
        const uint32_t fk = Fprev[t];
        if (t <= T) best = min(best, fk | (uint32_t)t);
        F_row[TH_IDX(408, t, pitch)] = fk >= kInfKey ? THEMIS_G_INF : (int32_t)(fk >> kIdxBits);
    }
    best = __reduce_min_sync(0xFFFFFFFFu, best);
    if ((tid & 31) == 0) red[tid >> 5] = best;
    __syncthreads();                            // also orders this block's A stores
    if (tid == 0) {
        for (int w = 1; w < kPrunedWarps; ++w) best = min(best, red[w]);
        if (best >= kInfKey) {
            write_unsolved(THEMIS_STATUS_INFEASIBLE);
        } else {
            const int tstar = (int)(best & kIdxMask);
            int t = tstar;
            const int C = p.prob.c_max, NB = p.prob.n_batch;
            for (int s = S - 1; s >= 0; --s) {
                const size_t row = ((size_t)n * S + s) * pitch;
                const int ell = s > 0 ? (int)p.A[TH_IDX(409, row + t, (size_t)p.prob.n_instances * S * pitch)] : t;
                const int idx = (int)p.Garg[TH_IDX(410, row + ell, (size_t)p.prob.n_instances * S * pitch)];
                const int bi = idx % NB, rest = idx / NB;
                b_o[s] = p.prob.batch_sizes[bi];
                c_o[s] = rest % C + 1;
                h_o[s] = p.vertical ? p.replicas[(size_t)n * S + s]
                       : p.horizontal ? G_inst[(size_t)s * pitch + ell] : rest / C + 1;
                t -= ell;
            }
            p.out.total_cost[n] = (int32_t)(best >> kIdxBits);
            p.out.latency_buckets[n] = tstar;
            p.out.status[n] = THEMIS_STATUS_OK;
        }
    }
}

}  // namespace

cudaError_t launch_minplus_pruned(const Params &p, cudaStream_t stream)
{
    const size_t smem = pruned_smem_bytes(p.pitch);
    static std::atomic<uint64_t> ready{0};
    cudaError_t e = allow_max_smem(reinterpret_cast<const void *>(minplus_pruned_kernel), ready);
    if (e != cudaSuccess) return e;
    minplus_pruned_kernel<<<p.prob.n_instances, kPrunedThreads, smem, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace themis

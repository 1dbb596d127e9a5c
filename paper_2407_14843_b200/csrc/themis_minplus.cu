// Min-plus stage recurrence, final scan and backtrack (Algorithm 1's budget
// loop with the candidate minimum hoisted out), one thread block per instance:
//
//   F_0 = G_0,   F_s[t] = min_{0<=l<=t} F_{s-1}[t-l] + G_s[l],   A_s[t] = lowest such l
//
// Arithmetic.  Both operands are kept as packed unsigned keys
//   Fk[i] = cost << 14                (low 14 bits zero)
//   Gk[l] = cost << 14 | l
// so one fused add-min per (t, l) cell carries the argmin along: the smallest
// sum has the smallest cost and, among equal costs, the smallest l.  The cost
// field is 17 bits with "unreachable" = 2^17 - 1; the sum of two fields fits 18
// bits, so no cell needs a branch or can overflow.
//
// Tiling.  A thread owns R consecutive budget cells t0..t0+R-1 and walks l
// upward in chunks of R.  Per chunk it loads R new words of F (its window
// slides down by R) and R words of G (the same address for every lane of the
// warp, a broadcast) and performs R*R cell updates from registers.  F is stored
// in chunks of R words padded to R+4 so that the 16-byte loads of consecutive
// lanes fall into distinct bank groups; one extra chunk of "unreachable" in
// front of F[0] stands for every negative index.
//
// Staging.  Row s+1 of G is fetched by a bulk asynchronous copy into the other
// half of a double buffer, completion signalled on an mbarrier, while stage s
// computes.  Every wait on an mbarrier is bounded; on expiry the block reports
// THEMIS_STATUS_TIMEOUT for its instance and leaves.
#include "themis_async.cuh"
#include "themis_internal.h"
#include "themis_minplus_step.cuh"

namespace themis {
namespace {

template <int R, int MAXT>
__global__ void __launch_bounds__(MAXT)
minplus_kernel(const Params p)
{
    extern __shared__ __align__(128) uint32_t smem[];
    constexpr int CS = Tile<R>::kChunkStride;
    const int n = blockIdx.x;
    if (p.active && !p.active[n]) return;
    const int tid = threadIdx.x;
    const int NT = blockDim.x;
    const int T = p.T, pitch = p.pitch, S = p.prob.n_stages;
    const int Tp = NT * R;                              // padded budget length, >= pitch

    uint32_t *Fs = smem;                                // (NT + 1) chunks of CS words; chunk -1 first
    uint32_t *Gbuf0 = Fs + (NT + 1) * CS;
    uint32_t *Gbuf1 = Gbuf0 + Tp;
    uint64_t *mbar = reinterpret_cast<uint64_t *>(Gbuf1 + Tp);
    uint32_t *red = reinterpret_cast<uint32_t *>(mbar + 2);   // 32 words for the block reduction

    const int tile = ((int)p.warp_group[tid >> 5] << 5) | (tid & 31);                   // groups dealt by assign_warp_groups
    const int t0 = tile * R;
    const int f_words = (NT + 1) * CS;                  // words of F in shared memory
    (void)f_words;
    uint32_t *my_chunk = Fs + TH_IDX(301, tile + 1, NT + 1) * CS;
    const uint32_t row_bytes = (uint32_t)pitch * 4u;
    const int32_t *G_inst = p.G + (size_t)n * S * pitch;

    int32_t *h_o = p.out.h + (size_t)n * S, *c_o = p.out.c + (size_t)n * S, *b_o = p.out.b + (size_t)n * S;
    // Writes the "no configuration" result with the given status (one thread).
    auto write_unsolved = [&](int status) {
        for (int s = 0; s < S; ++s) { h_o[s] = 0; c_o[s] = 0; b_o[s] = 0; }
        p.out.total_cost[n] = -1;
        p.out.latency_buckets[n] = -1;
        p.out.status[n] = status;
    };
    if (p.only_flagged) {                               // second pass: only what the packed kernel left over
        if (p.inst_flag[TH_IDX(302, n, p.prob.n_instances)] != kFlagNeedsWide) return;
    } else if (p.inst_flag[n] == kFlagBadInput) {       // bad input seen while scoring
        if (tid == 0) write_unsolved(THEMIS_STATUS_BAD_INPUT);
        return;
    }

    if (tid == 0) {
        mbar_init(&mbar[0], 1);
        mbar_init(&mbar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // "unreachable" in front of F[0], and behind the loaded part of each G buffer
    if (tid < CS) Fs[tid] = kInfKey;
    for (int l = pitch + tid; l < Tp; l += NT) {
        Gbuf0[TH_IDX(303, l, Tp)] = kInfKey | (uint32_t)l;
        Gbuf1[TH_IDX(304, l, Tp)] = kInfKey | (uint32_t)l;
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
    int failed = 0;                                     // a bounded wait ran out
    int pend0 = 0, pend1 = S > 1 ? 0 : -1;              // phase parity of a copy in flight, or -1

    // stage 0: F_0 = G_0
    if (!mbar_wait(&mbar[0], 0)) failed = 1; else pend0 = -1;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const uint32_t raw = Gbuf0[TH_IDX(305, t0 + r, Tp)];   // raw cost, or >= kInfCost when empty/padding
        my_chunk[r] = min(raw, kInfCost) << kIdxBits;
    }
    failed = __syncthreads_or(failed);

    for (int s = 1; s < S && !failed; ++s) {
        const int cur = s & 1;
        uint32_t *Gk = cur ? Gbuf1 : Gbuf0;
        const int parity = (s >> 1) & 1;
        if (!mbar_wait(&mbar[cur], (uint32_t)parity)) failed = 1;
        else if (cur) pend1 = -1; else pend0 = -1;
        // raw costs -> packed keys, in place (own R entries)
        if (t0 < pitch) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const uint32_t raw = Gk[TH_IDX(306, t0 + r, Tp)];
                Gk[TH_IDX(307, t0 + r, Tp)] = (min(raw, kInfCost) << kIdxBits) | (uint32_t)(t0 + r);
            }
        }
        failed = __syncthreads_or(failed);               // keys and F_{s-1} visible to all
        if (failed) break;
        if (s + 1 < S) {                                 // the other buffer is free again
            const int nxt = cur ^ 1;
            if (tid == 0) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect_tx(&mbar[nxt], row_bytes);
                bulk_load(nxt ? Gbuf1 : Gbuf0, G_inst + (size_t)(s + 1) * pitch, row_bytes, &mbar[nxt]);
            }
            if (nxt) pend1 = ((s + 1) >> 1) & 1; else pend0 = ((s + 1) >> 1) & 1;
        }

        uint32_t acc[R], wa[R], wb[R];
#pragma unroll
        for (int r = 0; r < R; ++r) { acc[r] = 0xFFFFFFFFu; wa[r] = my_chunk[r]; }
        // All lanes of a warp walk the same l so that G is a broadcast; lanes
        // that run past their own range read the "unreachable" chunk in front.
        const int q_end = tile | 31;
        int f_off = tile * CS;                           // word offset of chunk tile-1
        const uint32_t *g = Gk;
        for (int q = 0; q <= q_end; q += 2) {
            chunk_step<R>(wa, wb, acc, Fs + TH_IDX(308, max(f_off, 0), f_words - R + 1), TH_PTR(309, g, Gk, Tp - R + 1));
            chunk_step<R>(wb, wa, acc, Fs + TH_IDX(310, max(f_off - CS, 0), f_words - R + 1),
                          TH_PTR(311, g + R, Gk, Tp - R + 1));
            f_off -= 2 * CS;
            g += 2 * R;
        }
        __syncthreads();                                 // every read of F_{s-1} is done

        uint32_t a16[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const bool inf = acc[r] >= kInfKey;
            my_chunk[r] = inf ? kInfKey : (acc[r] & ~kIdxMask);
            a16[r] = inf ? 0u : (acc[r] & kIdxMask);
        }
        if (t0 + R <= pitch) {
            uint16_t *A_row = p.A + TH_IDX(312, ((size_t)n * S + s) * pitch + t0, (size_t)p.prob.n_instances * S * pitch - R + 1);
#pragma unroll
            for (int v = 0; v < R / 8; ++v) {
                uint4 o;
                o.x = a16[8 * v + 0] | (a16[8 * v + 1] << 16);
                o.y = a16[8 * v + 2] | (a16[8 * v + 3] << 16);
                o.z = a16[8 * v + 4] | (a16[8 * v + 5] << 16);
                o.w = a16[8 * v + 6] | (a16[8 * v + 7] << 16);
                *reinterpret_cast<uint4 *>(A_row + 8 * v) = o;
            }
        }
    }
    failed = __syncthreads_or(failed);

    if (failed) {
        // Let our own copies land (bounded) before the block's shared memory goes away.
        if (pend0 >= 0) mbar_wait(&mbar[0], (uint32_t)pend0);
        if (pend1 >= 0) mbar_wait(&mbar[1], (uint32_t)pend1);
        if (tid == 0) write_unsolved(THEMIS_STATUS_TIMEOUT);
        return;
    }

    // last prefix table to the workspace, and the final scan: cheapest total,
    // lowest total latency among equals
    uint32_t best = 0xFFFFFFFFu;
    int32_t *F_row = p.F + (size_t)n * pitch;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int t = t0 + r;
        const uint32_t fk = my_chunk[r];
        if (t <= T) best = min(best, fk | (uint32_t)t);
        if (t < pitch) F_row[TH_IDX(313, t, pitch)] = fk >= kInfKey ? THEMIS_G_INF : (int32_t)(fk >> kIdxBits);
    }
    best = __reduce_min_sync(0xFFFFFFFFu, best);
    if ((tid & 31) == 0) red[TH_IDX(314, tid >> 5, 32)] = best;
    __syncthreads();                                     // also orders this block's A stores
    if (tid == 0) {
        for (int w = 1; w < (NT >> 5); ++w) best = min(best, red[w]);
        if (best >= kInfKey) {
            write_unsolved(THEMIS_STATUS_INFEASIBLE);
        } else {
            const int tstar = (int)(best & kIdxMask);
            int t = tstar;
            const int C = p.prob.c_max, NB = p.prob.n_batch;
            for (int s = S - 1; s >= 0; --s) {
                const size_t row = ((size_t)n * S + s) * pitch;
                const int ell = s > 0 ? (int)p.A[TH_IDX(315, row + t, (size_t)p.prob.n_instances * S * pitch)] : t;
                const int idx = (int)p.Garg[TH_IDX(316, row + ell, (size_t)p.prob.n_instances * S * pitch)];
                const int bi = idx % NB, rest = idx / NB;
                b_o[s] = p.prob.batch_sizes[TH_IDX(317, bi, THEMIS_MAX_BATCH_SIZES)];
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

template <int R, int MAXT>
cudaError_t launch_variant(const Params &p_in, int threads, size_t smem, cudaStream_t stream)
{
    Params p = p_in;
    assign_warp_groups(threads / 32, p.warp_group);
    static std::atomic<uint64_t> ready{0};
    cudaError_t e = allow_max_smem(reinterpret_cast<const void *>(minplus_kernel<R, MAXT>), ready);
    if (e != cudaSuccess) return e;
    minplus_kernel<R, MAXT><<<p.prob.n_instances, threads, smem, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_minplus(const Params &p, int tile, cudaStream_t stream)
{
    if (minplus_warp_fits(p, tile)) return launch_minplus_warp(p, stream);   // short budgets: a warp per instance
    const int cells = p.T + 1;
    int R = tile;
    if (R != 8 && R != 16) R = 8;                       // (4 is a packed-kernel tile only)
    if (R == 8 && (cells + 7) / 8 > 1024) R = 16;
    const int chunks = (cells + R - 1) / R;
    const int threads = (chunks + 31) / 32 * 32;
    const size_t words = (size_t)(threads + 1) * (R + 4) + 2u * (size_t)threads * R + 4 + 32;
    const size_t smem = words * sizeof(uint32_t);
    if (R == 8)
        return threads <= 512 ? launch_variant<8, 512>(p, threads, smem, stream)
                              : launch_variant<8, 1024>(p, threads, smem, stream);
    return threads <= 512 ? launch_variant<16, 512>(p, threads, smem, stream)
                          : launch_variant<16, 1024>(p, threads, smem, stream);
}

}  // namespace themis

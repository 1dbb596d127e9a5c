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
// front of F[0] stands for every negative index.  Column length grows with the
// tile index, so a warp takes a group of 32 long tiles and then a group of 32
// short ones (group last - w, then group w): all warps walk the same number of
// chunks.  Chunks that can only give "unreachable" (below G_s's first entry, or
// meeting F_{s-1} only below its first reachable budget) are skipped.
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
    const int n_warps = NT >> 5;
    const int T = p.T, pitch = p.pitch, S = p.prob.n_stages;
    // Folding: column length grows with the tile index and all lanes of a warp run to the
    // longest column of their 32 tiles, so a warp takes a group of 32 long tiles and then a
    // group of 32 short ones: group (last - w), then group w.  Every warp of the block then
    // walks the same number of chunks.  The tiling is right-aligned: the tiles that pad the
    // budget to a whole (even) number of groups lie in front of cell 0, where columns are
    // shortest, and stay "unreachable".
    const int n_groups = 2 * n_warps;
    const int n_tiles = n_groups * 32;
    const int Tc = n_tiles * R;
    const int Tp = max(Tc, pitch);                      // length of the G buffers
    const int n_dummy = (Tc - (T + 1)) / R;             // tiles in front of cell 0

    uint32_t *Fs = smem;                                // (n_tiles + 1) chunks of CS words; chunk -1 first
    uint32_t *Gbuf0 = Fs + (n_tiles + 1) * CS;
    uint32_t *Gbuf1 = Gbuf0 + Tp;
    uint64_t *mbar = reinterpret_cast<uint64_t *>(Gbuf1 + Tp);
    uint32_t *red = reinterpret_cast<uint32_t *>(mbar + 2);   // 32 words for the block reduction
    uint32_t *first_l = red + 32;                             // 2 words: first reachable l of the row in each G buffer

    const int warp = tid >> 5, lane = tid & 31;
    const int tile_a = (n_groups - 1 - warp) * 32 + lane, tile_b = warp * 32 + lane;
    const int t0_a = (tile_a - n_dummy) * R, t0_b = (tile_b - n_dummy) * R;
    const int f_words = (n_tiles + 1) * CS;             // words of F in shared memory
    (void)f_words;
    uint32_t *chunk_a = Fs + TH_IDX(301, tile_a + 1, n_tiles + 1) * CS;
    uint32_t *chunk_b = Fs + TH_IDX(318, tile_b + 1, n_tiles + 1) * CS;
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
        first_l[0] = first_l[1] = 0xFFFFFFFFu;
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

    // Raw costs of the row in Gk -> packed keys, in place, the block's threads striding over
    // the row; the first reachable l of the row goes to *first (complete after a barrier).
    auto to_keys = [&](uint32_t *Gk, uint32_t *first) {
        uint32_t lo = 0xFFFFFFFFu;
        for (int l4 = tid * 4; l4 < pitch; l4 += NT * 4) {
            uint4 v4 = *reinterpret_cast<const uint4 *>(Gk + TH_IDX(306, l4, Tp - 3));
            uint32_t *v = reinterpret_cast<uint32_t *>(&v4);
#pragma unroll
            for (int i = 3; i >= 0; --i) {
                if (v[i] < kInfCost && l4 + i <= T) lo = min(lo, (uint32_t)(l4 + i));
                v[i] = (min(v[i], kInfCost) << kIdxBits) | (uint32_t)(l4 + i);
            }
            *reinterpret_cast<uint4 *>(Gk + TH_IDX(307, l4, Tp - 3)) = v4;
        }
        lo = __reduce_min_sync(0xFFFFFFFFu, lo);
        if (lane == 0 && lo != 0xFFFFFFFFu) atomicMin(first, lo);
    };

    // stage 0: F_0 = G_0
    if (!mbar_wait(&mbar[0], 0)) failed = 1; else pend0 = -1;
    to_keys(Gbuf0, &first_l[0]);
    failed = __syncthreads_or(failed);
    if (!failed) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            chunk_a[r] = t0_a < 0 ? kInfKey : (Gbuf0[TH_IDX(305, t0_a + r, Tp)] & ~kIdxMask);
            chunk_b[r] = t0_b < 0 ? kInfKey : (Gbuf0[TH_IDX(319, t0_b + r, Tp)] & ~kIdxMask);
        }
    }
    uint32_t prefix_min = first_l[0];                   // lowest budget F_{s-1} can reach (0xFFFFFFFF: none)
    __syncthreads();                                    // F_0 complete, first_l[0] read by all
    if (tid == 0) first_l[0] = 0xFFFFFFFFu;

    for (int s = 1; s < S && !failed; ++s) {
        const int cur = s & 1;
        uint32_t *Gk = cur ? Gbuf1 : Gbuf0;
        const int parity = (s >> 1) & 1;
        if (!mbar_wait(&mbar[cur], (uint32_t)parity)) failed = 1;
        else if (cur) pend1 = -1; else pend0 = -1;
        if (!failed) to_keys(Gk, &first_l[cur]);
        failed = __syncthreads_or(failed);               // keys, their first entry and F_{s-1} visible to all
        if (failed) break;
        if (s + 1 < S) {                                 // the other buffer is free again
            const int nxt = cur ^ 1;
            if (tid == 0) {
                first_l[nxt] = 0xFFFFFFFFu;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect_tx(&mbar[nxt], row_bytes);
                bulk_load(nxt ? Gbuf1 : Gbuf0, G_inst + (size_t)(s + 1) * pitch, row_bytes, &mbar[nxt]);
            }
            if (nxt) pend1 = ((s + 1) >> 1) & 1; else pend0 = ((s + 1) >> 1) & 1;
        }
        // Chunks of l below G_s's first reachable entry, and chunks that only meet F_{s-1} below
        // its first reachable budget, can only give "unreachable" and are skipped (in pairs).
        const uint32_t g_min = first_l[cur];
        const bool dead = g_min == 0xFFFFFFFFu || prefix_min == 0xFFFFFFFFu;
        const int q_lo = dead ? 0 : (int)(g_min / R) & ~1;
        const int q_shift = dead ? 0 : ((int)(prefix_min / R) + n_dummy) & ~1;   // in tiles

        uint32_t acc[R], res_a[R], wa[R], wb[R];
        // All lanes of a warp walk the same l so that G is a broadcast; lanes that run past their
        // own range read the "unreachable" chunk in front.
        auto walk = [&](int tile) {
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r] = 0xFFFFFFFFu;
            const int steps = dead ? 0 : max(0, (tile | 31) - q_shift - q_lo + 1);   // even
            int f_off = (tile - q_lo) * CS;              // word offset of the chunk below the first one read
            if (steps > 0) {
                const uint32_t *f_hi = Fs + TH_IDX(320, max(f_off + CS, 0), f_words - R + 1);
#pragma unroll
                for (int r = 0; r < R; ++r) wa[r] = f_hi[r];
            }
            const uint32_t *g = Gk + q_lo * R;
            for (int q = 0; q < steps; q += 2) {
                chunk_step<R>(wa, wb, acc, Fs + TH_IDX(308, max(f_off, 0), f_words - R + 1), TH_PTR(309, g, Gk, Tp - R + 1));
                chunk_step<R>(wb, wa, acc, Fs + TH_IDX(310, max(f_off - CS, 0), f_words - R + 1),
                              TH_PTR(311, g + R, Gk, Tp - R + 1));
                f_off -= 2 * CS;
                g += 2 * R;
            }
        };
        walk(tile_a);
#pragma unroll
        for (int r = 0; r < R; ++r) res_a[r] = acc[r];
        walk(tile_b);
        prefix_min = dead ? 0xFFFFFFFFu : prefix_min + g_min;
        __syncthreads();                                 // every read of F_{s-1} is done

        auto store = [&](const uint32_t (&v)[R], uint32_t *chunk, int t0) {
            uint32_t a16[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const bool inf = v[r] >= kInfKey;
                chunk[r] = inf ? kInfKey : (v[r] & ~kIdxMask);
                a16[r] = inf ? 0u : (v[r] & kIdxMask);
            }
            if (t0 >= 0 && t0 + R <= pitch) {
                uint16_t *A_row = p.A + TH_IDX(312, ((size_t)n * S + s) * pitch + t0, (size_t)p.prob.n_instances * S * pitch - R + 1);
#pragma unroll
                for (int v8 = 0; v8 < R / 8; ++v8) {
                    uint4 o;
                    o.x = a16[8 * v8 + 0] | (a16[8 * v8 + 1] << 16);
                    o.y = a16[8 * v8 + 2] | (a16[8 * v8 + 3] << 16);
                    o.z = a16[8 * v8 + 4] | (a16[8 * v8 + 5] << 16);
                    o.w = a16[8 * v8 + 6] | (a16[8 * v8 + 7] << 16);
                    *reinterpret_cast<uint4 *>(A_row + 8 * v8) = o;
                }
            }
        };
        store(res_a, chunk_a, t0_a);
        store(acc, chunk_b, t0_b);
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
    auto scan = [&](const uint32_t *chunk, int t0) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int t = t0 + r;
            const uint32_t fk = chunk[r];
            if (t >= 0 && t <= T) best = min(best, fk | (uint32_t)t);
            if (t >= 0 && t < pitch) F_row[TH_IDX(313, t, pitch)] = fk >= kInfKey ? THEMIS_G_INF : (int32_t)(fk >> kIdxBits);
        }
    };
    scan(chunk_a, t0_a);
    scan(chunk_b, t0_b);
    best = __reduce_min_sync(0xFFFFFFFFu, best);
    if ((tid & 31) == 0) red[TH_IDX(314, tid >> 5, 32)] = best;
    __syncthreads();                                     // also orders this block's A stores
    if (tid == 0) {
        for (int w = 1; w < n_warps; ++w) best = min(best, red[w]);
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
cudaError_t launch_variant(const Params &p, int threads, size_t smem, cudaStream_t stream)
{
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
    int R = tile == 16 ? 16 : 8;                        // (4 is a packed-kernel tile only)
    int threads = 0;
    size_t smem = 0;
    for (;;) {
        // a warp takes two groups of 32 tiles (a long and a short one)
        const int groups = ((cells + R - 1) / R + 31) / 32;
        const int warps = (groups + 1) / 2;
        threads = warps * 32;                           // <= 1024: 16384 cells are 2048 tiles of 8
        const int n_tiles = 2 * warps * 32;
        const size_t g_words = (size_t)(n_tiles * R > p.pitch ? n_tiles * R : p.pitch);
        smem = sizeof(uint32_t) * ((size_t)(n_tiles + 1) * (R + 4) + 2u * g_words + 4 + 32 + 2);
        if (smem <= kMaxDynamicSmem || R == 16) break;
        R = 16;                                         // the longest budgets: fewer, wider chunks of F
    }
    if (R == 8)
        return threads <= 512 ? launch_variant<8, 512>(p, threads, smem, stream)
                              : launch_variant<8, 1024>(p, threads, smem, stream);
    return threads <= 512 ? launch_variant<16, 512>(p, threads, smem, stream)
                          : launch_variant<16, 1024>(p, threads, smem, stream);
}

}  // namespace themis

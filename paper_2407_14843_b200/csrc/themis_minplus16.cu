// Min-plus stage recurrence on packed 16-bit costs: two budget cells per
// register, two cell updates per fused add-min instruction.
//
//   F_0 = G_0,   F_s[t] = min_{0<=l<=t} F_{s-1}[t-l] + G_s[l]       (Algorithm 1's budget loop)
//
// Values.  Costs are held as unsigned half-words: exact below 0x7FFF and
// saturated there (0x7FFF = "unreachable or at least 32767").  Costs are
// non-negative, so any total below 0x7FFF only ever sums exact parts: the
// saturating tables equal the true ones wherever the true value is below 0x7FFF.
// Two half-words add without a carry into the neighbour (at most 0xFFFE).
//
// Packing.  Word k of F holds (F[2k], F[2k+1]).  For an even l = 2e the operand
// pair of output word j, (F[2j-l], F[2j+1-l]), is the aligned word j-e.  For an
// odd l = 2e+1 the same word j-e is the operand pair of outputs (2j+1, 2j+2), so
// every thread keeps two accumulator sets, acc for even l (cells 2j, 2j+1) and
// accp for odd l (cells 2j+1, 2j+2), and merges them once per stage with a
// half-word shift; the half-word that belongs to the next thread travels by a
// warp shuffle (and through shared memory across warps).  G is stored with each
// cost duplicated into both halves.
//
// Argmin.  No argmin is carried.  The prefix tables F_s are kept (uint16, in the
// workspace rows that the 32-bit kernel uses for its argmin tables) and the
// backtrack recovers, stage by stage along the optimal path only, the lowest l
// with F_{s-1}[t-l] + G_s[l] == F_s[t] by a block-wide scan.
//
// Saturation.  If the best total is 0x7FFF the instance is either infeasible
// (decided exactly: the fastest configurations of all stages do not fit the
// budget) or too expensive for 16 bits; the latter is flagged and redone by the
// 32-bit kernel in a second launch.
#include "themis_async.cuh"
#include "themis_internal.h"

namespace themis {
namespace {

constexpr uint32_t kInf16x2 = (kInf16 << 16) | kInf16;
constexpr int kPadChunks = 32;   // "unreachable" chunks in front of F[0]: one per lane of a warp
// Budgets just above a whole number of tile groups (T a power of two gives T + 1 cells) would cost
// a whole extra warp walking the longest columns for a handful of cells.  Up to this many cells
// beyond the last full group are instead computed by a block-wide reduction per stage.
constexpr int kMaxExtra = 8;

template <int R>
struct Tile16 {
    static constexpr int H = R / 2;                       // words per chunk
    static constexpr int CS = (H % 8 == 0) ? H + 4 : H;   // chunk stride: keeps 16-byte loads of
                                                          // consecutive lanes in distinct bank groups
};

// H consecutive words (H = 2, 4 or 8) from / to 8- or 16-byte aligned memory.
template <int H>
__device__ __forceinline__ void load_words(uint32_t (&w)[H], const uint32_t *src)
{
    if constexpr (H == 2) {
        const uint2 x = *reinterpret_cast<const uint2 *>(src);
        w[0] = x.x; w[1] = x.y;
    } else {
#pragma unroll
        for (int v = 0; v < H / 4; ++v) {
            const uint4 x = *reinterpret_cast<const uint4 *>(src + 4 * v);
            w[4 * v + 0] = x.x; w[4 * v + 1] = x.y; w[4 * v + 2] = x.z; w[4 * v + 3] = x.w;
        }
    }
}

template <int H>
__device__ __forceinline__ void store_words(const uint32_t (&w)[H], uint32_t *dst)
{
    if constexpr (H == 2) {
        *reinterpret_cast<uint2 *>(dst) = make_uint2(w[0], w[1]);
    } else {
#pragma unroll
        for (int v = 0; v < H / 4; ++v)
            *reinterpret_cast<uint4 *>(dst + 4 * v) = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
    }
}

// One chunk step: R values of l (H even/odd pairs) against the thread's R cells.
// w_hi holds words m .. m+H-1 of F, w_lo receives words m-H .. m-1 (m = J - q*H).
template <int R>
__device__ __forceinline__ void chunk_step16(const uint32_t (&w_hi)[R / 2], uint32_t (&w_lo)[R / 2],
                                             uint32_t (&acc)[R / 2], uint32_t (&accp)[R / 2],
                                             const uint32_t *f_chunk, const uint32_t *g_chunk)
{
    constexpr int H = R / 2;
    load_words<H>(w_lo, f_chunk);
#pragma unroll
    for (int v = 0; v < R / 4; ++v) {
        const uint4 g4 = *reinterpret_cast<const uint4 *>(g_chunk + 4 * v);   // l = l0+4v .. l0+4v+3
        const uint32_t g_even[2] = {g4.x, g4.z};
        const uint32_t g_odd[2] = {g4.y, g4.w};
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
            const int k = 2 * v + kk;                      // pair index within the chunk
#pragma unroll
            for (int r = 0; r < H; ++r) {
                const int i = H + r - k;                   // 1 .. 2H-1
                const uint32_t f = i >= H ? w_hi[i - H] : w_lo[i];
                acc[r] = __viaddmin_u16x2(f, g_even[kk], acc[r]);
                accp[r] = __viaddmin_u16x2(f, g_odd[kk], accp[r]);
            }
        }
    }
}

// Block-wide unsigned minimum; every thread gets the result.  Two barriers.
__device__ __forceinline__ uint32_t block_min(uint32_t v, uint32_t *red, int tid, int n_warps)
{
    v = __reduce_min_sync(0xFFFFFFFFu, v);
    if ((tid & 31) == 0) red[tid >> 5] = v;
    __syncthreads();
    uint32_t m = red[0];
    for (int w = 1; w < n_warps; ++w) m = min(m, red[w]);
    __syncthreads();
    return m;
}

// EXTRA: the block also computes up to kMaxExtra cells beyond its tiles (see kMaxExtra).
template <int R, int MAXT, bool EXTRA>
__global__ void __launch_bounds__(MAXT)
minplus16_kernel(const Params p)
{
    extern __shared__ __align__(128) uint32_t smem[];
    constexpr int H = Tile16<R>::H, CS = Tile16<R>::CS;
    constexpr int U = 32 / R;                             // chunk steps per loop iteration (2, 4 or 8)
    const int n = blockIdx.x;
    if (p.active && !p.active[n]) return;
    const int tid = threadIdx.x;
    const int NT = blockDim.x;
    const int n_warps = NT >> 5;
    const int T = p.T, pitch = p.pitch, S = p.prob.n_stages;
    const int Tc = NT * R;                                // cells covered by the tiles
    const int Tp = EXTRA ? max(Tc, pitch) : Tc;           // length of the G buffers (Tc >= pitch without extras)
    const int n_extra = EXTRA ? max(0, T + 1 - Tc) : 0;   // cells beyond the tiles, at most kMaxExtra

    uint32_t *Fw = smem;                                  // (kPadChunks + NT) chunks of CS words
    uint32_t *Gbuf0 = Fw + (kPadChunks + NT) * CS;
    uint32_t *Gbuf1 = Gbuf0 + Tp;
    uint64_t *mbar = reinterpret_cast<uint64_t *>(Gbuf1 + Tp);
    uint32_t *red = reinterpret_cast<uint32_t *>(mbar + 2);   // 32 words
    uint32_t *xchg = red + 32;                                // 32 words: last accp word of each warp
    uint32_t *stage_lmin = xchg + 32;                         // 64 words: first reachable l of every G_s
    uint32_t *fx_prev = stage_lmin + THEMIS_MAX_STAGES;       // kMaxExtra words: F_{s-1} at the extra cells
    uint32_t *fx_acc = fx_prev + kMaxExtra;                   // kMaxExtra words: F_s at the extra cells, building

    // Which tile (R consecutive cells) this thread owns: lanes keep consecutive tiles,
    // warps take the tile groups the host dealt them (see assign_warp_groups).
    const int tile = ((int)p.warp_group[tid >> 5] << 5) | (tid & 31);
    const int t0 = tile * R;
    uint32_t *my_chunk = Fw + (kPadChunks + tile) * CS;
    const uint32_t row_bytes = (uint32_t)pitch * 4u;
    const int32_t *G_inst = p.G + (size_t)n * S * pitch;
    uint16_t *F16_inst = p.A + (size_t)n * S * pitch;     // prefix tables F_s as uint16 rows

    int32_t *h_o = p.out.h + (size_t)n * S, *c_o = p.out.c + (size_t)n * S, *b_o = p.out.b + (size_t)n * S;
    auto write_unsolved = [&](int status) {
        for (int s = 0; s < S; ++s) { h_o[s] = 0; c_o[s] = 0; b_o[s] = 0; }
        p.out.total_cost[n] = -1;
        p.out.latency_buckets[n] = -1;
        p.out.status[n] = status;
    };
    if (p.inst_flag[n] != 0) {                            // bad input seen while scoring
        if (tid == 0) write_unsolved(THEMIS_STATUS_BAD_INPUT);
        return;
    }

    if (tid == 0) {
        mbar_init(&mbar[0], 1);
        mbar_init(&mbar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < kPadChunks * CS; i += NT) Fw[i] = kInf16x2;
    for (int i = tid; i < THEMIS_MAX_STAGES; i += NT) stage_lmin[i] = 0xFFFFFFFFu;
    for (int l = pitch + tid; l < Tp; l += NT) {
        Gbuf0[l] = kInf16x2;
        Gbuf1[l] = kInf16x2;
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
    int failed = 0;                                       // a bounded wait ran out
    int pend0 = 0, pend1 = S > 1 ? 0 : -1;                // phase parity of a copy in flight, or -1

    // Stores the thread's H words of F_s to shared memory and to the uint16 table.
    auto store_chunk = [&](const uint32_t (&w)[H], int s) {
        store_words<H>(w, my_chunk);
        if (t0 + R <= pitch)
            store_words<H>(w, reinterpret_cast<uint32_t *>(F16_inst + (size_t)s * pitch + t0));
    };

    // stage 0: F_0 = G_0
    if (!mbar_wait(&mbar[0], 0)) failed = 1; else pend0 = -1;
    // Records the lowest reachable index among this thread's R entries of row s.
    auto note_first_reachable = [&](uint32_t first, int s) {
        first = __reduce_min_sync(0xFFFFFFFFu, first);
        if ((tid & 31) == 0 && first != 0xFFFFFFFFu) atomicMin(&stage_lmin[s], first);
    };
    {
        uint32_t w[H], first = 0xFFFFFFFFu;
#pragma unroll
        for (int r = H - 1; r >= 0; --r) {
            // raw costs; entries beyond the loaded row hold kInf16x2, far above kInf16
            const uint32_t lo = min(Gbuf0[t0 + 2 * r], kInf16), hi = min(Gbuf0[t0 + 2 * r + 1], kInf16);
            w[r] = lo | (hi << 16);
            if (hi < kInf16) first = (uint32_t)(t0 + 2 * r + 1);
            if (lo < kInf16) first = (uint32_t)(t0 + 2 * r);
        }
        note_first_reachable(first, 0);
        store_chunk(w, 0);
        if (tid < n_extra) {
            const uint32_t v = min(Gbuf0[Tc + tid], kInf16);
            fx_prev[tid] = v;
            F16_inst[Tc + tid] = (uint16_t)v;
        }
    }
    failed = __syncthreads_or(failed);
    // Half-word i (< Tc) of the prefix table in shared memory.
    auto f_at = [&](int i) -> uint32_t {
        const uint32_t w = Fw[(kPadChunks + i / R) * CS + ((i % R) >> 1)];
        return (i & 1) ? (w >> 16) : (w & 0xFFFFu);
    };
    // Lowest reachable budget of the prefix F_{s-1} (0xFFFFFFFF: nothing reachable).  Everything
    // below it, and every G_s[l] below that row's first reachable l, can only give "unreachable".
    uint32_t prefix_min = stage_lmin[0];

    for (int s = 1; s < S && !failed; ++s) {
        const int cur = s & 1;
        uint32_t *Gk = cur ? Gbuf1 : Gbuf0;
        const int parity = (s >> 1) & 1;
        if (!mbar_wait(&mbar[cur], (uint32_t)parity)) failed = 1;
        else if (cur) pend1 = -1; else pend0 = -1;
        // raw costs -> saturated cost duplicated into both half-words, in place
        {
            uint32_t first = 0xFFFFFFFFu;
            if (t0 < pitch) {
#pragma unroll
                for (int r = R - 1; r >= 0; --r) {
                    const uint32_t v = min(Gk[t0 + r], kInf16);
                    Gk[t0 + r] = v | (v << 16);
                    if (v < kInf16) first = (uint32_t)(t0 + r);
                }
            }
            note_first_reachable(first, s);
            if (EXTRA && tid < kMaxExtra) fx_acc[tid] = 0xFFFFFFFFu;
        }
        failed = __syncthreads_or(failed);                // G_s and F_{s-1} visible to all
        if (failed) break;
        if (s + 1 < S) {                                  // the other buffer is free again
            const int nxt = cur ^ 1;
            if (tid == 0) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_expect_tx(&mbar[nxt], row_bytes);
                bulk_load(nxt ? Gbuf1 : Gbuf0, G_inst + (size_t)(s + 1) * pitch, row_bytes, &mbar[nxt]);
            }
            if (nxt) pend1 = ((s + 1) >> 1) & 1; else pend0 = ((s + 1) >> 1) & 1;
        }

        uint32_t acc[H], accp[H], wa[H], wb[H];
#pragma unroll
        for (int r = 0; r < H; ++r) { acc[r] = 0xFFFFFFFFu; accp[r] = 0xFFFFFFFFu; }
        // All lanes of a warp walk the same l so that G is a broadcast; lanes that run
        // past their own range read the "unreachable" chunks in front of F[0].  Chunks of
        // l below G_s's first reachable entry, and chunks that only meet F_{s-1} below its
        // first reachable budget, are skipped (whole steps of U chunks, block-uniform).
        const uint32_t g_min = stage_lmin[s];
        const bool dead = g_min == 0xFFFFFFFFu || prefix_min == 0xFFFFFFFFu;
        const int q_lo = dead ? 0 : (int)(g_min / R) & ~(U - 1);
        const int q_hi = dead ? -1 : (tile | 31) - ((int)(prefix_min / R) & ~(U - 1));
        if (q_lo <= q_hi) {
            const uint32_t *f_hi = my_chunk - q_lo * CS;  // chunk tile - q_lo: at worst a pad chunk
#pragma unroll
            for (int r = 0; r < H; ++r) wa[r] = f_hi[r];
            const uint32_t *f_lo = f_hi - CS;
            const uint32_t *g = Gk + q_lo * R;
            for (int q = q_lo; q <= q_hi; q += U) {
#pragma unroll
                for (int u = 0; u < U; u += 2) {
                    chunk_step16<R>(wa, wb, acc, accp, f_lo - u * CS, g + u * R);
                    chunk_step16<R>(wb, wa, acc, accp, f_lo - (u + 1) * CS, g + (u + 1) * R);
                }
                f_lo -= U * CS;
                g += U * R;
            }
        }
        prefix_min = dead ? 0xFFFFFFFFu : prefix_min + g_min;
        if (EXTRA && n_extra > 0) {
            // Extra cells t = Tc + e: this thread's share of min_l F_{s-1}[t-l] + G_s[l] is its own
            // tile's l range; thread 0 adds l >= Tc (those entries of G are still raw costs).
            uint32_t ex[kMaxExtra];
#pragma unroll
            for (int e = 0; e < kMaxExtra; ++e) ex[e] = 0xFFFFFFFFu;
            for (int r = 0; r < R; ++r) {
                const int l = t0 + r;
                const uint32_t g = Gk[l] & 0xFFFFu;
#pragma unroll
                for (int e = 0; e < kMaxExtra; ++e)
                    if (e < n_extra) {
                        const int i = Tc + e - l;             // >= 1
                        ex[e] = min(ex[e], (i < Tc ? f_at(i) : fx_prev[i - Tc]) + g);
                    }
            }
            if (tid == 0) {
#pragma unroll
                for (int e = 0; e < kMaxExtra; ++e)
                    for (int l = Tc; l <= Tc + e && e < n_extra; ++l)
                        ex[e] = min(ex[e], f_at(Tc + e - l) + min(Gk[l], kInf16));
            }
#pragma unroll
            for (int e = 0; e < kMaxExtra; ++e)
                if (e < n_extra) {
                    const uint32_t m = __reduce_min_sync(0xFFFFFFFFu, ex[e]);
                    if ((tid & 31) == 0) atomicMin(&fx_acc[e], m);
                }
        }
        if ((tid & 31) == 31) xchg[tile >> 5] = accp[H - 1];
        __syncthreads();                                  // every read of F_{s-1} is done

        // merge: cell 2j comes from acc[j].lo and accp[j-1].hi, cell 2j+1 from acc[j].hi and accp[j].lo
        uint32_t left = __shfl_up_sync(0xFFFFFFFFu, accp[H - 1], 1);
        if ((tid & 31) == 0) left = tile == 0 ? 0xFFFFFFFFu : xchg[(tile >> 5) - 1];
        uint32_t w[H];
#pragma unroll
        for (int r = 0; r < H; ++r) {
            const uint32_t odd = __byte_perm(r == 0 ? left : accp[r - 1], accp[r], 0x5432);
            w[r] = __vminu2(__vminu2(acc[r], odd), kInf16x2);
        }
        store_chunk(w, s);
        if (tid < n_extra) {                              // every share arrived before the barrier above
            const uint32_t v = min(fx_acc[tid], kInf16);
            fx_prev[tid] = v;
            F16_inst[(size_t)s * pitch + Tc + tid] = (uint16_t)v;
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

    // final scan: cheapest total, lowest total latency among equals
    uint32_t best = 0xFFFFFFFFu;
#pragma unroll
    for (int r = 0; r < H; ++r) {
        const uint32_t w = my_chunk[r];
        const int t = t0 + 2 * r;
        if (t <= T) best = min(best, ((w & 0xFFFFu) << 16) | (uint32_t)t);
        if (t + 1 <= T) best = min(best, (w & 0xFFFF0000u) | (uint32_t)(t + 1));
    }
    if (tid < n_extra) best = min(best, (fx_prev[tid] << 16) | (uint32_t)(Tc + tid));
    best = block_min(best, red, tid, n_warps);
    const uint32_t best_cost = best >> 16;
    const int tstar = (int)(best & 0xFFFFu);

    if (best_cost >= kInf16) {
        // Infeasible, or a total of at least 32767?  Feasible iff the fastest
        // candidates of all stages fit the budget.
        long long fastest = 0;
        for (int s = 0; s < S; ++s) {
            uint32_t lmin = 0xFFFFFFFFu;
            const int32_t *G_row = G_inst + (size_t)s * pitch;
            for (int l = tid; l <= T; l += NT)
                if (G_row[l] != THEMIS_G_INF) { lmin = (uint32_t)l; break; }
            lmin = block_min(lmin, red, tid, n_warps);
            fastest += lmin == 0xFFFFFFFFu ? (long long)T + 1 : (long long)lmin;
        }
        if (tid == 0) {
            if (fastest > T) write_unsolved(THEMIS_STATUS_INFEASIBLE);
            else p.inst_flag[n] = kFlagNeedsWide;         // results come from the 32-bit kernel
        }
        return;
    }

    // last prefix table as int32 (same table the 32-bit kernel leaves)
    {
        int32_t *F_row = p.F + (size_t)n * pitch;
#pragma unroll
        for (int r = 0; r < H; ++r) {
            const uint32_t w = my_chunk[r];
            const int t = t0 + 2 * r;
            if (t < pitch) {
                F_row[t] = (w & 0xFFFFu) >= kInf16 ? THEMIS_G_INF : (int32_t)(w & 0xFFFFu);
                F_row[t + 1] = (w >> 16) >= kInf16 ? THEMIS_G_INF : (int32_t)(w >> 16);
            }
        }
    }

    if (tid < n_extra)
        p.F[(size_t)n * pitch + Tc + tid] = fx_prev[tid] >= kInf16 ? THEMIS_G_INF : (int32_t)fx_prev[tid];

    // backtrack along the optimal path: lowest l with F_{s-1}[t-l] + G_s[l] == F_s[t]
    int t = tstar;
    uint32_t target = best_cost;
    for (int s = S - 1; s >= 1; --s) {
        const int32_t *G_row = G_inst + (size_t)s * pitch;
        const uint16_t *Fprev = F16_inst + (size_t)(s - 1) * pitch;
        uint32_t cand = 0xFFFFFFFFu;
        for (int l = tid; l <= t; l += NT) {
            const uint32_t g = min((uint32_t)G_row[l], kInf16);
            if ((uint32_t)Fprev[t - l] + g == target) { cand = (uint32_t)l; break; }
        }
        const uint32_t ell = block_min(cand, red, tid, n_warps);
        if (ell > (uint32_t)t) { failed = 1; break; }     // cannot happen for consistent tables
        t -= (int)ell;
        target = Fprev[t];
        if (tid == 0) {
            const int idx = (int)p.Garg[((size_t)n * S + s) * pitch + ell];
            const int C = p.prob.c_max, NB = p.prob.n_batch;
            const int bi = idx % NB, rest = idx / NB;
            b_o[s] = p.prob.batch_sizes[bi];
            c_o[s] = rest % C + 1;
            h_o[s] = p.vertical ? p.replicas[(size_t)n * S + s]
                       : p.horizontal ? G_inst[(size_t)s * pitch + ell] : rest / C + 1;
        }
    }
    if (tid == 0) {
        if (failed) {
            write_unsolved(THEMIS_STATUS_TIMEOUT);
        } else {
            const int idx = (int)p.Garg[(size_t)n * S * pitch + t];
            const int C = p.prob.c_max, NB = p.prob.n_batch;
            const int bi = idx % NB, rest = idx / NB;
            b_o[0] = p.prob.batch_sizes[bi];
            c_o[0] = rest % C + 1;
            h_o[0] = p.vertical ? p.replicas[(size_t)n * S] : p.horizontal ? G_inst[t] : rest / C + 1;
            p.out.total_cost[n] = (int32_t)best_cost;
            p.out.latency_buckets[n] = tstar;
            p.out.status[n] = THEMIS_STATUS_OK;
        }
    }
}

template <int R, int MAXT, bool EXTRA>
cudaError_t launch_variant16x(const Params &p, int threads, size_t smem, cudaStream_t stream)
{
    cudaError_t e = cudaFuncSetAttribute(minplus16_kernel<R, MAXT, EXTRA>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    minplus16_kernel<R, MAXT, EXTRA><<<p.prob.n_instances, threads, smem, stream>>>(p);
    return cudaGetLastError();
}

template <int R, int MAXT>
cudaError_t launch_variant16(const Params &p_in, int threads, size_t smem, cudaStream_t stream)
{
    Params p = p_in;
    assign_warp_groups(threads / 32, p.warp_group);
    return threads * R < p.T + 1 ? launch_variant16x<R, MAXT, true>(p, threads, smem, stream)
                                 : launch_variant16x<R, MAXT, false>(p, threads, smem, stream);
}

}  // namespace

cudaError_t launch_minplus16(const Params &p, int tile, cudaStream_t stream)
{
    const int cells = p.T + 1;
    int R = tile;
    // Finer tiles waste fewer cells past the diagonal (a warp spans 32 tiles and all its lanes
    // run to its longest column) but pay more loads per update: 4 cells per thread up to 1024
    // budget cells, 8 up to 8192, else 16.
    if (R != 4 && R != 8 && R != 16) R = cells <= 1024 + kMaxExtra ? 4 : 8;
    if (R == 4 && (cells - kMaxExtra + 3) / 4 > 1024) R = 8;
    if (R == 8 && (cells - kMaxExtra + 7) / 8 > 1024) R = 16;
    const int chunks = (cells + R - 1) / R;
    int groups = (chunks + 31) / 32;
    // a few cells beyond a whole number of tile groups are handled outside the tiles
    if (groups > 1 && cells - (groups - 1) * 32 * R <= kMaxExtra) --groups;
    const int threads = groups * 32;
    const int CS = R == 16 ? 12 : R / 2;
    const size_t g_words = (size_t)(threads * R > p.pitch ? threads * R : p.pitch);
    const size_t words = (size_t)(kPadChunks + threads) * CS + 2u * g_words + 4 + 32 + 32 + THEMIS_MAX_STAGES +
                         2 * kMaxExtra;
    const size_t smem = words * sizeof(uint32_t);
    if (R == 4)
        return threads <= 512 ? launch_variant16<4, 512>(p, threads, smem, stream)
                              : launch_variant16<4, 1024>(p, threads, smem, stream);
    if (R == 8)
        return threads <= 512 ? launch_variant16<8, 512>(p, threads, smem, stream)
                              : launch_variant16<8, 1024>(p, threads, smem, stream);
    return threads <= 512 ? launch_variant16<16, 512>(p, threads, smem, stream)
                          : launch_variant16<16, 1024>(p, threads, smem, stream);
}

}  // namespace themis

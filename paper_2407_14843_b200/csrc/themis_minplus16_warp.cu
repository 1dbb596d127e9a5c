// Min-plus stage recurrence on packed 16-bit costs for short budgets: one warp per
// instance.
//
//   F_0 = G_0,   F_s[t] = min_{0<=l<=t} F_{s-1}[t-l] + G_s[l]       (Algorithm 1's budget loop)
//
// Values, packing, the prefix tables kept instead of an argmin and the budget limit are
// those of the block kernel (themis_minplus16.cu): half-word costs relative to every row's
// cheapest entry and saturated at 0x7FFF, two budget cells per register, even and odd l in
// two accumulator sets, uint16 prefix tables in the workspace rows, budgets the later
// stages cannot complete left "unreachable".
//
// What differs is the division of work.  With a budget of a thousand buckets a stage is a
// few hundred chunk steps, and a thread block per instance spends a large part of its time
// at its two barriers per stage, with the warps that hold the short columns idle.  Here a
// warp owns the instance: its two half-warps each walk a list of half-groups of 16 tiles
// (dealt longest first, alternately, so that the two lists cost the same within one
// half-group step), all synchronisation is __syncwarp, and the prefix table is double
// buffered in shared memory, so that a finished tile is stored at once instead of waiting
// in registers for a barrier.  The half-word a tile's odd-l accumulators spill into the
// next tile is merged in a pass over the stage's tiles at its end, which also caps the
// values, blanks the budgets above the limit and writes the uint16 row.
//
// A block is a few such warps that share nothing but the launch.
#include "themis_async.cuh"
#include "themis_internal.h"
#include "themis_minplus16_step.cuh"

namespace themis {
namespace {

constexpr uint32_t kInf16x2 = (kInf16 << 16) | kInf16;
// "Unreachable" chunks in front of F[0]: the lanes of a half-group walk to its longest column,
// so the one with the shortest column reads up to 16 chunks below its own first, and the step
// after the last still loads one more.
constexpr int kPadChunks = 18;
// four per-stage arrays (padded to an even number of words) and the barrier
__host__ __device__ inline int meta_words(int S) { return 4 * ((S + 1) & ~1) + 4; }

// Words of shared memory of one warp.
__host__ __device__ inline int warp_words(int R, int n_tiles, int pitch, int S)
{
    const int H = R / 2, CS = (H % 8 == 0) ? H + 4 : H;
    const int Tc = n_tiles * R;
    const int Tp = Tc > pitch ? Tc : pitch;
    return Tp + 2 * (kPadChunks + n_tiles) * CS + n_tiles + meta_words(S);
}

template <int R>
__global__ void __launch_bounds__(128, R == 8 ? 6 : 7)   // 77 and 70 registers: no spills; shared memory allows no more warps anyway
minplus16_warp_kernel(const Params p)
{
    extern __shared__ __align__(128) uint32_t smem[];
    constexpr int H = Tile16<R>::H, CS = Tile16<R>::CS;
    constexpr int U = 64 / R;                             // chunk steps per iteration of the main loop
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = blockIdx.x * (blockDim.x >> 5) + warp;
    if (n >= p.prob.n_instances) return;
    if (p.active && !p.active[n]) return;
    const int T = p.T, pitch = p.pitch, S = p.prob.n_stages;
    const int NHG = p.n_half_groups;
    const int n_tiles = NHG * 16;
    const int Tc = n_tiles * R;
    const int Tp = max(Tc, pitch);
    const int n_dummy = (Tc - (T + 1)) / R;               // tiles in front of cell 0 (right-aligned tiling)
    const int f_words = (kPadChunks + n_tiles) * CS;

    uint32_t *Gk = smem + (size_t)warp * warp_words(R, n_tiles, pitch, S);
    uint32_t *Fbuf0 = Gk + Tp;
    uint32_t *Fbuf1 = Fbuf0 + f_words;
    uint32_t *xchg = Fbuf1 + f_words;                     // every tile's last odd-l word
    uint32_t *stage_lmin = xchg + n_tiles;                // first reachable l of every G_s (0xFFFFFFFF: none)
    const int S2 = (S + 1) & ~1;
    uint32_t *stage_cmin = stage_lmin + S2;               // cheapest entry of every G_s
    uint32_t *later_first = stage_cmin + S2;              // sum of the later stages' first buckets
    uint32_t *ell_of = later_first + S2;                  // backtrack: l_s of the path
    uint64_t *mbar = reinterpret_cast<uint64_t *>(ell_of + S2);

    const int slot = lane >> 4, lane16 = lane & 15;
    const uint32_t row_bytes = (uint32_t)pitch * 4u;
    const int32_t *G_inst = p.G + (size_t)n * S * pitch;
    uint16_t *F16_inst = p.A + (size_t)n * S * pitch;     // prefix tables F_s as uint16 rows

    int32_t *h_o = p.out.h + (size_t)n * S, *c_o = p.out.c + (size_t)n * S, *b_o = p.out.b + (size_t)n * S;
    auto write_unsolved = [&](int status) {               // one lane
        for (int s = 0; s < S; ++s) { h_o[s] = 0; c_o[s] = 0; b_o[s] = 0; }
        p.out.total_cost[n] = -1;
        p.out.latency_buckets[n] = -1;
        p.out.status[n] = status;
    };
    if (p.inst_flag[TH_IDX(801, n, p.prob.n_instances)] == kFlagBadInput) {
        if (lane == 0) write_unsolved(THEMIS_STATUS_BAD_INPUT);
        return;
    }

    if (lane == 0) {
        mbar_init(mbar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = lane; i < 2 * f_words; i += 32) Fbuf0[TH_IDX(802, i, 2 * f_words)] = kInf16x2;
    for (int l = pitch + lane; l < Tp; l += 32) Gk[TH_IDX(803, l, Tp)] = kInf16x2;
    __syncwarp();
    auto fetch_row = [&](int s) {                         // after a __syncwarp: every read of Gk is done
        if (lane == 0) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_expect_tx(mbar, row_bytes);
            bulk_load(Gk, G_inst + (size_t)s * pitch, row_bytes, mbar);
        }
    };
    fetch_row(0);

    // First non-empty bucket of every row, from the table in global memory while row 0 is on
    // its way (eight rows' first 32 buckets in flight at a time): the budget limit of stage s
    // is T minus the sum over the later stages.
    for (int s0 = 0; s0 < S; s0 += 8) {
        int32_t head[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            head[j] = (s0 + j < S && lane <= T) ? G_inst[TH_IDX(804, (size_t)(s0 + j) * pitch + lane, (size_t)S * pitch)]
                                                : THEMIS_G_INF;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (s0 + j >= S) break;
            const int32_t *row = G_inst + (size_t)(s0 + j) * pitch;
            unsigned hit = __ballot_sync(0xFFFFFFFFu, head[j] != THEMIS_G_INF);
            uint32_t first = hit ? (uint32_t)(__ffs((int)hit) - 1) : 0xFFFFFFFFu;
            for (int base = 32; base <= T && !hit; base += 32) {
                const int l = base + lane;
                hit = __ballot_sync(0xFFFFFFFFu, l <= T && row[TH_IDX(832, l, pitch)] != THEMIS_G_INF);
                if (hit) first = (uint32_t)(base + __ffs((int)hit) - 1);
            }
            if (lane == 0) stage_lmin[TH_IDX(805, s0 + j, S)] = first;
        }
    }
    __syncwarp();
    if (lane == 0) {
        uint32_t later = 0;
        for (int s = S - 1; s >= 0; --s) {
            later_first[s] = later;
            const uint32_t own = stage_lmin[s] == 0xFFFFFFFFu ? (uint32_t)T + 1u : stage_lmin[s];
            later = min(later + own, (uint32_t)T + 1u);
        }
    }
    __syncwarp();
    auto half_groups_in_use = [&](int t_max) -> int {
        return t_max < 0 ? 0 : min(NHG, (n_dummy + t_max / R) / 16 + 1);
    };
    // Half-group of this half-warp in round k of a stage that uses the first `nhg` half-groups:
    // round k deals the two longest left, the longer one to slot k & 1.  -1: none.
    auto my_half_group = [&](int k, int nhg) -> int {
        const int a = nhg - 1 - 2 * k;
        return slot == (k & 1) ? a : a - 1;
    };
    auto chunk_in = [&](uint32_t *F, int tile) -> uint32_t * {
        return F + TH_IDX(806, kPadChunks + tile, kPadChunks + n_tiles) * CS;
    };
    // "unreachable" for the cells of a tile above the budget limit
    auto mask_above = [&](uint32_t (&w)[H], int tile, int t_max) {
        const int t0 = (tile - n_dummy) * R;
        if (t0 + R - 1 > t_max) {
#pragma unroll
            for (int r = 0; r < H; ++r) {
                if (t0 + 2 * r > t_max) w[r] = kInf16x2;
                else if (t0 + 2 * r + 1 > t_max) w[r] = (w[r] & 0xFFFFu) | (kInf16 << 16);
            }
        }
    };
    // A tile's H words of F_s to shared memory and to the uint16 table.
    auto store_tile = [&](uint32_t *F, int tile, const uint32_t (&w)[H], int s) {
        store_words<H>(w, chunk_in(F, tile));
        const int t0 = (tile - n_dummy) * R;
        if (t0 >= 0 && t0 + R <= pitch)
            store_words<H>(w, reinterpret_cast<uint32_t *>(
                F16_inst + TH_IDX(807, (size_t)s * pitch + t0, (size_t)S * pitch - R + 1)));
    };
    // "unreachable" for the cells of row s of the uint16 table that no tile in use covers
    auto blank_unused = [&](int s, int nhg_used) {
        const int t_first = max(0, (nhg_used * 16 - n_dummy) * R);
        uint32_t *row = reinterpret_cast<uint32_t *>(F16_inst + (size_t)s * pitch);
        for (int w = t_first / 2 + lane; w < pitch / 2; w += 32) row[TH_IDX(808, w, pitch / 2)] = kInf16x2;
    };
    // Cheapest entry of the raw row in Gk (0xFFFFFFFF... never: an empty row gives THEMIS_G_INF).
    auto row_min = [&]() -> uint32_t {
        uint32_t m = 0xFFFFFFFFu;
        for (int l4 = lane * 4; l4 < pitch; l4 += 128) {
            const uint4 v = *reinterpret_cast<const uint4 *>(Gk + TH_IDX(809, l4, Tp - 3));
            m = min(m, min(min(v.x, v.y), min(v.z, v.w)));
        }
        return __reduce_min_sync(0xFFFFFFFFu, m);
    };

    int failed = 0;
    uint32_t cost_offset = 0;                             // sum of the rows' cheapest entries so far

    // stage 0: F_0 = G_0 relative to its cheapest entry
    failed = __any_sync(0xFFFFFFFFu, !mbar_wait(mbar, 0));
    if (!failed) {
        const uint32_t m = row_min();
        if (lane == 0) stage_cmin[0] = m;
        const uint32_t c_off0 = m >= (uint32_t)THEMIS_G_INF ? 0u : m;
        cost_offset = c_off0;
        const int t_max = T - (int)later_first[0];
        const int nhg_used = half_groups_in_use(t_max);
        blank_unused(0, nhg_used);
        for (int k = 0; 2 * k < nhg_used; ++k) {
            const int hg = my_half_group(k, nhg_used);
            if (hg < 0) continue;
            const int tile = hg * 16 + lane16;
            const int t0 = (tile - n_dummy) * R;
            uint32_t w[H];
#pragma unroll
            for (int r = 0; r < H; ++r) {
                // raw costs; entries beyond the loaded row hold kInf16x2, far above kInf16
                const uint32_t lo = t0 < 0 ? kInf16 : min(Gk[TH_IDX(810, t0 + 2 * r, Tp)] - c_off0, kInf16);
                const uint32_t hi = t0 < 0 ? kInf16 : min(Gk[TH_IDX(811, t0 + 2 * r + 1, Tp)] - c_off0, kInf16);
                w[r] = lo | (hi << 16);
            }
            mask_above(w, tile, t_max);
            store_tile(Fbuf0, tile, w, 0);
        }
        __syncwarp();
        if (S > 1) fetch_row(1);
    }
    uint32_t prefix_min = stage_lmin[0];                  // lowest budget F_{s-1} can reach
    uint32_t *Fprev = Fbuf0, *Fcur = Fbuf1;

    for (int s = 1; s < S && !failed; ++s) {
        failed = __any_sync(0xFFFFFFFFu, !mbar_wait(mbar, (uint32_t)(s & 1)));
        if (failed) break;
        // raw costs -> saturated relative cost duplicated into both half-words, in place
        const uint32_t m = row_min();
        if (lane == 0) stage_cmin[TH_IDX(812, s, S)] = m;
        const uint32_t c_off = m >= (uint32_t)THEMIS_G_INF ? 0u : m;
        cost_offset += c_off;
        for (int l4 = lane * 4; l4 < pitch; l4 += 128) {
            uint4 v4 = *reinterpret_cast<const uint4 *>(Gk + TH_IDX(813, l4, Tp - 3));
            uint32_t *v = reinterpret_cast<uint32_t *>(&v4);
#pragma unroll
            for (int i = 0; i < 4; ++i) v[i] = min(v[i] - c_off, kInf16) * 0x10001u;
            *reinterpret_cast<uint4 *>(Gk + l4) = v4;
        }
        const int t_max = T - (int)later_first[s];
        const int nhg_used = half_groups_in_use(t_max);
        blank_unused(s, nhg_used);
        const uint32_t g_min = stage_lmin[s];
        const bool dead = g_min == 0xFFFFFFFFu || prefix_min == 0xFFFFFFFFu;
        // Chunks of l below G_s's first reachable entry, and chunks that only meet F_{s-1} below
        // its first reachable budget, are skipped (in pairs of chunks).
        const int q_lo = dead ? 0 : (int)(g_min / R) & ~1;
        const int q_shift = dead ? 0 : ((int)(prefix_min / R) + n_dummy) & ~1;   // in tiles
        __syncwarp();                                     // G_s converted; F_{s-1} complete

        uint32_t acc[H], accp[H], wa[H], wb[H];
        const uint32_t *f_lo = Fprev, *g = Gk;
        int tile = 0, remaining = 0, k = 0;
        const int rounds = (nhg_used + 1) / 2;
        // Stores the tile in hand as its accumulators leave it (cell 2j from acc[j].lo and
        // accp[j-1].hi, cell 2j+1 from acc[j].hi and accp[j].lo) and takes the next tile of this
        // half-warp's list that has steps to walk; tiles without any are stored as they are.
        auto next_tile = [&](bool store_current) {
            for (;;) {
                if (store_current) {
                    uint32_t w[H];
#pragma unroll
                    for (int r = 0; r < H; ++r)
                        w[r] = __vminu2(acc[r], __byte_perm(r == 0 ? 0xFFFFFFFFu : accp[r - 1], accp[r], 0x5432));
                    store_words<H>(w, chunk_in(Fcur, tile));
                    xchg[TH_IDX(814, tile, n_tiles)] = accp[H - 1];
                }
                int hg = -1;
                while (k < rounds && hg < 0) hg = my_half_group(k++, nhg_used);
                if (hg < 0) { remaining = 0; return; }
                tile = hg * 16 + lane16;
#pragma unroll
                for (int r = 0; r < H; ++r) { acc[r] = 0xFFFFFFFFu; accp[r] = 0xFFFFFFFFu; }
                remaining = dead ? 0 : max(0, (tile | 15) - q_shift - q_lo + 1);
                store_current = true;
                if (remaining > 0) {
                    const uint32_t *f_hi = chunk_in(Fprev, tile) - q_lo * CS;   // at worst a pad chunk
                    load_words<H>(wa, TH_PTR(815, f_hi, Fprev, f_words - H + 1));
                    f_lo = f_hi - CS;
                    g = Gk + q_lo * R;
                    return;
                }
            }
        };
        next_tile(false);
        // Segments with a warp-uniform trip count: up to the next moment at which a half-warp
        // finishes a tile.
        for (;;) {
            const unsigned n_seg = __reduce_min_sync(0xFFFFFFFFu, remaining > 0 ? (unsigned)remaining : 0xFFFFFFFFu);
            if (n_seg == 0xFFFFFFFFu) break;
            if (remaining > 0) {
                unsigned q = 0;
                for (; q + U <= n_seg; q += U) {
#pragma unroll
                    for (int u = 0; u < U; u += 2) {
                        chunk_step16<R>(wa, wb, acc, accp, TH_PTR(816, f_lo - u * CS, Fprev, f_words - H + 1),
                                        TH_PTR(817, g + u * R, Gk, Tp - R + 1));
                        chunk_step16<R>(wb, wa, acc, accp, TH_PTR(818, f_lo - (u + 1) * CS, Fprev, f_words - H + 1),
                                        TH_PTR(819, g + (u + 1) * R, Gk, Tp - R + 1));
                    }
                    f_lo -= U * CS;
                    g += U * R;
                }
                for (; q < n_seg; q += 2) {               // segments are even, not multiples of U
                    chunk_step16<R>(wa, wb, acc, accp, TH_PTR(820, f_lo, Fprev, f_words - H + 1),
                                    TH_PTR(821, g, Gk, Tp - R + 1));
                    chunk_step16<R>(wb, wa, acc, accp, TH_PTR(822, f_lo - CS, Fprev, f_words - H + 1),
                                    TH_PTR(823, g + R, Gk, Tp - R + 1));
                    f_lo -= 2 * CS;
                    g += 2 * R;
                }
                remaining -= (int)n_seg;
                if (remaining == 0) next_tile(true);
            }
        }
        prefix_min = dead ? 0xFFFFFFFFu : prefix_min + g_min;
        __syncwarp();                                     // every read of G_s is done, every tile stored
        if (s + 1 < S) fetch_row(s + 1);
        // Pass over the stage's tiles: cell 0 also takes the half-word the tile to the left
        // spilled; cap at "unreachable"; blank what lies above the budget limit; uint16 row.
        for (int kk = 0; kk < rounds; ++kk) {
            const int hg = my_half_group(kk, nhg_used);
            if (hg < 0) continue;
            const int tl = hg * 16 + lane16;
            uint32_t w[H];
            load_words<H>(w, chunk_in(Fcur, tl));
            const uint32_t left = tl == 0 ? 0xFFFFFFFFu : xchg[TH_IDX(824, tl - 1, n_tiles)];
            w[0] = __vminu2(w[0], __byte_perm(left, 0xFFFFFFFFu, 0x5432));
#pragma unroll
            for (int r = 0; r < H; ++r) w[r] = __vminu2(w[r], kInf16x2);
            mask_above(w, tl, t_max);
            store_tile(Fcur, tl, w, s);
        }
        __syncwarp();
        uint32_t *t = Fprev; Fprev = Fcur; Fcur = t;      // Fprev: the table just finished
    }

    if (failed) {
        mbar_wait(mbar, 0, 1u << 10);                     // let a late copy land (bounded) before leaving
        if (lane == 0) write_unsolved(THEMIS_STATUS_TIMEOUT);
        return;
    }

    // final scan: cheapest total, lowest total latency among equals (every tile is in use at the
    // last stage: nothing comes after it)
    uint32_t best = 0xFFFFFFFFu;
    for (int hg = slot; hg < NHG; hg += 2) {
        const int tile = hg * 16 + lane16;
        const uint32_t *chunk = chunk_in(Fprev, tile);
#pragma unroll
        for (int r = 0; r < H; ++r) {
            const uint32_t w = chunk[r];
            const int t = (tile - n_dummy) * R + 2 * r;
            if (t < 0) continue;
            if (t <= T) best = min(best, ((w & 0xFFFFu) << 16) | (uint32_t)t);
            if (t + 1 <= T) best = min(best, (w & 0xFFFF0000u) | (uint32_t)(t + 1));
        }
    }
    best = __reduce_min_sync(0xFFFFFFFFu, best);
    const uint32_t best_cost = best >> 16;
    const int tstar = (int)(best & 0xFFFFu);

    if (best_cost >= kInf16) {
        // Infeasible, or a total of at least 32767?  Feasible iff the fastest candidates of all
        // stages fit the budget.
        if (lane == 0) {
            long long fastest = 0;
            for (int s = 0; s < S; ++s)
                fastest += stage_lmin[s] == 0xFFFFFFFFu ? (long long)T + 1 : (long long)stage_lmin[s];
            if (fastest > T) write_unsolved(THEMIS_STATUS_INFEASIBLE);
            else p.inst_flag[n] = kFlagNeedsWide;         // results come from the 32-bit kernel
        }
        return;
    }

    // last prefix table as int32 (same table the 32-bit kernel leaves)
    {
        int32_t *F_row = p.F + (size_t)n * pitch;
        for (int hg = slot; hg < NHG; hg += 2) {
            const int tile = hg * 16 + lane16;
            const uint32_t *chunk = chunk_in(Fprev, tile);
#pragma unroll
            for (int r = 0; r < H; ++r) {
                const uint32_t w = chunk[r];
                const int t = (tile - n_dummy) * R + 2 * r;
                if (t >= 0 && t < pitch) {
                    F_row[TH_IDX(825, t, pitch - 1)] = (w & 0xFFFFu) >= kInf16 ? THEMIS_G_INF : (int32_t)((w & 0xFFFFu) + cost_offset);
                    F_row[t + 1] = (w >> 16) >= kInf16 ? THEMIS_G_INF : (int32_t)((w >> 16) + cost_offset);
                }
            }
        }
    }

    // Backtrack along the optimal path: lowest l with F_{s-1}[t-l] + G_s[l] == F_s[t].  The warp
    // scans l upward, 256 values a round (two 16-byte loads of G per lane), and stops at the
    // first round with a match; the reduction key (l << 16 | F_{s-1}[t-l]) brings the next
    // stage's target along.
    __syncwarp();                                         // the uint16 rows written by other lanes
    int t = tstar;
    uint32_t target = best_cost;
    for (int s = S - 1; s >= 1 && !failed; --s) {
        const int32_t *G_row = G_inst + (size_t)s * pitch;
        const uint16_t *Frow = F16_inst + (size_t)(s - 1) * pitch;
        const uint32_t c_off = stage_cmin[s] >= (uint32_t)THEMIS_G_INF ? 0u : stage_cmin[s];
        uint32_t key = 0xFFFFFFFFu;
        // l below the row's first entry has no candidate (l_first is even a multiple of 4 here)
        for (int base = (int)(stage_lmin[s] & ~3u); base <= t && key == 0xFFFFFFFFu; base += 256) {
            uint32_t cand = 0xFFFFFFFFu;
#pragma unroll
            for (int grp = 1; grp >= 0; --grp) {
                const int l4 = base + (grp * 32 + lane) * 4;
                if (l4 <= t) {
                    const int4 g4 = *reinterpret_cast<const int4 *>(G_row + TH_IDX(826, l4, pitch - 3));
                    const int32_t gv[4] = {g4.x, g4.y, g4.z, g4.w};
#pragma unroll
                    for (int i = 3; i >= 0; --i)
                        if (l4 + i <= t) {
                            const uint32_t f = Frow[TH_IDX(827, t - l4 - i, pitch)];
                            if (f + min((uint32_t)gv[i] - c_off, kInf16) == target) cand = ((uint32_t)(l4 + i) << 16) | f;
                        }
                }
            }
            key = __reduce_min_sync(0xFFFFFFFFu, cand);
        }
        if (key == 0xFFFFFFFFu) { failed = 1; break; }    // cannot happen for consistent tables
        const int ell = (int)(key >> 16);
        if (lane == 0) ell_of[TH_IDX(828, s, S)] = (uint32_t)ell;
        t -= ell;
        target = key & 0xFFFFu;
    }
    if (lane == 0) ell_of[0] = (uint32_t)t;
    __syncwarp();
    if (failed) {
        if (lane == 0) write_unsolved(THEMIS_STATUS_TIMEOUT);
        return;
    }
    // one lane per stage turns (s, l_s) into the stage's configuration
    for (int s = lane; s < S; s += 32) {
        const int ell = (int)ell_of[s];
        const int idx = (int)p.Garg[TH_IDX(829, ((size_t)n * S + s) * pitch + ell, (size_t)p.prob.n_instances * S * pitch)];
        const int C = p.prob.c_max, NB = p.prob.n_batch;
        const int bi = idx % NB, rest = idx / NB;
        b_o[s] = p.prob.batch_sizes[TH_IDX(830, bi, THEMIS_MAX_BATCH_SIZES)];
        c_o[s] = rest % C + 1;
        h_o[s] = p.vertical ? p.replicas[(size_t)n * S + s]
                   : p.horizontal ? G_inst[TH_IDX(831, (size_t)s * pitch + ell, (size_t)S * pitch)] : rest / C + 1;
    }
    if (lane == 0) {
        p.out.total_cost[n] = (int32_t)(best_cost + cost_offset);
        p.out.latency_buckets[n] = tstar;
        p.out.status[n] = THEMIS_STATUS_OK;
    }
}

template <int R>
cudaError_t launch_warp_variant(const Params &p_in, int half_groups, cudaStream_t stream)
{
    static std::atomic<uint64_t> ready{0};
    cudaError_t e = allow_max_smem(reinterpret_cast<const void *>(minplus16_warp_kernel<R>), ready);
    if (e != cudaSuccess) return e;
    Params p = p_in;
    p.n_half_groups = half_groups;
    const size_t warp_bytes = sizeof(uint32_t) * (size_t)warp_words(R, half_groups * 16, p.pitch, p.prob.n_stages);
    int warps = 4;
    while (warps > 1 && warps * warp_bytes > kMaxDynamicSmem) warps >>= 1;
    const int N = p.prob.n_instances;
    minplus16_warp_kernel<R><<<(N + warps - 1) / warps, warps * 32, warps * warp_bytes, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

// Budgets up to this many cells go to the warp kernel (one warp walks the whole triangle of a
// stage: about cells^2 / (2 R^2) chunk steps).  Measured against the block kernel on 8192 and
// 16384 instances of 8 stages: 4 to 11 % faster between 1300 and 1800 cells, even at 2000, 5 to
// 20 % slower from 2200 cells on (shared memory then leaves fewer than three warps a scheduler).
constexpr int kWarpKernelMaxCells = 1900;

bool minplus16_warp_fits(const Params &p, int tile)
{
    if (tile == 16) return false;                         // the warp kernel has tiles of 4 and 8 cells
    return p.T + 1 <= kWarpKernelMaxCells;
}

cudaError_t launch_minplus16_warp(const Params &p, int tile, cudaStream_t stream)
{
    const int cells = p.T + 1;
    const int R = (tile == 4 || tile == 8) ? tile : (cells <= 904 ? 4 : 8);
    const int half_groups = ((cells + R - 1) / R + 15) / 16;
    return R == 4 ? launch_warp_variant<4>(p, half_groups, stream) : launch_warp_variant<8>(p, half_groups, stream);
}

}  // namespace themis

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
// Every row G_s enters relative to its cheapest entry, G_s[l] - min G_s, which
// shifts F_s by the running sum of those minima and changes no argmin: the 15
// bits then only have to hold what the latency budget costs on top of the
// cheapest configurations.  The sum is added back to the reported total and to
// the last prefix table; the stored uint16 tables stay relative.
//
// Packing.  Word k of F holds (F[2k], F[2k+1]).  For an even l = 2e the operand
// pair of output word j, (F[2j-l], F[2j+1-l]), is the aligned word j-e.  For an
// odd l = 2e+1 the same word j-e is the operand pair of outputs (2j+1, 2j+2), so
// every thread keeps two accumulator sets, acc for even l (cells 2j, 2j+1) and
// accp for odd l (cells 2j+1, 2j+2), and merges them once per stage with a
// half-word shift; the half-word that belongs to the next tile travels through
// shared memory.  G is stored with each cost duplicated into both halves.
//
// Argmin.  No argmin is carried.  The prefix tables F_s are kept (uint16, in the
// workspace rows that the 32-bit kernel uses for its argmin tables) and the
// backtrack recovers, stage by stage along the optimal path only, the lowest l
// with F_{s-1}[t-l] + G_s[l] == F_s[t] by a block-wide scan.
//
// Folding.  Tiles are grouped in half-groups of 16 (one per half-warp).  Column length
// grows with the tile index, and all lanes of a half-warp run to their half-group's
// longest column, so half-group g costs g + 1 units.  A half-warp takes a long half-group
// and then a short one, paired so that the two half-warps of every warp carry equal sums
// (a warp runs as long as its longer half): (last, first), (last-1, second), ... when the
// number of half-groups is a multiple of four; otherwise the one or two shortest, or the
// longest, stand alone and the rest is paired the same way (deal_half_groups).  The two
// halves of a warp may stand at different l (two broadcast addresses instead of one).  A
// finished tile's result waits in registers for the stage's barrier; only the word that
// spills into the next tile goes through shared memory.
//
// Budget limit.  A state of stages 0..s can only be completed if the fastest candidates of
// the later stages still fit, so stage s computes budgets up to T minus the sum of the
// later stages' first non-empty buckets only; the half-groups above that limit are not
// walked (they are the longest columns) and the remaining ones are dealt anew every stage.
//
// Saturation.  If the best total is 0x7FFF the instance is either infeasible
// (decided exactly: the fastest configurations of all stages do not fit the
// budget) or too expensive for 16 bits; the latter is flagged and redone by the
// 32-bit kernel in a second launch.
#include "themis_async.cuh"
#include "themis_internal.h"
#include "themis_minplus16_step.cuh"

namespace themis {
namespace {

constexpr uint32_t kInf16x2 = (kInf16 << 16) | kInf16;
constexpr int kPadChunks = 32;   // "unreachable" chunks in front of F[0]: one per lane of a warp
// Budgets just above a whole number of tile groups (T a power of two gives T + 1 cells) would cost
// a whole extra warp walking the longest columns for a handful of cells.  Up to this many cells
// beyond the last full group are instead computed by a block-wide reduction per stage.
constexpr int kMaxExtra = 8;

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
__global__ void __launch_bounds__(MAXT, (R == 16 || MAXT > 512) ? 1 : 2)   // 64 registers: two blocks of 512
minplus16_kernel(const Params p)
{
    extern __shared__ __align__(128) uint32_t smem[];
    constexpr int H = Tile16<R>::H, CS = Tile16<R>::CS;
    constexpr int U = R == 16 ? 2 : 64 / R;               // chunk steps per iteration of the main loop
    const int n = blockIdx.x;
    if (p.active && !p.active[n]) return;
    const int tid = threadIdx.x;
    const int NT = blockDim.x;
    const int n_warps = NT >> 5;
    const int T = p.T, pitch = p.pitch, S = p.prob.n_stages;
    const int NHG = p.n_half_groups;                      // half-groups of 16 tiles
    const int n_tiles = NHG * 16;
    const int Tc = n_tiles * R;                           // cells covered by the tiles
    const int Tp = max(Tc, pitch);                        // length of the G buffers
    const int n_extra = EXTRA ? max(0, T + 1 - Tc) : 0;   // cells beyond the tiles, at most kMaxExtra
    // The tiling is right-aligned: the first n_dummy tiles lie in front of cell 0 and stay
    // "unreachable", so that the columns the padding adds are the shortest, not the longest.
    const int n_dummy = max(0, Tc - (T + 1)) / R;

    uint32_t *Fw = smem;                                  // (kPadChunks + n_tiles) chunks of CS words
    uint32_t *Gbuf0 = Fw + (kPadChunks + n_tiles) * CS;
    uint32_t *Gbuf1 = Gbuf0 + Tp;
    uint32_t *xchg = Gbuf1 + Tp;                          // n_tiles words: every tile's last odd-l word
    uint64_t *mbar = reinterpret_cast<uint64_t *>(xchg + n_tiles);
    uint32_t *red = reinterpret_cast<uint32_t *>(mbar + 2);   // 32 words
    uint32_t *stage_lmin = red + 32;                          // 64 words: first reachable l of every G_s
    uint32_t *fx_prev = stage_lmin + THEMIS_MAX_STAGES;       // kMaxExtra words: F_{s-1} at the extra cells
    uint32_t *fx_acc = fx_prev + kMaxExtra;                   // kMaxExtra words: F_s at the extra cells, building
    uint32_t *stage_cmin = fx_acc + kMaxExtra;                // 64 words: cheapest entry of every G_s
    uint32_t *later_first = stage_cmin + THEMIS_MAX_STAGES;   // 64 words: sum over the later stages of their
                                                              // first non-empty bucket (T + 1 if a stage is empty)

    // The two tiles of this thread in the stage in hand: its half-warp takes one half-group
    // (long columns) and then another (short columns); either may be absent.  Only the budgets
    // a stage can still complete are computed (see budget_limit below), so the half-groups in
    // use, and with them the pairing, change from stage to stage (deal_half_groups).
    const int slot = tid >> 4, lane16 = tid & 15;
    bool has_a = false, has_b = false;
    int tile_a = 0, tile_b = 0;
    // Deals the first `nhg` half-groups (half-group g costs g + 1 units) to the block's half-warp
    // slots, at most two each, so that the sum over warps of the longer of a warp's two halves is
    // smallest: pair longest with shortest, after setting aside the shortest (count = 1 mod 4),
    // the two shortest (2 mod 4) or the longest (3 mod 4) as slots of their own behind the pairs
    // (their sums are equal to the pairs' or below), so that the two halves of a warp are equal or
    // nearly so.  Found optimal by exhaustive search for up to 13 half-groups and within half a
    // unit of the ideal (half the total) beyond.
    auto deal_half_groups = [&](int nhg) {
        int lo = 0, hi = nhg - 1, single0 = -1, single1 = -1;
        if ((nhg & 3) == 1) single0 = lo++;
        if ((nhg & 3) == 2) { single1 = lo++; single0 = lo++; }   // the longer of the two first
        if ((nhg & 3) == 3) single0 = hi--;
        const int pairs = (hi - lo + 1) / 2;
        has_b = slot < pairs;
        const int hg_a = has_b ? hi - slot : slot == pairs ? single0 : slot == pairs + 1 ? single1 : -1;
        has_a = hg_a >= 0;
        tile_a = hg_a * 16 + lane16;
        tile_b = (lo + slot) * 16 + lane16;
    };
    const uint32_t row_bytes = (uint32_t)pitch * 4u;
    const int32_t *G_inst = p.G + (size_t)n * S * pitch;
    uint16_t *F16_inst = p.A + (size_t)n * S * pitch;     // prefix tables F_s as uint16 rows
    const int f_words = (kPadChunks + n_tiles) * CS;      // words of F in shared memory
    (void)f_words;
    auto chunk_of = [&](int tile) -> uint32_t * { return Fw + TH_IDX(201, kPadChunks + tile, kPadChunks + n_tiles) * CS; };

    int32_t *h_o = p.out.h + (size_t)n * S, *c_o = p.out.c + (size_t)n * S, *b_o = p.out.b + (size_t)n * S;
    auto write_unsolved = [&](int status) {
        for (int s = 0; s < S; ++s) { h_o[s] = 0; c_o[s] = 0; b_o[s] = 0; }
        p.out.total_cost[TH_IDX(202, n, p.prob.n_instances)] = -1;
        p.out.latency_buckets[n] = -1;
        p.out.status[n] = status;
    };
    if (p.inst_flag[TH_IDX(203, n, p.prob.n_instances)] == kFlagBadInput) {   // bad input seen while scoring (a leftover
                                                          // kFlagNeedsWide of an earlier pass is re-decided below)
        if (tid == 0) write_unsolved(THEMIS_STATUS_BAD_INPUT);
        return;
    }

    if (tid == 0) {
        mbar_init(&mbar[0], 1);
        mbar_init(&mbar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // every half-word of F stays at or below kInf16 from here on (tiles a stage does not use keep
    // an older, equally harmless value), so sums with an "unreachable" G never wrap
    for (int i = tid; i < (kPadChunks + n_tiles) * CS; i += NT) Fw[i] = kInf16x2;
    for (int i = tid; i < THEMIS_MAX_STAGES; i += NT) stage_cmin[i] = 0xFFFFFFFFu;
    for (int l = pitch + tid; l < Tp; l += NT) {
        Gbuf0[TH_IDX(204, l, Tp)] = kInf16x2;
        Gbuf1[TH_IDX(205, l, Tp)] = kInf16x2;
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

    // Budget limit.  A state of stages 0..s with budget t can only be completed if the fastest
    // candidates of the later stages still fit: t <= T - sum over later stages of their first
    // non-empty bucket.  Budgets above that limit are never part of a solution and are not
    // computed: the uint16 table holds kInf16 there.  The first non-empty buckets are read from
    // the table in global memory (the rows reach shared memory one at a time), a warp per row,
    // while the first two rows are on their way.
    for (int s = tid >> 5; s < S; s += n_warps) {
        const int32_t *row = G_inst + (size_t)s * pitch;
        uint32_t first = (uint32_t)T + 1u;
        for (int base = 0; base <= T; base += 32) {
            const int l = base + (tid & 31);
            const unsigned hit = __ballot_sync(0xFFFFFFFFu, l <= T && row[TH_IDX(206, l, pitch)] != THEMIS_G_INF);
            if (hit) { first = (uint32_t)(base + __ffs((int)hit) - 1); break; }
        }
        if ((tid & 31) == 0) {
            later_first[TH_IDX(207, s, THEMIS_MAX_STAGES)] = first;
            stage_lmin[s] = first > (uint32_t)T ? 0xFFFFFFFFu : first;   // also the bound the stage skips by
        }
    }
    __syncthreads();
    if (tid == 0) {
        uint32_t later = 0;
        for (int s = S - 1; s >= 0; --s) {
            const uint32_t own = later_first[s];
            later_first[s] = later;
            later = min(later + own, (uint32_t)T + 1u);
        }
    }
    __syncthreads();
    auto budget_limit = [&](int s) -> int { return T - (int)later_first[s]; };          // -1: nothing
    auto half_groups_in_use = [&](int t_max) -> int { return t_max < 0 ? 0 : min(NHG, (n_dummy + t_max / R) / 16 + 1); };
    // "unreachable" for the cells of row s of the uint16 table that no tile in use covers
    auto blank_unused = [&](int s, int nhg_used) {
        const int t_first = max(0, (nhg_used * 16 - n_dummy) * R);
        uint32_t *row = reinterpret_cast<uint32_t *>(F16_inst + (size_t)s * pitch);
        for (int w = t_first / 2 + tid; w < pitch / 2; w += NT)
            row[TH_IDX(208, (size_t)s * (pitch / 2) + w, (size_t)S * (pitch / 2)) - (size_t)s * (pitch / 2)] = kInf16x2;
    };
    // "unreachable" for the cells of a tile above the budget limit (only the last tiles in use reach it)
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

    // Stores a tile's H words of F_s to shared memory and to the uint16 table.
    auto store_chunk = [&](int tile, const uint32_t (&w)[H], int s) {
        store_words<H>(w, chunk_of(tile));
        const int t0 = (tile - n_dummy) * R;
        if (t0 >= 0 && t0 + R <= pitch)
            store_words<H>(w, reinterpret_cast<uint32_t *>(
                F16_inst + TH_IDX(209, (size_t)s * pitch + t0, (size_t)S * pitch - R + 1)));
    };

    // The kernel works on costs relative to every row's cheapest entry, G_s[l] - min G_s, so that
    // the 15 bits hold the cost paid beyond the cheapest configurations rather than the whole
    // total.  note_row_cmin adds this thread's share of the raw row s in Gk to stage_cmin[s]
    // (complete after the next block barrier); row_cmin reads it (0 for a row without a candidate).
    auto note_row_cmin = [&](const uint32_t *Gk, int s) {
        uint32_t m = 0xFFFFFFFFu;
        for (int l4 = tid * 4; l4 < pitch; l4 += NT * 4) {
            const uint4 v = *reinterpret_cast<const uint4 *>(Gk + TH_IDX(210, l4, Tp - 3));
            m = min(m, min(min(v.x, v.y), min(v.z, v.w)));
        }
        m = __reduce_min_sync(0xFFFFFFFFu, m);
        if ((tid & 31) == 0) atomicMin(&stage_cmin[s], m);
    };
    auto row_cmin = [&](int s) -> uint32_t {
        const uint32_t m = stage_cmin[s];
        return m >= (uint32_t)THEMIS_G_INF ? 0u : m;
    };
    uint32_t cost_offset = 0;                             // sum of the rows' cheapest entries so far

    // stage 0: F_0 = G_0 (relative to its cheapest entry); both first rows are waited for here
    if (!mbar_wait(&mbar[0], 0)) failed = 1; else pend0 = -1;
    note_row_cmin(Gbuf0, 0);
    if (S > 1) {
        if (!mbar_wait(&mbar[1], 0)) failed = 1; else pend1 = -1;
        note_row_cmin(Gbuf1, 1);
    }
    __syncthreads();
    const uint32_t c_off0 = row_cmin(0);
    cost_offset += c_off0;
    {
        const int t_max = budget_limit(0);
        const int nhg_used = half_groups_in_use(t_max);
        deal_half_groups(nhg_used);
        blank_unused(0, nhg_used);
        auto init_tile = [&](int tile) {
            const int t0 = (tile - n_dummy) * R;
            uint32_t w[H];
#pragma unroll
            for (int r = H - 1; r >= 0; --r) {
                // raw costs; entries beyond the loaded row hold kInf16x2, far above kInf16
                const uint32_t lo = t0 < 0 ? kInf16 : min(Gbuf0[TH_IDX(211, t0 + 2 * r, Tp)] - c_off0, kInf16);
                const uint32_t hi = t0 < 0 ? kInf16 : min(Gbuf0[TH_IDX(212, t0 + 2 * r + 1, Tp)] - c_off0, kInf16);
                w[r] = lo | (hi << 16);
            }
            mask_above(w, tile, t_max);
            store_chunk(tile, w, 0);
        };
        if (has_a) init_tile(tile_a);
        if (has_b) init_tile(tile_b);
        if (tid < n_extra) {
            const uint32_t v = Tc + tid <= t_max ? min(Gbuf0[TH_IDX(213, Tc + tid, Tp)] - c_off0, kInf16) : kInf16;
            fx_prev[TH_IDX(214, tid, kMaxExtra)] = v;
            F16_inst[TH_IDX(215, Tc + tid, pitch)] = (uint16_t)v;
        }
    }
    failed = __syncthreads_or(failed);
    // Half-word i (< Tc) of the prefix table in shared memory.
    auto f_at = [&](int i) -> uint32_t {
        const uint32_t w = Fw[TH_IDX(216, (kPadChunks + n_dummy + i / R) * CS + ((i % R) >> 1), f_words)];
        return (i & 1) ? (w >> 16) : (w & 0xFFFFu);
    };
    // Lowest budget the prefix F_{s-1} can reach: the sum of the earlier rows' first non-empty
    // buckets (0xFFFFFFFF: nothing reachable).  Everything below it, and every G_s[l] below that
    // row's first non-empty bucket, can only give "unreachable".
    uint32_t prefix_min = stage_lmin[0];

    // `failed` is block-uniform here and after every __syncthreads_or below; between those it is
    // a thread's own, so the loop may only leave at the uniform test.
    for (int s = 1; s < S; ++s) {
        if (s == 1 && failed) break;
        const int cur = s & 1;
        uint32_t *Gk = cur ? Gbuf1 : Gbuf0;
        // raw costs -> saturated relative cost duplicated into both half-words, in place
        // (the row has arrived and its cheapest entry is known: see the end of the stage before)
        const uint32_t c_off = row_cmin(s);
        cost_offset += c_off;
        {
            for (int l4 = tid * 4; l4 < pitch; l4 += NT * 4) {
                uint4 v4 = *reinterpret_cast<const uint4 *>(Gk + TH_IDX(217, l4, Tp - 3));
                uint32_t *v = reinterpret_cast<uint32_t *>(&v4);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t c = min(v[i] - c_off, kInf16);
                    v[i] = c * 0x10001u;
                }
                *reinterpret_cast<uint4 *>(Gk + TH_IDX(218, l4, Tp - 3)) = v4;
            }
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

        const int t_max = budget_limit(s);
        const int nhg_used = half_groups_in_use(t_max);
        deal_half_groups(nhg_used);                       // this stage's tiles: budgets up to the limit only
        blank_unused(s, nhg_used);
        const bool extra_in_use = EXTRA && n_extra > 0 && Tc <= t_max;
        uint32_t acc[H], accp[H], wa[H], wb[H];
        // All lanes of a half-warp walk the same l so that G is a broadcast; lanes that run
        // past their own range read the "unreachable" chunks in front of F[0].  Chunks of
        // l below G_s's first reachable entry, and chunks that only meet F_{s-1} below its
        // first reachable budget, are skipped (pairs of chunks, block-uniform).
        const uint32_t g_min = stage_lmin[s];
        const bool dead = g_min == 0xFFFFFFFFu || prefix_min == 0xFFFFFFFFu;
        const int q_lo = dead ? 0 : (int)(g_min / R) & ~1;
        const int q_shift = dead ? 0 : ((int)(prefix_min / R) + n_dummy) & ~1;   // in tiles
        auto steps_of = [&](int tile) { return dead ? 0 : max(0, (tile | 15) - q_shift - q_lo + 1); };
        const int steps_a = has_a ? steps_of(tile_a) : 0, steps_b = has_b ? steps_of(tile_b) : 0;
        const uint32_t *f_lo = Fw, *g = Gk;
        auto begin_tile = [&](int tile) {
#pragma unroll
            for (int r = 0; r < H; ++r) { acc[r] = 0xFFFFFFFFu; accp[r] = 0xFFFFFFFFu; }
            const uint32_t *f_hi = chunk_of(tile) - q_lo * CS;   // chunk tile - q_lo: at worst a pad chunk
            if (steps_of(tile) > 0) load_words<H>(wa, TH_PTR(219, f_hi, Fw, f_words - H + 1));
            f_lo = f_hi - CS;
            g = Gk + q_lo * R;
        };
        // Parks a finished tile in registers: cell 2j comes from acc[j].lo and accp[j-1].hi, cell
        // 2j+1 from acc[j].hi and accp[j].lo.  The last odd-l word also holds cell 0 of the tile to
        // the right, which picks it up from shared memory after the barrier.
        uint32_t res_a[H], res_b[H];
        auto park_tile = [&](uint32_t (&dst)[H], int tile) {
#pragma unroll
            for (int r = 0; r < H; ++r)
                dst[r] = __vminu2(acc[r], __byte_perm(r == 0 ? 0xFFFFFFFFu : accp[r - 1], accp[r], 0x5432));
            xchg[TH_IDX(220, tile, n_tiles)] = accp[H - 1];
        };
        int phase = 0, remaining = steps_a;          // phase 0: first tile, 1: second tile, 2: done
        if (has_a) begin_tile(tile_a);
        auto advance = [&]() {
            while (phase < 2 && remaining == 0) {
                if (phase == 0 && has_a) park_tile(res_a, tile_a);
                if (phase == 1 && has_b) park_tile(res_b, tile_b);
                ++phase;
                if (phase == 1 && has_b) { begin_tile(tile_b); remaining = steps_b; }
            }
        };
        advance();
        // Segments with a warp-uniform trip count: up to the next moment at which a half-warp
        // finishes a tile (both halves on long tiles; one long, one short; both on short tiles).
        for (;;) {
            const unsigned n_seg = __reduce_min_sync(0xFFFFFFFFu, remaining > 0 ? (unsigned)remaining : 0xFFFFFFFFu);
            if (n_seg == 0xFFFFFFFFu) break;
            if (remaining > 0) {
                unsigned q = 0;
                for (; q + U <= n_seg; q += U) {
#pragma unroll
                    for (int u = 0; u < U; u += 2) {
                        chunk_step16<R>(wa, wb, acc, accp, TH_PTR(221, f_lo - u * CS, Fw, f_words - H + 1),
                                        TH_PTR(222, g + u * R, Gk, Tp - R + 1));
                        chunk_step16<R>(wb, wa, acc, accp, TH_PTR(223, f_lo - (u + 1) * CS, Fw, f_words - H + 1),
                                        TH_PTR(224, g + (u + 1) * R, Gk, Tp - R + 1));
                    }
                    f_lo -= U * CS;
                    g += U * R;
                }
                for (; q < n_seg; q += 2) {               // segments are even, not multiples of U
                    chunk_step16<R>(wa, wb, acc, accp, TH_PTR(225, f_lo, Fw, f_words - H + 1), TH_PTR(226, g, Gk, Tp - R + 1));
                    chunk_step16<R>(wb, wa, acc, accp, TH_PTR(227, f_lo - CS, Fw, f_words - H + 1),
                                    TH_PTR(228, g + R, Gk, Tp - R + 1));
                    f_lo -= 2 * CS;
                    g += 2 * R;
                }
                remaining -= (int)n_seg;
                advance();
            }
        }
        prefix_min = dead ? 0xFFFFFFFFu : prefix_min + g_min;
        if (extra_in_use) {
            // Extra cells t = Tc + e (every tile is in use then): this thread's share of min_l F_{s-1}[t-l] + G_s[l] is its own
            // tile's l range; thread 0 adds l >= Tc.
            uint32_t ex[kMaxExtra];
#pragma unroll
            for (int e = 0; e < kMaxExtra; ++e) ex[e] = 0xFFFFFFFFu;
            auto share_of_tile = [&](int tile) {
                for (int r = 0; r < R; ++r) {
                    const int l = tile * R + r;
                    const uint32_t gl = Gk[TH_IDX(229, l, Tp)] & 0xFFFFu;
#pragma unroll
                    for (int e = 0; e < kMaxExtra; ++e)
                        if (e < n_extra) {
                            const int i = Tc + e - l;         // >= 1
                            ex[e] = min(ex[e], (i < Tc ? f_at(i) : fx_prev[TH_IDX(230, i - Tc, kMaxExtra)]) + gl);
                        }
                }
            };
            if (has_a) share_of_tile(tile_a);
            if (has_b) share_of_tile(tile_b);
            if (tid == 0) {
#pragma unroll
                for (int e = 0; e < kMaxExtra; ++e)
                    for (int l = Tc; l <= Tc + e && e < n_extra; ++l)
                        ex[e] = min(ex[e], f_at(Tc + e - l) + (Gk[TH_IDX(231, l, Tp)] & 0xFFFFu));
            }
#pragma unroll
            for (int e = 0; e < kMaxExtra; ++e)
                if (e < n_extra) {
                    const uint32_t m = __reduce_min_sync(0xFFFFFFFFu, ex[e]);
                    if ((tid & 31) == 0) atomicMin(&fx_acc[e], m);
                }
        }
        if (s + 1 < S) {                                  // the next row arrived long ago: its cheapest entry
            const int nxt = cur ^ 1;
            if (!mbar_wait(&mbar[nxt], (uint32_t)(((s + 1) >> 1) & 1))) failed = 1;
            else if (nxt) pend1 = -1; else pend0 = -1;
            note_row_cmin(nxt ? Gbuf1 : Gbuf0, s + 1);
        }
        __syncthreads();                                  // every read of F_{s-1} is done, every tile parked

        auto finish_tile = [&](uint32_t (&w)[H], int tile) {
            const uint32_t left = tile == 0 ? 0xFFFFFFFFu : xchg[TH_IDX(232, tile - 1, n_tiles)];
            w[0] = __vminu2(w[0], __byte_perm(left, 0xFFFFFFFFu, 0x5432));
#pragma unroll
            for (int r = 0; r < H; ++r) w[r] = __vminu2(w[r], kInf16x2);
            mask_above(w, tile, t_max);
            store_chunk(tile, w, s);
        };
        if (has_a) finish_tile(res_a, tile_a);
        if (has_b) finish_tile(res_b, tile_b);
        if (tid < n_extra) {                              // every share arrived before the barrier above
            const uint32_t v = extra_in_use && Tc + tid <= t_max ? min(fx_acc[tid], kInf16) : kInf16;
            fx_prev[tid] = v;
            F16_inst[TH_IDX(233, (size_t)s * pitch + Tc + tid, (size_t)S * pitch)] = (uint16_t)v;
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
    auto scan_tile = [&](int tile) {
        const uint32_t *chunk = chunk_of(tile);
#pragma unroll
        for (int r = 0; r < H; ++r) {
            const uint32_t w = chunk[r];
            const int t = (tile - n_dummy) * R + 2 * r;
            if (t < 0) continue;
            if (t <= T) best = min(best, ((w & 0xFFFFu) << 16) | (uint32_t)t);
            if (t + 1 <= T) best = min(best, (w & 0xFFFF0000u) | (uint32_t)(t + 1));
        }
    };
    if (has_a) scan_tile(tile_a);
    if (has_b) scan_tile(tile_b);
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
                if (G_row[TH_IDX(234, l, pitch)] != THEMIS_G_INF) { lmin = (uint32_t)l; break; }
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
        auto write_tile = [&](int tile) {
            const uint32_t *chunk = chunk_of(tile);
#pragma unroll
            for (int r = 0; r < H; ++r) {
                const uint32_t w = chunk[r];
                const int t = (tile - n_dummy) * R + 2 * r;
                if (t >= 0 && t < pitch) {
                    F_row[TH_IDX(235, t, pitch - 1)] = (w & 0xFFFFu) >= kInf16 ? THEMIS_G_INF : (int32_t)((w & 0xFFFFu) + cost_offset);
                    F_row[t + 1] = (w >> 16) >= kInf16 ? THEMIS_G_INF : (int32_t)((w >> 16) + cost_offset);
                }
            }
        };
        if (has_a) write_tile(tile_a);
        if (has_b) write_tile(tile_b);
    }

    if (tid < n_extra)
        p.F[TH_IDX(236, (size_t)n * pitch + Tc + tid, (size_t)p.prob.n_instances * pitch)] =
            fx_prev[tid] >= kInf16 ? THEMIS_G_INF : (int32_t)(fx_prev[tid] + cost_offset);

    // backtrack along the optimal path: lowest l with F_{s-1}[t-l] + G_s[l] == F_s[t].
    // The block scans l upward, kScanGroups * 4 * NT values a round (four consecutive l per
    // thread and group: one 16-byte load of G), and stops at the first round with a match.
    // The reduction key (l << 16 | F_{s-1}[t-l]) brings the next stage's target along;
    // the two reduction buffers alternate, so a round costs one barrier.
    constexpr int kScanGroups = 2;
    int t = tstar;
    uint32_t target = best_cost;
    uint32_t *red_alt = stage_lmin;                       // the stage minima are no longer needed
    uint32_t *ell_of = Gbuf0;                             // the G buffers are free: l_s of the path
    int round = 0;
    for (int s = S - 1; s >= 1 && !failed; --s) {
        const int32_t *G_row = G_inst + (size_t)s * pitch;
        const uint16_t *Fprev = F16_inst + (size_t)(s - 1) * pitch;
        const uint32_t c_off = stage_cmin[s] >= (uint32_t)THEMIS_G_INF ? 0u : stage_cmin[s];
        uint32_t key = 0xFFFFFFFFu;
        for (int base = 0; base <= t; base += kScanGroups * 4 * NT) {
            uint32_t cand = 0xFFFFFFFFu;
#pragma unroll
            for (int k = kScanGroups - 1; k >= 0; --k) {
                const int l4 = base + (k * NT + tid) * 4;
                if (l4 <= t) {
                    const int4 g4 = *reinterpret_cast<const int4 *>(G_row + TH_IDX(237, l4, pitch - 3));   // pitch covers l4 + 3
                    const int32_t gv[4] = {g4.x, g4.y, g4.z, g4.w};
#pragma unroll
                    for (int i = 3; i >= 0; --i)
                        if (l4 + i <= t) {
                            const uint32_t f = Fprev[TH_IDX(238, t - l4 - i, pitch)];
                            if (f + min((uint32_t)gv[i] - c_off, kInf16) == target) cand = ((uint32_t)(l4 + i) << 16) | f;
                        }
                }
            }
            cand = __reduce_min_sync(0xFFFFFFFFu, cand);
            uint32_t *rbuf = (round++ & 1) ? red_alt : red;
            if ((tid & 31) == 0) rbuf[TH_IDX(239, tid >> 5, 32)] = cand;
            __syncthreads();
            key = rbuf[0];
            for (int w = 1; w < n_warps; ++w) key = min(key, rbuf[w]);
            if (key != 0xFFFFFFFFu) break;
        }
        if (key == 0xFFFFFFFFu) { failed = 1; break; }    // cannot happen for consistent tables
        const int ell = (int)(key >> 16);
        if (tid == 0) ell_of[TH_IDX(240, s, Tp)] = (uint32_t)ell;
        t -= ell;
        target = key & 0xFFFFu;
    }
    if (tid == 0) ell_of[0] = (uint32_t)t;
    __syncthreads();
    if (failed) {
        if (tid == 0) write_unsolved(THEMIS_STATUS_TIMEOUT);
        return;
    }
    // one thread per stage turns (s, l_s) into the stage's configuration
    for (int s = tid; s < S; s += NT) {
        const int ell = (int)ell_of[s];
        const int idx = (int)p.Garg[TH_IDX(241, ((size_t)n * S + s) * pitch + ell, (size_t)p.prob.n_instances * S * pitch)];
        const int C = p.prob.c_max, NB = p.prob.n_batch;
        const int bi = idx % NB, rest = idx / NB;
        b_o[s] = p.prob.batch_sizes[TH_IDX(242, bi, THEMIS_MAX_BATCH_SIZES)];
        c_o[s] = rest % C + 1;
        h_o[s] = p.vertical ? p.replicas[(size_t)n * S + s]
                   : p.horizontal ? G_inst[TH_IDX(243, (size_t)s * pitch + ell, (size_t)S * pitch)] : rest / C + 1;
    }
    if (tid == 0) {
        p.out.total_cost[n] = (int32_t)(best_cost + cost_offset);
        p.out.latency_buckets[n] = tstar;
        p.out.status[n] = THEMIS_STATUS_OK;
    }
}

template <int R, int MAXT, bool EXTRA>
cudaError_t launch_variant16x(const Params &p, int threads, size_t smem, cudaStream_t stream)
{
    static std::atomic<uint64_t> ready{0};
    cudaError_t e = allow_max_smem(reinterpret_cast<const void *>(minplus16_kernel<R, MAXT, EXTRA>), ready);
    if (e != cudaSuccess) return e;
    minplus16_kernel<R, MAXT, EXTRA><<<p.prob.n_instances, threads, smem, stream>>>(p);
    return cudaGetLastError();
}

// Shape of a launch: cells per tile, half-groups of 16 tiles, threads (16 per pair of
// half-groups, whole warps), whether a few cells are left to the block-wide reduction.
struct Shape16 { int R, half_groups, threads; bool extra; size_t smem; };

Shape16 shape_of(int cells, int pitch, int tile)
{
    Shape16 sh;
    // Finer tiles waste fewer cells past the diagonal (all lanes of a half-warp run to its
    // longest column) but pay more loads per update: 4 cells per tile up to about 900 budget
    // cells, else 8; 16 only on request.
    sh.R = (tile == 4 || tile == 8 || tile == 16) ? tile : (cells <= 896 + kMaxExtra ? 4 : 8);
    for (;;) {
        const int tiles = (cells + sh.R - 1) / sh.R;
        sh.half_groups = (tiles + 15) / 16;
        sh.extra = false;
        // a few cells beyond a whole number of half-groups are handled outside the tiles
        if (sh.half_groups > 1 && cells - (sh.half_groups - 1) * 16 * sh.R <= kMaxExtra) {
            --sh.half_groups;
            sh.extra = true;
        }
        const int slots = (sh.half_groups + 1) / 2;          // half-warps, two half-groups each
        sh.threads = (slots + 1) / 2 * 32;
        if (sh.threads <= 1024 || sh.R == 16) break;
        sh.R *= 2;
    }
    const int n_tiles = sh.half_groups * 16;
    const int CS = sh.R == 16 ? 12 : sh.R / 2;
    const size_t g_words = (size_t)(n_tiles * sh.R > pitch ? n_tiles * sh.R : pitch);
    const size_t words = (size_t)(kPadChunks + n_tiles) * CS + 2u * g_words + (size_t)n_tiles + 4 + 32 +
                         3 * THEMIS_MAX_STAGES + 2 * kMaxExtra;
    sh.smem = words * sizeof(uint32_t);
    return sh;
}

template <int R, int MAXT>
cudaError_t launch_variant16(const Params &p_in, const Shape16 &sh, cudaStream_t stream)
{
    Params p = p_in;
    p.n_half_groups = sh.half_groups;
    return sh.extra ? launch_variant16x<R, MAXT, true>(p, sh.threads, sh.smem, stream)
                    : launch_variant16x<R, MAXT, false>(p, sh.threads, sh.smem, stream);
}

}  // namespace

cudaError_t launch_minplus16(const Params &p, int tile, cudaStream_t stream)
{
    const Shape16 sh = shape_of(p.T + 1, p.pitch, tile);
    if (sh.R == 4)
        return sh.threads <= 512 ? launch_variant16<4, 512>(p, sh, stream) : launch_variant16<4, 1024>(p, sh, stream);
    if (sh.R == 8)
        return sh.threads <= 512 ? launch_variant16<8, 512>(p, sh, stream) : launch_variant16<8, 1024>(p, sh, stream);
    return sh.threads <= 512 ? launch_variant16<16, 512>(p, sh, stream) : launch_variant16<16, 1024>(p, sh, stream);
}

}  // namespace themis

// Min-plus stage recurrence on 32-bit packed keys for short budgets: one warp per instance.
//
//   F_0 = G_0,   F_s[t] = min_{0<=l<=t} F_{s-1}[t-l] + G_s[l],   A_s[t] = lowest such l
//
// Keys, the fused add-min that carries the argmin, the uint16 argmin tables and the walk back
// through them are those of the block kernel (themis_minplus.cu).  The division of work is
// that of the packed warp kernel (themis_minplus16_warp.cu): a warp owns the instance, its two
// half-warps each walk a list of half-groups of 16 tiles (dealt longest first, alternately),
// all synchronisation is __syncwarp, and the prefix table is double buffered in shared memory
// so that a finished tile is stored at once.  Chunks of l below G_s's first reachable entry
// and chunks that only meet F_{s-1} below its first reachable budget are skipped (they can
// only give "unreachable"); every cell of every table is still written.
#include "themis_async.cuh"
#include "themis_internal.h"
#include "themis_minplus_step.cuh"

namespace themis {
namespace {

constexpr int kR = 8;                      // budget cells per thread
constexpr int kCS = kR;                    // words between chunk starts of F in shared memory
constexpr int kPadChunks = 18;             // "unreachable" chunks in front of F[0] (see the packed warp kernel)

// Words of shared memory of one warp.
__host__ __device__ inline int warp_words32(int n_tiles, int pitch, int S)
{
    const int Tc = n_tiles * kR;
    const int Tp = Tc > pitch ? Tc : pitch;
    return Tp + 2 * (kPadChunks + n_tiles) * kCS + ((S + 3) & ~3) + 4;
}

__global__ void __launch_bounds__(128, 4)
minplus_warp_kernel(const Params p)
{
    extern __shared__ __align__(128) uint32_t smem[];
    constexpr int R = kR, CS = kCS;
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

    uint32_t *Gk = smem + (size_t)warp * warp_words32(n_tiles, pitch, S);
    uint32_t *Fbuf0 = Gk + Tp;
    uint32_t *Fbuf1 = Fbuf0 + f_words;
    uint32_t *ell_of = Fbuf1 + f_words;                   // backtrack: l_s of the path
    uint64_t *mbar = reinterpret_cast<uint64_t *>(ell_of + ((S + 3) & ~3));

    const int slot = lane >> 4, lane16 = lane & 15;
    const uint32_t row_bytes = (uint32_t)pitch * 4u;
    const int32_t *G_inst = p.G + (size_t)n * S * pitch;

    int32_t *h_o = p.out.h + (size_t)n * S, *c_o = p.out.c + (size_t)n * S, *b_o = p.out.b + (size_t)n * S;
    auto write_unsolved = [&](int status) {               // one lane
        for (int s = 0; s < S; ++s) { h_o[s] = 0; c_o[s] = 0; b_o[s] = 0; }
        p.out.total_cost[n] = -1;
        p.out.latency_buckets[n] = -1;
        p.out.status[n] = status;
    };
    if (p.only_flagged) {                                 // second pass: only what the packed kernel left over
        if (p.inst_flag[TH_IDX(901, n, p.prob.n_instances)] != kFlagNeedsWide) return;
    } else if (p.inst_flag[n] == kFlagBadInput) {         // bad input seen while scoring
        if (lane == 0) write_unsolved(THEMIS_STATUS_BAD_INPUT);
        return;
    }

    if (lane == 0) {
        mbar_init(mbar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = lane; i < 2 * f_words; i += 32) Fbuf0[TH_IDX(902, i, 2 * f_words)] = kInfKey;
    for (int l = pitch + lane; l < Tp; l += 32) Gk[TH_IDX(903, l, Tp)] = kInfKey | (uint32_t)l;
    __syncwarp();
    auto fetch_row = [&](int s) {                         // after a __syncwarp: every read of Gk is done
        if (lane == 0) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_expect_tx(mbar, row_bytes);
            bulk_load(Gk, G_inst + (size_t)s * pitch, row_bytes, mbar);
        }
    };
    fetch_row(0);
    // Half-group of this half-warp in round k: round k deals the two longest left, the longer
    // one to slot k & 1.  -1: none.
    auto my_half_group = [&](int k) -> int {
        const int a = NHG - 1 - 2 * k;
        return slot == (k & 1) ? a : a - 1;
    };
    const int rounds = (NHG + 1) / 2;
    auto chunk_in = [&](uint32_t *F, int tile) -> uint32_t * {
        return F + TH_IDX(904, kPadChunks + tile, kPadChunks + n_tiles) * CS;
    };
    // Raw costs of the row in Gk -> packed keys, in place; returns the first reachable l
    // (0xFFFFFFFF: none).
    auto to_keys = [&]() -> uint32_t {
        uint32_t first = 0xFFFFFFFFu;
        for (int l4 = lane * 4; l4 < pitch; l4 += 128) {
            uint4 v4 = *reinterpret_cast<const uint4 *>(Gk + TH_IDX(905, l4, Tp - 3));
            uint32_t *v = reinterpret_cast<uint32_t *>(&v4);
#pragma unroll
            for (int i = 3; i >= 0; --i) {
                if (v[i] < kInfCost && l4 + i <= T) first = min(first, (uint32_t)(l4 + i));
                v[i] = (min(v[i], kInfCost) << kIdxBits) | (uint32_t)(l4 + i);
            }
            *reinterpret_cast<uint4 *>(Gk + l4) = v4;
        }
        return __reduce_min_sync(0xFFFFFFFFu, first);
    };

    int failed = __any_sync(0xFFFFFFFFu, !mbar_wait(mbar, 0));
    uint32_t prefix_min = 0xFFFFFFFFu;                    // lowest budget F_{s-1} can reach
    if (!failed) {
        // stage 0: F_0 = G_0
        prefix_min = to_keys();
        __syncwarp();
        for (int k = 0; k < rounds; ++k) {
            const int hg = my_half_group(k);
            if (hg < 0) continue;
            const int tile = hg * 16 + lane16;
            const int t0 = (tile - n_dummy) * R;
            uint32_t *chunk = chunk_in(Fbuf0, tile);
#pragma unroll
            for (int r = 0; r < R; ++r)
                chunk[r] = t0 < 0 ? kInfKey : (Gk[TH_IDX(906, t0 + r, Tp)] & ~kIdxMask);
        }
        __syncwarp();
        if (S > 1) fetch_row(1);
    }
    uint32_t *Fprev = Fbuf0, *Fcur = Fbuf1;

    for (int s = 1; s < S && !failed; ++s) {
        failed = __any_sync(0xFFFFFFFFu, !mbar_wait(mbar, (uint32_t)(s & 1)));
        if (failed) break;
        const uint32_t g_min = to_keys();
        const bool dead = g_min == 0xFFFFFFFFu || prefix_min == 0xFFFFFFFFu;
        const int q_lo = dead ? 0 : (int)(g_min / R) & ~1;
        const int q_shift = dead ? 0 : ((int)(prefix_min / R) + n_dummy) & ~1;   // in tiles
        uint16_t *A_row = p.A + ((size_t)n * S + s) * pitch;
        __syncwarp();                                     // keys of G_s and F_{s-1} complete

        uint32_t acc[R], wa[R], wb[R];
        const uint32_t *f_lo = Fprev, *g = Gk;
        int tile = 0, remaining = 0, k = 0;
        // Stores the tile in hand (keys to the table in shared memory, argmins to the uint16 row)
        // and takes the next tile of this half-warp's list that has steps to walk; tiles without
        // any are stored as "unreachable" right away.
        auto next_tile = [&](bool store_current) {
            for (;;) {
                if (store_current) {
                    uint32_t *chunk = chunk_in(Fcur, tile);
                    uint32_t a16[R];
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const bool inf = acc[r] >= kInfKey;
                        chunk[r] = inf ? kInfKey : (acc[r] & ~kIdxMask);
                        a16[r] = inf ? 0u : (acc[r] & kIdxMask);
                    }
                    const int t0 = (tile - n_dummy) * R;
                    if (t0 >= 0 && t0 + R <= pitch)
                        *reinterpret_cast<uint4 *>(A_row + TH_IDX(907, t0, pitch - R + 1)) =
                            make_uint4(a16[0] | (a16[1] << 16), a16[2] | (a16[3] << 16), a16[4] | (a16[5] << 16),
                                       a16[6] | (a16[7] << 16));
                }
                int hg = -1;
                while (k < rounds && hg < 0) hg = my_half_group(k++);
                if (hg < 0) { remaining = 0; return; }
                tile = hg * 16 + lane16;
#pragma unroll
                for (int r = 0; r < R; ++r) acc[r] = 0xFFFFFFFFu;
                remaining = dead ? 0 : max(0, (tile | 15) - q_shift - q_lo + 1);
                store_current = true;
                if (remaining > 0) {
                    const uint32_t *f_hi = chunk_in(Fprev, tile) - q_lo * CS;   // at worst a pad chunk
#pragma unroll
                    for (int r = 0; r < R; ++r) wa[r] = f_hi[r];
                    f_lo = f_hi - CS;
                    g = Gk + q_lo * R;
                    return;
                }
            }
        };
        next_tile(false);
        // Segments with a warp-uniform trip count: up to the next moment at which a half-warp
        // finishes a tile (trip counts are even).
        for (;;) {
            const unsigned n_seg = __reduce_min_sync(0xFFFFFFFFu, remaining > 0 ? (unsigned)remaining : 0xFFFFFFFFu);
            if (n_seg == 0xFFFFFFFFu) break;
            if (remaining > 0) {
                for (unsigned q = 0; q < n_seg; q += 2) {
                    chunk_step<R>(wa, wb, acc, TH_PTR(908, f_lo, Fprev, f_words - R + 1), TH_PTR(909, g, Gk, Tp - R + 1));
                    chunk_step<R>(wb, wa, acc, TH_PTR(910, f_lo - CS, Fprev, f_words - R + 1),
                                  TH_PTR(911, g + R, Gk, Tp - R + 1));
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
        uint32_t *t = Fprev; Fprev = Fcur; Fcur = t;      // Fprev: the table just finished
    }

    if (failed) {
        mbar_wait(mbar, 0, 1u << 10);                     // let a late copy land (bounded) before leaving
        if (lane == 0) write_unsolved(THEMIS_STATUS_TIMEOUT);
        return;
    }

    // last prefix table to the workspace, and the final scan: cheapest total, lowest total
    // latency among equals
    uint32_t best = 0xFFFFFFFFu;
    int32_t *F_row = p.F + (size_t)n * pitch;
    for (int hg = slot; hg < NHG; hg += 2) {
        const int tile = hg * 16 + lane16;
        const uint32_t *chunk = chunk_in(Fprev, tile);
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int t = (tile - n_dummy) * R + r;
            const uint32_t fk = chunk[r];
            if (t >= 0 && t <= T) best = min(best, fk | (uint32_t)t);
            if (t >= 0 && t < pitch) F_row[TH_IDX(912, t, pitch)] = fk >= kInfKey ? THEMIS_G_INF : (int32_t)(fk >> kIdxBits);
        }
    }
    best = __reduce_min_sync(0xFFFFFFFFu, best);
    if (best >= kInfKey) {
        if (lane == 0) write_unsolved(THEMIS_STATUS_INFEASIBLE);
        return;
    }
    __syncwarp();                                         // the argmin rows written by other lanes
    const int tstar = (int)(best & kIdxMask);
    if (lane == 0) {                                      // walk the argmin tables back
        int t = tstar;
        for (int s = S - 1; s >= 1; --s) {
            const int ell = (int)p.A[TH_IDX(913, ((size_t)n * S + s) * pitch + t, (size_t)p.prob.n_instances * S * pitch)];
            ell_of[TH_IDX(914, s, S)] = (uint32_t)ell;
            t -= ell;
        }
        ell_of[0] = (uint32_t)t;
    }
    __syncwarp();
    // one lane per stage turns (s, l_s) into the stage's configuration
    for (int s = lane; s < S; s += 32) {
        const int ell = (int)ell_of[s];
        const int idx = (int)p.Garg[TH_IDX(915, ((size_t)n * S + s) * pitch + ell, (size_t)p.prob.n_instances * S * pitch)];
        const int C = p.prob.c_max, NB = p.prob.n_batch;
        const int bi = idx % NB, rest = idx / NB;
        b_o[s] = p.prob.batch_sizes[TH_IDX(916, bi, THEMIS_MAX_BATCH_SIZES)];
        c_o[s] = rest % C + 1;
        h_o[s] = p.vertical ? p.replicas[(size_t)n * S + s]
                   : p.horizontal ? G_inst[(size_t)s * pitch + ell] : rest / C + 1;
    }
    if (lane == 0) {
        p.out.total_cost[n] = (int32_t)(best >> kIdxBits);
        p.out.latency_buckets[n] = tstar;
        p.out.status[n] = THEMIS_STATUS_OK;
    }
}

}  // namespace

// Budgets the 32-bit warp kernel takes (cells).  Measured against the block kernel on 8192
// instances of 8 stages: 2.2 x as fast at 500 and 800 cells, 1.3 to 1.8 x between 1000 and 2200,
// 1.14 x at 2600, even at 3000, 6 % slower at 4000.
constexpr int kWarpKernel32MaxCells = 2800;

bool minplus_warp_fits(const Params &p, int tile)
{
    return tile != 16 && p.T + 1 <= kWarpKernel32MaxCells;   // tiles of 8 cells only
}

cudaError_t launch_minplus_warp(const Params &p_in, cudaStream_t stream)
{
    static std::atomic<uint64_t> ready{0};
    cudaError_t e = allow_max_smem(reinterpret_cast<const void *>(minplus_warp_kernel), ready);
    if (e != cudaSuccess) return e;
    Params p = p_in;
    p.n_half_groups = ((p.T + 1 + kR - 1) / kR + 15) / 16;
    const size_t warp_bytes = sizeof(uint32_t) * (size_t)warp_words32(p.n_half_groups * 16, p.pitch, p.prob.n_stages);
    int warps = 4;
    while (warps > 1 && warps * warp_bytes > kMaxDynamicSmem) warps >>= 1;
    const int N = p.prob.n_instances;
    minplus_warp_kernel<<<(N + warps - 1) / warps, warps * 32, warps * warp_bytes, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace themis

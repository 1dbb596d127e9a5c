// Internal declarations shared by the translation units of libthemis.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "themis.h"

namespace themis {

// Cost field of a packed key: 17 bits.  Valid totals are <= THEMIS_MAX_TOTAL_COST
// = kInfCost - 1, so the sum of two fields (<= 2^18 - 2) plus a 14-bit index still
// fits an unsigned 32-bit word and "unreachable" never needs a branch.
constexpr uint32_t kIdxBits = 14;
constexpr uint32_t kIdxMask = (1u << kIdxBits) - 1u;
constexpr uint32_t kInfCost = (1u << 17) - 1u;
constexpr uint32_t kInfKey = kInfCost << kIdxBits;

// inst_flag values: 0 clean, 1 bad input seen while scoring, 2 set by the packed
// 16-bit min-plus kernel when a total reached its saturation value and the
// instance has to be redone by the 32-bit kernel.
constexpr int32_t kFlagBadInput = 1;
constexpr int32_t kFlagNeedsWide = 2;
// 3: set by the sparse warp kernels for an instance whose lists outgrew their capacities; it
// is on the redo list and the block kernel solves it.
constexpr int32_t kFlagRedo = 3;

// Packed 16-bit path: costs are exact below kInf16 and saturate there; two of
// them add without carrying into the neighbouring half-word.
constexpr uint32_t kInf16 = 0x7FFFu;

// Rows of the workspace tables are padded to a multiple of this many entries,
// so every row starts 64-byte aligned (uint16) / 128-byte aligned (int32) and
// bulk copies of whole rows meet the 16-byte rule.
constexpr int kRowAlign = 32;

// Candidate list of one (profile, stage), built by score_lists_kernel and read by score_kernel,
// in 32-bit words:
//   [0] entries  [1] entries of batch size 1 (they come first)  [2] 1 if a latency is not positive
//   [3] joint tasks
//   [4 ..)       uint4 per joint task {batch index | first joint entry << 4 | entries << 24,
//                smallest latency of that batch size in buckets, the same in us, 0}
//   [single ..)  uint4 per entry {latency [us], latency in buckets, cores, batch index}, sorted by
//                batch index, then cores
//   [joint ..)   uint2 per entry {latency [us], latency in buckets << 2 | cores << 17}, the same
//                order, every batch size padded with entries that never fit to a multiple of the
//                entries one pass of the scoring loop takes (at most 32)
struct ScoreListLayout { int tasks, single, joint, words; };
__host__ __device__ inline ScoreListLayout score_list_layout(int c_max, int n_batch)
{
    ScoreListLayout L;
    const int CB = c_max * n_batch;
    L.tasks = 4;
    L.single = L.tasks + 4 * n_batch * (c_max / 32 + 2);
    L.joint = L.single + 4 * CB;
    L.words = (L.joint + 2 * (CB + 32 * n_batch) + 3) & ~3;   // every list starts 16-byte aligned
    return L;
}

struct Params {
    themis_problem_t prob;
    int32_t T;          // budget in buckets
    int32_t pitch;      // row pitch of G / Garg / A / F in entries
    int32_t vertical;   // 1: h fixed per stage from replicas[]
    int32_t horizontal; // 1: Algorithm 2, one candidate per batch size with the fewest replicas
                        //    that sustain lambda; candidate index = batch index, stage cost = h
    int32_t only_flagged;  // wide min-plus kernel: solve only instances flagged kFlagNeedsWide
    int32_t n_half_groups;   // packed min-plus kernel: half-groups of 16 tiles
    const int32_t *lat_us;
    const int32_t *profile_id;
    const uint32_t *lambda_mrps;
    const int32_t *replicas;
    const int32_t *active;   // [N] or NULL: blocks of instances with active[n] == 0 leave at once
    int32_t *G;
    uint16_t *Garg;
    uint16_t *A;
    int32_t *F;
    uint32_t *lists;     // scoring: candidate lists per (profile, stage), score_list_layout().words words each
    int32_t *check;      // bounds-checked build: {site of the first violation (0 = none), index, limit, 0}
    int32_t *redo_count; // sparse warp kernel: number of instances handed to the block kernel ...
    int32_t *redo_list;  // ... and their indices [N]
    int32_t *inst_flag;  // [N] kFlagBadInput: bad input seen by the scoring kernel; kFlagNeedsWide: see above
    themis_result_t out;
};

constexpr size_t kMaxDynamicSmem = 226u * 1024u;   // 227 KB per block less room for static variables

// Raises a kernel's dynamic shared-memory limit to kMaxDynamicSmem, once per device and
// kernel (`done` has one bit per device ordinal and belongs to the launch site), so that a
// launch costs no attribute call.
inline cudaError_t allow_max_smem(const void *kernel, std::atomic<uint64_t> &done)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const uint64_t bit = 1ull << (dev & 63);
    if (done.load(std::memory_order_acquire) & bit) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxDynamicSmem);
    if (e == cudaSuccess) done.fetch_or(bit, std::memory_order_release);
    return e;
}

// Bounds-checked build (-DTHEMIS_CHECK_BOUNDS; stands in for a memory sanitizer).  Every index
// into shared or global memory that a kernel computes goes through TH_IDX(site, index, limit):
// an index outside [0, limit) is recorded once in Params::check (site number, index, limit)
// and clamped into range, so the access itself stays legal, the kernel runs to its end and the
// host reads the record (themis_bounds_check_report).  Nothing traps.  Site numbers: 1xx
// scoring, 2xx packed recurrence, 3xx 32-bit recurrence, 4xx pruned recurrence, 5xx sparse
// block kernel, 6xx stage fronts, 7xx prefix fronts.  In the normal build TH_IDX is its index.
#ifdef THEMIS_CHECK_BOUNDS
#ifdef __CUDACC__
__device__ __forceinline__ int th_checked_index(int site, long long i, long long n, int32_t *check)
{
    if (i >= 0 && i < n) return (int)i;
    if (atomicCAS(&check[0], 0, site) == 0) {
        check[1] = (int)i;
        check[2] = (int)n;
    }
    return i < 0 || n < 1 ? 0 : (int)(n - 1);
}
#endif
#define TH_IDX(site, i, n) th_checked_index((site), (long long)(i), (long long)(n), p.check)
// a pointer that must stay within [base, base + n)
#define TH_PTR(site, ptr, base, n) ((base) + TH_IDX(site, (ptr) - (base), n))
constexpr int kBoundsChecked = 1;
#else
#define TH_IDX(site, i, n) (i)
#define TH_PTR(site, ptr, base, n) (ptr)
constexpr int kBoundsChecked = 0;
#endif

cudaError_t launch_score(const Params &p, cudaStream_t stream);
cudaError_t launch_minplus(const Params &p, int tile, cudaStream_t stream);
// The 32-bit kernel with one warp per instance, for short budgets (tiles of 8 cells); launch_minplus uses it.
bool minplus_warp_fits(const Params &p, int tile);
cudaError_t launch_minplus_warp(const Params &p, cudaStream_t stream);
cudaError_t launch_minplus16(const Params &p, int tile, cudaStream_t stream);
// The packed kernel with one warp per instance, for short budgets (tiles of 4 or 8 cells).
bool minplus16_warp_fits(const Params &p, int tile);
cudaError_t launch_minplus16_warp(const Params &p, int tile, cudaStream_t stream);
cudaError_t launch_minplus_pruned(const Params &p, cudaStream_t stream);
// Scoring and recurrence on undominated entries in one kernel (needs lat_us, lambda, out set),
// one block per instance; only_listed: a fixed grid works through redo_list instead.
size_t sparse_smem_bytes(const Params &p);
cudaError_t launch_solve_sparse(const Params &p, bool only_listed, cudaStream_t stream);
// The same on short sorted lists, one warp per instance; instances that outgrow the lists are
// appended to redo_list (redo_count must be zero before the launch).
bool front_kernel_fits(const Params &p);
cudaError_t launch_solve_front(const Params &p, cudaStream_t stream);
// Dynamic shared memory of the pruned kernel for a row pitch; it cannot run above 227 KB.
inline size_t pruned_smem_bytes(int pitch) { return sizeof(uint32_t) * (5u * (size_t)pitch + 4 + 32); }
cudaError_t launch_configs_equal(int N, int S, themis_result_t a, themis_result_t b, int32_t *stable, cudaStream_t st);
cudaError_t launch_fb_init(int N, uint32_t res, const int32_t *status, const uint32_t *lambda, uint32_t *lo,
                           uint32_t *hi, int32_t *active, cudaStream_t st);
cudaError_t launch_fb_bisect(const Params &p, int rounds, uint32_t res, const int32_t *active, uint32_t *lo,
                             uint32_t *hi, cudaStream_t st);
cudaError_t launch_fb_final_trial(int N, uint32_t res, const uint32_t *lo, const int32_t *active,
                                  int32_t *iter_active, uint32_t *trial_lambda, cudaStream_t st);
cudaError_t launch_fb_finish(const Params &p, uint32_t res, const uint32_t *lo, const uint32_t *hi,
                             const int32_t *active, uint32_t *lambda_vertical, int32_t *extra, cudaStream_t st);
cudaError_t launch_fit_profiles(int n_models, int n_samples, const int32_t *sample_b, const int32_t *sample_c,
                                const double *latency_ms, int c_max, int n_batch, const int32_t *d_batch_sizes,
                                double *coeffs, int32_t *lat_us, int32_t *status, cudaStream_t st);
cudaError_t launch_alu_probe(int mode, int blocks, int threads, int iters, uint32_t *sink,
                             cudaStream_t stream);
cudaError_t launch_wait_probe(uint32_t max_polls, const uint32_t *src16, uint32_t *dst16, int32_t *status,
                              cudaStream_t stream);

}  // namespace themis

// Candidate scoring: reduces every stage's candidate configurations to the
// per-bucket minimum-cost vector G_s and its argmin Garg_s (the inner loops of
// Algorithm 1, with the queuing delay of Eq. 4 and the throughput constraint of
// Eq. 6), one thread block per instance.
//
// Everything that needs 64-bit arithmetic is hoisted out of the candidate loop
// into two small shared-memory tables indexed by (batch size, replicas):
//   Q[bi][h]    = ceil((b-1) * m * 1e9 / (lambda_m * w_us)),  m = h or 1   (Eq. 4 in buckets)
//   Lmax[bi][h] = floor(h * b * 1e9 / lambda_m)     largest latency [us] that still
//                 satisfies  h * b / l >= lambda                           (Eq. 6)
// (joint problem: one table for all stages; vertical variant: one row pair per
// stage, for that stage's fixed replica count), all filled before the first stage.
// A candidate is then two compares, a multiply-add and a shared-memory atomic
// min on the packed word (cost << 16 | candidate index), whose ordering gives
// "cheapest, then lowest index" directly.
//
// What depends on the latency table alone is done once per (profile, stage) by a
// small kernel in front (score_lists_kernel): the (cores, batch size) pairs whose
// latency differs from the one with a core fewer and fits the budget, with the
// latency rounded up to buckets, as lists sorted by batch size and cores, cut into
// warp tasks.  Every instance of the profile reads the lists instead of the table.
//  - Where the queuing delay grows with the replica count (joint problem, flag
//    THEMIS_QUEUE_PER_REPLICA, b > 1), a task is up to 32 entries of one batch
//    size; the lanes take one replica count each, every entry is read by all of
//    them (one 16-byte load brings two) and each lane scores its (h, c, b);
//  - elsewhere more replicas only cost more in the same bucket, so a task is 32
//    entries, one per lane, and each lane looks up the fewest replicas that
//    sustain lambda for its entry (binary search in the Lmax row) and scores
//    that one candidate.
// Two key rows alternate between stages, so a stage costs one block barrier.
#include "themis_internal.h"

namespace themis {
namespace {

constexpr uint32_t kEmptyKey = 0xFFFFFFFFu;
constexpr int kListWords = 64;        // per warp: 32 entries of two words
constexpr uint32_t kNeverFits = 0xFFFFFFFFu;   // latency of a padding entry: above every Lmax

// atomic min on a shared-memory word given by its 32-bit shared-space address
__device__ __forceinline__ void red_min_shared(uint32_t addr, uint32_t v)
{
    asm volatile("red.shared.min.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// Two list entries {latency [us], 4 * l_b | c << 17} at `entries` (shared memory, 16-byte
// aligned) against this lane's replica count: q4 = 4 * Q[b][h], lmax = Lmax[b][h],
// key = c * key_mul + key_add.  A lane whose candidate is infeasible or over budget sends
// its word to `idle` (a word nobody reads), so the reduction itself is unconditional and
// the loop body has no branch.
__device__ __forceinline__ void score_two_entries(uint32_t entries, uint32_t q4, uint32_t lmax, uint32_t t4,
                                                  uint32_t key_mul, uint32_t key_add, uint32_t keys,
                                                  uint32_t idle)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        ".reg .b32 e0, e1, e2, e3, x, y, l0, l1, c0, c1, k0, k1;\n\t"
        "ld.shared.v4.u32 {e0, e1, e2, e3}, [%0];\n\t"
        "add.u32 x, e1, %1;\n\t"
        "add.u32 y, e3, %1;\n\t"
        "and.b32 l0, x, 0x1FFFC;\n\t"
        "and.b32 l1, y, 0x1FFFC;\n\t"
        "setp.le.u32 p, e0, %2;\n\t"
        "setp.le.u32 q, e2, %2;\n\t"
        "setp.le.and.u32 p, l0, %3, p;\n\t"
        "setp.le.and.u32 q, l1, %3, q;\n\t"
        "shr.u32 c0, x, 17;\n\t"
        "shr.u32 c1, y, 17;\n\t"
        "mad.lo.u32 k0, c0, %4, %5;\n\t"
        "mad.lo.u32 k1, c1, %4, %5;\n\t"
        "add.u32 l0, l0, %6;\n\t"
        "add.u32 l1, l1, %6;\n\t"
        "selp.u32 l0, l0, %7, p;\n\t"
        "selp.u32 l1, l1, %7, q;\n\t"
        "red.shared.min.u32 [l0], k0;\n\t"
        "red.shared.min.u32 [l1], k1;\n\t"
        "}" ::"r"(entries), "r"(q4), "r"(lmax), "r"(t4), "r"(key_mul), "r"(key_add), "r"(keys), "r"(idle)
        : "memory");
}

// Four list entries in one go: the two at `entries` and the two at `entries + stride`, both
// loads issued before any arithmetic so that their latencies overlap.
__device__ __forceinline__ void score_four_entries(uint32_t entries, uint32_t stride, uint32_t q4, uint32_t lmax,
                                                   uint32_t t4, uint32_t key_mul, uint32_t key_add, uint32_t keys,
                                                   uint32_t idle)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p, q, u, v;\n\t"
        ".reg .b32 e0, e1, e2, e3, f0, f1, f2, f3, x, y, z, w, l0, l1, l2, l3, c0, c1, c2, c3, k0, k1, k2, k3, a2;\n\t"
        "add.u32 a2, %0, %8;\n\t"
        "ld.shared.v4.u32 {e0, e1, e2, e3}, [%0];\n\t"
        "ld.shared.v4.u32 {f0, f1, f2, f3}, [a2];\n\t"
        "add.u32 x, e1, %1;\n\t"
        "add.u32 y, e3, %1;\n\t"
        "add.u32 z, f1, %1;\n\t"
        "add.u32 w, f3, %1;\n\t"
        "and.b32 l0, x, 0x1FFFC;\n\t"
        "and.b32 l1, y, 0x1FFFC;\n\t"
        "and.b32 l2, z, 0x1FFFC;\n\t"
        "and.b32 l3, w, 0x1FFFC;\n\t"
        "setp.le.u32 p, e0, %2;\n\t"
        "setp.le.u32 q, e2, %2;\n\t"
        "setp.le.u32 u, f0, %2;\n\t"
        "setp.le.u32 v, f2, %2;\n\t"
        "setp.le.and.u32 p, l0, %3, p;\n\t"
        "setp.le.and.u32 q, l1, %3, q;\n\t"
        "setp.le.and.u32 u, l2, %3, u;\n\t"
        "setp.le.and.u32 v, l3, %3, v;\n\t"
        "shr.u32 c0, x, 17;\n\t"
        "shr.u32 c1, y, 17;\n\t"
        "shr.u32 c2, z, 17;\n\t"
        "shr.u32 c3, w, 17;\n\t"
        "mad.lo.u32 k0, c0, %4, %5;\n\t"
        "mad.lo.u32 k1, c1, %4, %5;\n\t"
        "mad.lo.u32 k2, c2, %4, %5;\n\t"
        "mad.lo.u32 k3, c3, %4, %5;\n\t"
        "add.u32 l0, l0, %6;\n\t"
        "add.u32 l1, l1, %6;\n\t"
        "add.u32 l2, l2, %6;\n\t"
        "add.u32 l3, l3, %6;\n\t"
        "selp.u32 l0, l0, %7, p;\n\t"
        "selp.u32 l1, l1, %7, q;\n\t"
        "selp.u32 l2, l2, %7, u;\n\t"
        "selp.u32 l3, l3, %7, v;\n\t"
        "red.shared.min.u32 [l0], k0;\n\t"
        "red.shared.min.u32 [l1], k1;\n\t"
        "red.shared.min.u32 [l2], k2;\n\t"
        "red.shared.min.u32 [l3], k3;\n\t"
        "}" ::"r"(entries), "r"(q4), "r"(lmax), "r"(t4), "r"(key_mul), "r"(key_add), "r"(keys), "r"(idle), "r"(stride)
        : "memory");
}

#ifdef THEMIS_CHECK_BOUNDS
// The same step with every address formed in C++ and range-checked (bounds-checked build).
__device__ __forceinline__ void score_two_entries_checked(const Params &p, uint32_t *smem, int smem_words,
                                                          int entries_word, uint32_t q4, uint32_t lmax, uint32_t t4,
                                                          uint32_t key_mul, uint32_t key_add, int keys_word,
                                                          int idle_word)
{
    for (int j = 0; j < 2; ++j) {
        const uint32_t e0 = smem[TH_IDX(140, entries_word + 2 * j, smem_words)];
        const uint32_t x = smem[TH_IDX(141, entries_word + 2 * j + 1, smem_words)] + q4;
        const uint32_t l = x & 0x1FFFCu;
        const bool ok = e0 <= lmax && l <= t4;
        const uint32_t key = (x >> 17) * key_mul + key_add;
        const int word = ok ? keys_word + (int)(l >> 2) : idle_word;
        atomicMin(&smem[TH_IDX(142, word, smem_words)], key);
    }
}
#endif

__device__ __forceinline__ uint32_t sat_u32(unsigned long long v, uint32_t cap)
{
    return v > (unsigned long long)cap ? cap : (uint32_t)v;
}

// In the joint loop the lanes of a warp cover 2^hn_log replica counts x (32 >> hn_log) entry
// pairs at a time.
__host__ __device__ inline int joint_hn_log(int HN)
{
    int hn_log = 1;
    while ((1 << hn_log) < HN && hn_log < 5) ++hn_log;
    return hn_log;
}

// Builds the candidate lists of one (profile, stage) (layout: score_list_layout).  One block
// per (profile, stage), one warp per batch size.
__global__ void __launch_bounds__(32 * THEMIS_MAX_BATCH_SIZES)
score_lists_kernel(const Params p, int joint_lists)
{
    const int C = p.prob.c_max, NB = p.prob.n_batch, CB = C * NB;
    const int lane = threadIdx.x & 31, bi = threadIdx.x >> 5;
    const uint32_t w_us = (uint32_t)p.prob.bucket_us;
    const int32_t *lat_s = p.lat_us + (size_t)blockIdx.x * CB;
    const ScoreListLayout L = score_list_layout(C, NB);
    uint32_t *hdr = p.lists + (size_t)blockIdx.x * L.words;
    uint4 *single = reinterpret_cast<uint4 *>(hdr + L.single);
    uint2 *joint = reinterpret_cast<uint2 *>(hdr + L.joint);
    const int joint_cap = CB + 32 * NB;
    (void)joint_cap;
    // entries one pass of the joint loop takes: 2 per group of lanes
    const int M = joint_lists ? 64 >> joint_hn_log(p.prob.h_max) : 1;
    __shared__ int count[THEMIS_MAX_BATCH_SIZES], padded[THEMIS_MAX_BATCH_SIZES], n_task[THEMIS_MAX_BATCH_SIZES];
    __shared__ int bad;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    const uint32_t lanemask_lt = (1u << lane) - 1u;
    int off_single = 0, off_joint = 0, off_task = 0;
    for (int pass = 0; pass < 2; ++pass) {
        int n = 0, saw_bad = 0;
        uint32_t min_lb = 0xFFFFFFFFu, min_lus = 0xFFFFFFFFu;
        for (int c0 = 0; c0 < C; c0 += 32) {
            const int cidx = c0 + lane;               // core count - 1
            int32_t v = 1, v_prev = 0;
            if (cidx < C) {
                v = lat_s[TH_IDX(151, cidx * NB + bi, CB)];
                v_prev = cidx > 0 ? lat_s[TH_IDX(152, (cidx - 1) * NB + bi, CB)] : 0;
            }
            if (v <= 0) saw_bad = 1;
            // Same latency with one core fewer: that candidate reaches the same buckets with the
            // same replica counts at a lower cost, so this one is never a minimum (latency
            // tables are flat over long runs of core counts).
            const uint32_t l_b = v > 0 ? ((uint32_t)v + w_us - 1u) / w_us : 0u;
            const bool keep = cidx < C && v > 0 && v != v_prev && l_b <= (uint32_t)p.T;
            const unsigned kept = __ballot_sync(0xFFFFFFFFu, keep);
            if (keep) {
                min_lb = min(min_lb, l_b);
                min_lus = min(min_lus, (uint32_t)v);
                if (pass == 1) {
                    const int at = n + __popc(kept & lanemask_lt);
                    single[TH_IDX(153, off_single + at, CB)] = make_uint4((uint32_t)v, l_b, (uint32_t)(cidx + 1), (uint32_t)bi);
                    if (joint_lists)
                        joint[TH_IDX(154, off_joint + at, joint_cap)] = make_uint2((uint32_t)v, (l_b << 2) | ((uint32_t)(cidx + 1) << 17));
                }
            }
            n += __popc(kept);
        }
        if (pass == 0) {
            if (lane == 0) {
                count[bi] = n;
                padded[bi] = joint_lists ? (n + M - 1) / M * M : 0;
                // batch size 1 has no queue: its entries go the one-candidate way
                n_task[bi] = joint_lists && p.prob.batch_sizes[bi] != 1 ? (padded[bi] + 31) / 32 : 0;
            }
            if (saw_bad) bad = 1;
            __syncthreads();
            for (int j = 0; j < bi; ++j) { off_single += count[j]; off_joint += padded[j]; off_task += n_task[j]; }
        } else {
            min_lb = __reduce_min_sync(0xFFFFFFFFu, min_lb);
            min_lus = __reduce_min_sync(0xFFFFFFFFu, min_lus);
            // entries that never fit behind the last one, up to the padded count
            if (lane < padded[bi] - n)
                joint[TH_IDX(155, off_joint + n + lane, joint_cap)] = make_uint2(kNeverFits, 0u);
            // this batch size's tasks: equal shares, whole passes of the loop
            const int nt = n_task[bi];
            if (lane < nt) {
                const int share = ((padded[bi] + nt - 1) / nt + M - 1) / M * M;
                const int first = lane * share;
                const int len = max(0, min(share, padded[bi] - first));
                reinterpret_cast<uint4 *>(hdr + L.tasks)[TH_IDX(156, off_task + lane, (L.single - L.tasks) / 4)] =
                    make_uint4((uint32_t)bi | ((uint32_t)(off_joint + first) << 4) | ((uint32_t)len << 24), min_lb, min_lus, 0u);
            }
        }
    }
    if (threadIdx.x == 0) {
        int total = 0, tasks = 0;
        for (int j = 0; j < NB; ++j) { total += count[j]; tasks += n_task[j]; }
        hdr[0] = (uint32_t)total;
        hdr[1] = p.prob.batch_sizes[0] == 1 ? (uint32_t)count[0] : 0u;
        hdr[2] = (uint32_t)bad;
        hdr[3] = (uint32_t)tasks;
    }
}

// THREADS: 256, or 128 for short budgets, where a stage is so little work that the per-warp
// cost of a stage (loop, barrier, row addresses) shows; registers for 1536 threads per SM.
template <int THREADS>
__global__ void __launch_bounds__(THREADS, 1280 / THREADS)
score_kernel(const Params p)
{
    constexpr int kScoreThreads = THREADS, kScoreWarps = THREADS / 32;
    extern __shared__ __align__(16) uint32_t smem[];
    const int n = blockIdx.x;
    if (p.active && !p.active[n]) return;
    const int tid = threadIdx.x;
    const int T = p.T, pitch = p.pitch;
    const int S = p.prob.n_stages, C = p.prob.c_max, NB = p.prob.n_batch;
    const int CB = C * NB;
    const int HN = p.vertical ? 1 : p.prob.h_max;   // replica values per table row
    const int SV = p.vertical ? S : 1;              // table sets: one per stage when h is per stage
    const uint32_t w_us = (uint32_t)p.prob.bucket_us;
    const int lane = tid & 31, warp = tid >> 5;

    // Shared memory, in words (every access is an offset from this one array):
    // key row 0 [pitch] | key row 1 [pitch] | Q [SV][NB][HN] | Lmax [SV][NB][HN] | pad to 4 |
    // one list per warp [kListWords] | one idle word per lane [32]
    const int q_off = 2 * pitch;
    const int lmax_off = q_off + SV * NB * HN;
    const int list_base = (lmax_off + SV * NB * HN + 3) & ~3;
    const int list_off = list_base + warp * kListWords;
    const int idle_off = list_base + kScoreWarps * kListWords;
    const int smem_words = idle_off + 32;           // what the launch provides
    (void)smem_words;
    const uint32_t smem_addr = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t idle_addr = smem_addr + 4u * (uint32_t)(idle_off + lane);
    __shared__ int s_bad;

    const uint32_t lambda_m = p.lambda_mrps[TH_IDX(101, n, p.prob.n_instances)];
    const int pid = p.profile_id ? p.profile_id[TH_IDX(102, n, p.prob.n_instances)] : 0;
    const int32_t *rep = p.vertical ? p.replicas + (size_t)n * S : nullptr;

    if (tid == 0) {
        int bad = (lambda_m == 0) || pid < 0 || pid >= p.prob.n_profiles;
        if (rep) {
            long long total = 0;
            for (int s = 0; s < S; ++s) {
                if (rep[s] < 1 || (long long)rep[s] * C > 65535) bad = 1;   // cost field is 16 bits
                total += (long long)rep[s] * C;
            }
            if (total > THEMIS_MAX_TOTAL_COST) bad = 1;
        }
        s_bad = bad;
    }
    for (int l4 = tid * 4; l4 < 2 * pitch; l4 += kScoreThreads * 4)
        *reinterpret_cast<uint4 *>(smem + TH_IDX(124, l4, 2 * pitch - 3)) = make_uint4(kEmptyKey, kEmptyKey, kEmptyKey, kEmptyKey);
    __syncthreads();
    const bool skip_all = s_bad != 0;

    if (!skip_all) {
        const unsigned long long q_den = (unsigned long long)lambda_m * w_us;
        for (int e = tid; e < SV * NB * HN; e += kScoreThreads) {
            const int sv = e / (NB * HN);
            const int bi = (e - sv * NB * HN) / HN;
            const int k = e - (sv * NB + bi) * HN;
            const unsigned long long h = (unsigned long long)((p.vertical ? rep[TH_IDX(105, sv, S)] : 1) + k);
            const unsigned long long b = (unsigned long long)p.prob.batch_sizes[TH_IDX(106, bi, NB)];
            const unsigned long long m = (p.prob.flags & THEMIS_QUEUE_PER_REPLICA) ? h : 1ull;
            const unsigned long long q_num = (b - 1ull) * m * 1000000000ull;
            smem[TH_IDX(103, q_off + e, lmax_off)] = sat_u32((q_num + q_den - 1ull) / q_den, (uint32_t)T + 1u);
            smem[TH_IDX(104, lmax_off + e, list_base)] = sat_u32(h * b * 1000000000ull / lambda_m, 0x7FFFFFFFu);
        }
    }
    __syncthreads();                            // tables ready, both key rows empty

    const bool q_grows_with_h = (p.prob.flags & THEMIS_QUEUE_PER_REPLICA) != 0;
    // one candidate per (c, b): q does not depend on h, or only one h is a candidate
    const bool single = !q_grows_with_h || p.horizontal || p.vertical || HN == 1;
    int saw_bad_latency = 0;
    // In the joint loop the lanes of a warp cover HNp replica counts x (32 / HNp) pairs of entries.
    const int hn_log = joint_hn_log(HN);
    const int HNp = 1 << hn_log;
    const int groups = 32 >> hn_log;
    const int group = lane >> hn_log, hk = lane & (HNp - 1);
    const ScoreListLayout LL = score_list_layout(C, NB);
    const uint32_t list_addr = smem_addr + 4u * (uint32_t)list_off + 16u * (uint32_t)group;

    for (int s = 0; s < S; ++s) {
        const int key_off = (s & 1) * pitch;
        const uint32_t key_addr = smem_addr + 4u * (uint32_t)key_off;
        if (!skip_all) {
            const int h_lo = p.vertical ? rep[s] : 1;
            const int row_s = p.vertical ? s * NB : 0;
            const uint32_t *hdr = p.lists + ((size_t)pid * S + s) * LL.words;
            const int n_entries = (int)hdr[0];
            // entries with one candidate each: all of them, or those of batch size 1 (no queue)
            const int n_single = single ? n_entries : (int)hdr[1];
            saw_bad_latency |= (int)hdr[2];
            const int nt_joint = single ? 0 : (int)hdr[3];
            const int nt_single = (n_single + 31) >> 5;
            const uint4 *entries = reinterpret_cast<const uint4 *>(hdr + LL.single);
            const uint2 *joint = reinterpret_cast<const uint2 *>(hdr + LL.joint);
            const uint4 *task_recs = reinterpret_cast<const uint4 *>(hdr + LL.tasks);
            uint4 recs = make_uint4(0u, 0u, 0u, 0u);         // joint tasks: this warp's next 32 task records, one per lane
            uint2 ahead = make_uint2(kNeverFits, 0u);        // this lane's entry of the task about to start
            for (int t = warp; t < nt_joint + nt_single; t += kScoreWarps) {
                if (t >= nt_joint) {
                    // More replicas only cost more in the same bucket: the fewest replicas that
                    // sustain lambda (feasibility is monotone in h) are the entry's one candidate.
                    const int e = 32 * (t - nt_joint) + lane;
                    if (e < n_single) {
                        const uint4 en = entries[TH_IDX(107, e, CB)];
                        const uint32_t l_us = en.x, l_b = en.y;
                        const int cidx = (int)en.z - 1, bi = (int)en.w;
                        const int q_row = q_off + (row_s + bi) * HN;
                        const int lmax_row = lmax_off + (row_s + bi) * HN;
                        int lo = 0, cnt = HN;
                        if (HN == 1) {                       // vertical variant: the one replica count
                            lo = smem[TH_IDX(109, lmax_row, list_base)] < l_us ? 1 : 0;
                            cnt = 0;
                        }
                        while (cnt > 0) {
                            const int half = cnt >> 1;
                            if (smem[TH_IDX(110, lmax_row + lo + half, list_base)] < l_us) { lo += half + 1; cnt -= half + 1; }
                            else cnt = half;
                        }
                        if (lo < HN) {
                            const uint32_t ell = l_b + smem[TH_IDX(111, q_row + lo, lmax_off)];
                            if (ell <= (uint32_t)T) {
                                const uint32_t cost = (uint32_t)(h_lo + lo) * (uint32_t)(cidx + 1);
                                const uint32_t idx = (uint32_t)((p.horizontal ? 0 : lo * CB) + cidx * NB + bi);
#ifdef THEMIS_CHECK_BOUNDS
                                atomicMin(&smem[TH_IDX(112, key_off + (int)ell, key_off + pitch)], (cost << 16) | idx);
#else
                                red_min_shared(key_addr + 4u * ell, (cost << 16) | idx);
#endif
                            }
                        }
                    }
                    continue;
                }
                // Joint problem with h_max >= 2 (so c <= 32767: at most 65535 candidates per stage):
                // one batch size, lanes over replica counts.  The task's entries come to the
                // warp's list in shared memory, the next task's are on their way meanwhile.
                const int j = (t - warp) / kScoreWarps;      // this warp's j-th task of the stage
                if ((j & 31) == 0) {                         // lane i: the record of task j + i
                    const int tj = t + lane * kScoreWarps;
                    recs = tj < nt_joint ? task_recs[TH_IDX(113, tj, (LL.single - LL.tasks) / 4)] : make_uint4(0u, 0u, 0u, 0u);
                    const uint32_t task0 = __shfl_sync(0xFFFFFFFFu, recs.x, 0);
                    const int first0 = (int)((task0 >> 4) & 0xFFFFFu), len0 = (int)(task0 >> 24);
                    ahead = lane < len0 ? joint[TH_IDX(116, first0 + lane, CB + 32 * NB)] : make_uint2(kNeverFits, 0u);
                }
                const uint32_t task = __shfl_sync(0xFFFFFFFFu, recs.x, j & 31);
                const uint32_t min_lb = __shfl_sync(0xFFFFFFFFu, recs.y, j & 31);
                const uint32_t min_lus = __shfl_sync(0xFFFFFFFFu, recs.z, j & 31);
                const int bi = (int)(task & 15u), len = (int)(task >> 24);
                *reinterpret_cast<uint2 *>(smem + TH_IDX(119, list_off + 2 * lane, smem_words - 1)) = ahead;
                if (((j + 1) & 31) != 0 && t + kScoreWarps < nt_joint) {
                    const uint32_t task1 = __shfl_sync(0xFFFFFFFFu, recs.x, (j + 1) & 31);
                    const int first1 = (int)((task1 >> 4) & 0xFFFFFu), len1 = (int)(task1 >> 24);
                    ahead = lane < len1 ? joint[TH_IDX(120, first1 + lane, CB + 32 * NB)] : make_uint2(kNeverFits, 0u);
                }
                __syncwarp();
                const int q_row = q_off + (row_s + bi) * HN;
                const int lmax_row = lmax_off + (row_s + bi) * HN;
                for (int h0 = 0; h0 < HN; h0 += HNp) {
                    // no entry fits the budget at this chunk's first replica count: q never shrinks with h
                    if (min_lb + smem[TH_IDX(114, q_row + h0, lmax_off)] > (uint32_t)T) break;
                    // no entry sustains lambda at its last
                    if (min_lus > smem[TH_IDX(115, lmax_row + min(h0 + HNp, HN) - 1, list_base)]) continue;
                    const int k = h0 + hk;                       // this lane's replica count - 1
                    const bool kv = k < HN;
                    const uint32_t q4 = 4u * (kv ? smem[TH_IDX(117, q_row + k, lmax_off)] : (uint32_t)T + 1u);
                    const uint32_t lmax = kv ? smem[TH_IDX(118, lmax_row + k, list_base)] : 0u;
                    // key = (h * c) << 16 | (h - 1) * CB + (c - 1) * NB + bi  =  c * key_mul + key_add
                    const uint32_t key_mul = ((uint32_t)(k + 1) << 16) + (uint32_t)NB;
                    const uint32_t key_add = (uint32_t)(k * CB - NB + bi);
#ifdef THEMIS_CHECK_BOUNDS
                    for (int i = 0; i < len; i += 2 * groups)
                        score_two_entries_checked(p, smem, smem_words, list_off + 4 * group + 2 * i, q4, lmax,
                                                  4u * (uint32_t)T, key_mul, key_add, key_off, idle_off + lane);
#else
                    uint32_t entries_addr = list_addr;
                    if (groups <= 8) {
                        // four entries a pass: a pass never leaves the warp's 32-entry list (len <= 32, the
                        // list's tail holds entries that never fit)
                        for (int i = 0; i < len; i += 4 * groups, entries_addr += 32u * (uint32_t)groups)
                            score_four_entries(entries_addr, 16u * (uint32_t)groups, q4, lmax, 4u * (uint32_t)T, key_mul,
                                               key_add, key_addr, idle_addr);
                    } else {
                        for (int i = 0; i < len; i += 2 * groups, entries_addr += 16u * (uint32_t)groups)
                            score_two_entries(entries_addr, q4, lmax, 4u * (uint32_t)T, key_mul, key_add, key_addr, idle_addr);
                    }
#endif
                }
                __syncwarp();                                // the list is free for the next task
            }
        }
        __syncthreads();
        // Unpack to G (int32) and Garg (uint16), four buckets per thread, and leave the
        // key row empty for the stage after next (the next stage uses the other row).
        int32_t *G_row = p.G + ((size_t)n * S + s) * pitch;
        uint16_t *Garg_row = p.Garg + ((size_t)n * S + s) * pitch;
        for (int l4 = tid * 4; l4 < pitch; l4 += kScoreThreads * 4) {
            const uint4 k4 = *reinterpret_cast<const uint4 *>(smem + TH_IDX(119, key_off + l4, key_off + pitch - 3));
            *reinterpret_cast<uint4 *>(smem + TH_IDX(120, key_off + l4, key_off + pitch - 3)) =
                make_uint4(kEmptyKey, kEmptyKey, kEmptyKey, kEmptyKey);
            const uint32_t kk[4] = {k4.x, k4.y, k4.z, k4.w};
            int4 g;
            int32_t *gv = reinterpret_cast<int32_t *>(&g);
            uint32_t a[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const bool empty = kk[i] == kEmptyKey;
                gv[i] = empty ? THEMIS_G_INF : (int32_t)(kk[i] >> 16);
                a[i] = empty ? 0u : kk[i];
            }
            *reinterpret_cast<int4 *>(G_row + TH_IDX(121, l4, pitch - 3)) = g;
            *reinterpret_cast<uint2 *>(Garg_row + TH_IDX(122, l4, pitch - 3)) =
                make_uint2(__byte_perm(a[0], a[1], 0x5410), __byte_perm(a[2], a[3], 0x5410));
        }
    }
    const int any_bad = __syncthreads_or(saw_bad_latency);
    if (tid == 0) p.inst_flag[TH_IDX(123, n, p.prob.n_instances)] = (skip_all || any_bad) ? kFlagBadInput : 0;
}

}  // namespace

cudaError_t launch_score(const Params &p, cudaStream_t stream)
{
    const size_t table = p.vertical ? (size_t)p.prob.n_stages * p.prob.n_batch
                                    : (size_t)p.prob.n_batch * p.prob.h_max;
    const int threads = p.pitch <= 1024 ? 128 : 256;
    const size_t smem = sizeof(uint32_t) * (2u * (size_t)p.pitch + 2u * table + 4u + (threads / 32) * kListWords + 32u);
    auto kernel = threads == 128 ? score_kernel<128> : score_kernel<256>;
    static std::atomic<uint64_t> ready128{0}, ready256{0};
    cudaError_t e = allow_max_smem(reinterpret_cast<const void *>(kernel), threads == 128 ? ready128 : ready256);
    if (e != cudaSuccess) return e;
    const bool joint_lists = (p.prob.flags & THEMIS_QUEUE_PER_REPLICA) && !p.horizontal && !p.vertical && p.prob.h_max > 1;
    score_lists_kernel<<<p.prob.n_profiles * p.prob.n_stages, 32 * p.prob.n_batch, 0, stream>>>(p, joint_lists ? 1 : 0);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    kernel<<<p.prob.n_instances, threads, smem, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace themis

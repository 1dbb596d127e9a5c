// The inner step of the 32-bit min-plus kernels: one chunk of R values of l against a thread's R
// budget cells, operands (packed keys, see themis_minplus.cu) from shared memory.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace themis {

template <int R>
struct Tile {
    static constexpr int kChunkStride = R + 4;   // words between chunk starts in shared F
};

// One chunk step: loads the next-lower chunk of F into w_lo and R keys of G, then
// updates acc[r] = min(acc[r], F[t0 + r - (l0 + k)] + G[l0 + k]) for all r, k.
// w_hi holds F[m .. m+R-1] and w_lo receives F[m-R .. m-1], m = t0 - l0.
template <int R>
__device__ __forceinline__ void chunk_step(const uint32_t (&w_hi)[R], uint32_t (&w_lo)[R], uint32_t (&acc)[R],
                                           const uint32_t *f_chunk, const uint32_t *g_chunk)
{
#pragma unroll
    for (int v = 0; v < R / 4; ++v) {
        const uint4 x = *reinterpret_cast<const uint4 *>(f_chunk + 4 * v);
        w_lo[4 * v + 0] = x.x; w_lo[4 * v + 1] = x.y; w_lo[4 * v + 2] = x.z; w_lo[4 * v + 3] = x.w;
    }
#pragma unroll
    for (int v = 0; v < R / 4; ++v) {
        const uint4 g4 = *reinterpret_cast<const uint4 *>(g_chunk + 4 * v);
        const uint32_t g[4] = {g4.x, g4.y, g4.z, g4.w};
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            const int k = 4 * v + kk;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int i = R + r - k;                       // 1 .. 2R-1
                const uint32_t f = i >= R ? w_hi[i - R] : w_lo[i];
                acc[r] = __viaddmin_u32(f, g[kk], acc[r]);
            }
        }
    }
}

}  // namespace themis

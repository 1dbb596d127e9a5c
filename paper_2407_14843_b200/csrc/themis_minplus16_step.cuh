// The inner step of the packed 16-bit min-plus kernel: one chunk of R values of l against a
// thread's R budget cells, operands from shared memory.  Shared by the recurrence kernel and by
// the throughput probe that times this step alone.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace themis {

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

}  // namespace themis

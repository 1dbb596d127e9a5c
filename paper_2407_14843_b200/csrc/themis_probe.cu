// Integer-ALU throughput probe: 16 independent add-then-min chains held in
// registers, the operation pair of the min-plus recurrence, in several
// instruction forms.  Every update reads two values produced one round earlier,
// so nothing can be hoisted and no memory is touched.  It measures what the
// arithmetic pipes sustain; it is not part of the method.
//
// Form 5 times the packed kernel's own inner step instead (themis_minplus16_step.cuh):
// columns of 256 chunk steps with the operands loaded from shared memory exactly as in
// the recurrence kernel, but no stages, barriers or global traffic around them.
#include "themis_async.cuh"
#include "themis_internal.h"
#include "themis_minplus16_step.cuh"

namespace themis {
namespace {

constexpr int kChains = 16;
constexpr int kRoundsPerIter = 4;

template <int MODE>
__global__ void alu_probe_kernel(int iters, uint32_t *sink)
{
    const uint32_t seed = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t g0 = (seed & 7u) + 1u, g1 = ((seed >> 3) & 7u) + 2u;
    uint32_t r = 0;
    if (MODE == 4) {
        float acc[kChains];
#pragma unroll
        for (int i = 0; i < kChains; ++i) acc[i] = 1.0e9f - (float)(seed * (i + 1) & 0xFFFF);
        const float fg0 = (float)g0, fg1 = (float)g1;
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int j = 0; j < kRoundsPerIter; ++j)
#pragma unroll
                for (int i = 0; i < kChains; ++i)
                    acc[i] = fminf(acc[i], acc[(i + 1) % kChains] + ((i & 1) ? fg1 : fg0));
        }
#pragma unroll
        for (int i = 0; i < kChains; ++i) r ^= __float_as_uint(acc[i]);
    } else {
        uint32_t acc[kChains];
#pragma unroll
        for (int i = 0; i < kChains; ++i) acc[i] = 0xF0000000u - seed * (i + 1);
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int j = 0; j < kRoundsPerIter; ++j) {
                if (MODE == 0) {            // add, then min: two instructions per update
#pragma unroll
                    for (int i = 0; i < kChains; ++i)
                        acc[i] = min(acc[i], acc[(i + 1) % kChains] + ((i & 1) ? g1 : g0));
                } else if (MODE == 1) {     // fused add-min: one instruction per update
#pragma unroll
                    for (int i = 0; i < kChains; ++i)
                        acc[i] = __viaddmin_u32(acc[(i + 1) % kChains], (i & 1) ? g1 : g0, acc[i]);
                } else if (MODE == 2) {     // two adds and one three-input min per two updates
#pragma unroll
                    for (int i = 0; i < kChains; i += 2) {
                        const uint32_t s0 = acc[(i + 1) % kChains] + g0;
                        const uint32_t s1 = acc[(i + 2) % kChains] + g1;
                        acc[i] = __vimin3_u32(acc[i], s0, s1);
                        const uint32_t s2 = acc[(i + 2) % kChains] + g0;
                        const uint32_t s3 = acc[(i + 3) % kChains] + g1;
                        acc[i + 1] = __vimin3_u32(acc[i + 1], s2, s3);
                    }
                } else {                    // MODE 3: packed 2 x 16-bit fused add-min
#pragma unroll
                    for (int i = 0; i < kChains; ++i)
                        acc[i] = __viaddmin_u16x2(acc[(i + 1) % kChains], (i & 1) ? g1 : g0, acc[i]);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < kChains; ++i) r ^= acc[i];
    }
    sink[blockIdx.x * blockDim.x + threadIdx.x] = r;
}

// 256 threads; thread i owns tile 256 + i of a 512-tile row and walks 256 chunks of l per
// column, `iters` columns.  One column = 256 * R * R / ... cell updates: 256 steps x R x R cells.
template <int R>
__global__ void __launch_bounds__(256) step_probe_kernel(int iters, uint32_t *sink)
{
    constexpr int H = Tile16<R>::H, CS = Tile16<R>::CS;
    constexpr int kTiles = 512, kSteps = 256, U = 64 / R;
    __shared__ __align__(16) uint32_t Fw[kTiles * CS];
    __shared__ __align__(16) uint32_t G[kSteps * R];
    const int tid = threadIdx.x;
    for (int i = tid; i < kTiles * CS; i += 256) Fw[i] = ((uint32_t)(i * 37 + blockIdx.x) & 0x3FFFu) * 0x00010001u;
    for (int i = tid; i < kSteps * R; i += 256) G[i] = ((uint32_t)(i * 11 + 5) & 0x0FFFu) * 0x00010001u;
    __syncthreads();
    uint32_t acc[H], accp[H], wa[H], wb[H];
#pragma unroll
    for (int r = 0; r < H; ++r) { acc[r] = 0xFFFFFFFFu; accp[r] = 0xFFFFFFFFu; }
    const uint32_t *f_hi = Fw + (256 + tid) * CS;
    for (int it = 0; it < iters; ++it) {
        load_words<H>(wa, f_hi);
        const uint32_t *f_lo = f_hi - CS, *g = G;
        for (int q = 0; q < kSteps; q += U) {
#pragma unroll
            for (int u = 0; u < U; u += 2) {
                chunk_step16<R>(wa, wb, acc, accp, f_lo - u * CS, g + u * R);
                chunk_step16<R>(wb, wa, acc, accp, f_lo - (u + 1) * CS, g + (u + 1) * R);
            }
            f_lo -= U * CS;
            g += U * R;
        }
    }
    uint32_t r = 0;
#pragma unroll
    for (int i = 0; i < H; ++i) r ^= acc[i] ^ accp[i];
    sink[blockIdx.x * blockDim.x + tid] = r;
}

// Bounded-wait probe: the same mbarrier wait the recurrence kernels use, once on a copy that
// is issued (must complete; the kernels' own limit, so that no copy is in flight when the block
// leaves) and once on a transaction that nothing delivers (must give up after `max_polls`
// attempts and report it).  One warp; the kernel returns normally in both cases.
__global__ void wait_probe_kernel(uint32_t max_polls, const uint32_t *src16, uint32_t *dst16, int32_t *status)
{
    __shared__ __align__(16) uint32_t buf[4];
    __shared__ __align__(8) uint64_t bar[2];
    if (threadIdx.x == 0) {
        mbar_init(&bar[0], 1);
        mbar_init(&bar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_expect_tx(&bar[0], 16);
        bulk_load(buf, src16, 16, &bar[0]);
        mbar_expect_tx(&bar[1], 16);              // these 16 bytes never come
    }
    const bool arrived = mbar_wait(&bar[0], 0);
    if (arrived && threadIdx.x < 4) dst16[threadIdx.x] = buf[threadIdx.x];
    const bool never = mbar_wait(&bar[1], 0, max_polls);
    if (threadIdx.x == 0) {
        status[0] = arrived ? THEMIS_STATUS_OK : THEMIS_STATUS_TIMEOUT;
        status[1] = never ? THEMIS_STATUS_OK : THEMIS_STATUS_TIMEOUT;
    }
}

}  // namespace

cudaError_t launch_alu_probe(int mode, int blocks, int threads, int iters, uint32_t *sink, cudaStream_t stream)
{
    switch (mode) {
        case 0: alu_probe_kernel<0><<<blocks, threads, 0, stream>>>(iters, sink); break;
        case 1: alu_probe_kernel<1><<<blocks, threads, 0, stream>>>(iters, sink); break;
        case 2: alu_probe_kernel<2><<<blocks, threads, 0, stream>>>(iters, sink); break;
        case 3: alu_probe_kernel<3><<<blocks, threads, 0, stream>>>(iters, sink); break;
        case 5:
            if (threads != 256) return cudaErrorInvalidValue;
            step_probe_kernel<8><<<blocks, 256, 0, stream>>>(iters, sink);
            break;
        default: alu_probe_kernel<4><<<blocks, threads, 0, stream>>>(iters, sink); break;
    }
    return cudaGetLastError();
}

cudaError_t launch_wait_probe(uint32_t max_polls, const uint32_t *src16, uint32_t *dst16, int32_t *status,
                              cudaStream_t stream)
{
    wait_probe_kernel<<<1, 32, 0, stream>>>(max_polls, src16, dst16, status);
    return cudaGetLastError();
}

}  // namespace themis

// Steady-state (cyclic) planning, preparation.  Section 4.2 notes that the inactive period of a global tensor may
// span two consecutive training iterations.  With the traced iteration repeating unchanged, the timeline is a cycle
// of K slots; unrolled slot k + K is slot k one iteration later.  This pass
//   - writes the unrolled clock start2[0 .. 2K] (start2[k + K] = start[k] + length of the iteration), and
//   - appends to the period list, after the ordinary periods, one wrap-around period (i, last use, first use + K)
//     for every used global tensor with at least one slot in between, in tensor order.
// One block: the mode is meant for traces that a single SM plans (a few thousand kernels).
#include "g10_device.cuh"
#include "g10_internal.h"

namespace g10 {

constexpr int kCycThreads = 1024;

__global__ void __launch_bounds__(kCycThreads) k_cyclic_prepare(int64_t K, int64_t N, const int64_t *__restrict__ start, int64_t *__restrict__ start2,
                                                                const uint8_t *__restrict__ glob, const int32_t *__restrict__ first_use,
                                                                const int32_t *__restrict__ last_use, int64_t periods_cap, int32_t *per_t,
                                                                int32_t *per_u, int32_t *per_v, int64_t *counts, ull *status)
{
    __shared__ int s_w[kCycThreads / 32];
    __shared__ long long s_base;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t T = start[K];
    for (int64_t k = threadIdx.x; k <= 2 * K; k += kCycThreads) start2[k] = k <= K ? start[k] : start[k - K] + T;
    if (threadIdx.x == 0) s_base = counts[1];
    __syncthreads();
    for (int64_t i0 = 0; i0 < N; i0 += kCycThreads) {
        const int64_t i = i0 + threadIdx.x;
        bool wrap = false;
        int f = -1, l = -1;
        if (i < N && glob && glob[i]) {
            f = first_use[i]; l = last_use[i];
            wrap = f >= 0 && (int64_t)f + K - l >= 2;
        }
        const unsigned m = __ballot_sync(0xffffffffu, wrap);
        if (lane == 0) s_w[warp] = __popc(m);
        __syncthreads();
        long long pos = s_base;
        int total = 0;
        for (int w = 0; w < kCycThreads / 32; ++w) { if (w < warp) pos += s_w[w]; total += s_w[w]; }
        pos += __popc(m & ((1u << lane) - 1u));
        if (wrap) {
            if (pos < periods_cap) { per_t[pos] = (int32_t)i; per_u[pos] = l; per_v[pos] = (int32_t)(f + K); }
            else raise_status(status, G10_DEV_PERIODS_OVERFLOW);
        }
        __syncthreads();
        if (threadIdx.x == 0) s_base += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) counts[1] = s_base;
}

cudaError_t launch_cyclic_prepare(const DeviceTrace &t, const Workspace &w, cudaStream_t s)
{
    k_cyclic_prepare<<<1, kCycThreads, 0, s>>>(t.K, t.N, w.start, w.start2, t.tensor_global, w.first_use, w.last_use, t.E,
                                               w.period_tensor, w.period_prev_use, w.period_next_use, w.counts, w.status); count_launch();
    return cudaGetLastError();
}

}  // namespace g10

// Smart tensor prefetching (Section 4.4): after the eviction plan is made, the evicted periods are visited in
// the order of their latest safe prefetch time and every prefetch is moved back to the earliest slot from which
// the GPU can hold the tensor with the space that is left; the pressure curve is updated as it goes.
//
// The pass is a strict sequence over the plan records (each move changes the pressure the next search sees), so
// one block does it: the records are ordered by a bitonic network over their indices, then, record by record, the
// block searches backward in chunks of its own width (a chunk stops the search as soon as one of its slots cannot
// take the tensor) and adds the tensor's size to the slots it regained.  Parallelism is inside each search.
#include "g10_device.cuh"
#include "g10_internal.h"

namespace g10 {

constexpr int kPfThreads = 1024;

__device__ __forceinline__ bool pf_before(const g10_migration *mig, int x, int y)
{
    const int64_t kx = mig[x].prefetch_issue_ns, ky = mig[y].prefetch_issue_ns;
    return kx < ky || (kx == ky && x < y);
}

__global__ void __launch_bounds__(kPfThreads) k_schedule_prefetch(int64_t K, int64_t n, const g10_migration *__restrict__ mig,
                                                                  const int64_t *__restrict__ start, const int64_t *__restrict__ bytes,
                                                                  int64_t cap, int64_t *P, int32_t *order, int32_t *new_last,
                                                                  int64_t *new_issue, int64_t *summary)
{
    __shared__ int s_stop;                 // highest slot of the current chunk that cannot take the tensor (-1: none)
    __shared__ long long s_mx[kPfThreads / 32];
    __shared__ int s_sl[kPfThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // ---- order the records by (latest safe prefetch time, record index)
    for (int64_t i = threadIdx.x; i < n; i += kPfThreads) order[i] = (int32_t)i;
    __syncthreads();
    int64_t n2 = 1;
    while (n2 < n) n2 <<= 1;
    for (int64_t k = 2; k <= n2; k <<= 1) {
        for (int64_t j = k >> 1; j > 0; j >>= 1) {
            const bool mirror = (j == (k >> 1));
            for (int64_t t = threadIdx.x; t < n2 / 2; t += kPfThreads) {
                const int64_t blk = t / j, off = t % j;
                const int64_t i = blk * 2 * j + off;
                const int64_t p = mirror ? (blk * 2 * j + 2 * j - 1 - off) : (i + j);
                if (p < n) {
                    const int32_t x = order[i], y = order[p];
                    if (pf_before(mig, y, x)) { order[i] = y; order[p] = x; }
                }
            }
            __syncthreads();
        }
    }
    // ---- visit the records in that order
    long long moved = 0, regained = 0;
    for (int64_t q = 0; q < n; ++q) {
        const int r = order[q];
        const int a_abs = mig[r].absent_first, b_abs = mig[r].absent_last;
        const int64_t s = bytes[mig[r].tensor];
        int hi = b_abs;                     // slots (j, b_abs] are known to take the tensor
        int j = a_abs - 1;                  // result: last slot that stays absent
        while (hi >= a_abs) {
            const int lo = hi - kPfThreads + 1 > a_abs ? hi - kPfThreads + 1 : a_abs;
            if (threadIdx.x == 0) s_stop = -1;
            __syncthreads();
            const int k = hi - (int)threadIdx.x;
            if (k >= lo && P[k] > cap - s) atomicMax(&s_stop, k);
            __syncthreads();
            const int stop = s_stop;
            __syncthreads();
            if (stop >= 0) { j = stop; break; }
            hi = lo - 1;
        }
        for (int k = j + 1 + (int)threadIdx.x; k <= b_abs; k += kPfThreads) P[k] += s;
        if (threadIdx.x == 0) {
            new_last[r] = j;
            new_issue[r] = j < b_abs ? start[j + 1] : mig[r].prefetch_issue_ns;
        }
        if (j < b_abs) { moved += 1; regained += b_abs - j; }
        __syncthreads();
    }
    // ---- new peak and its lowest slot
    long long mx = 0;
    int sl = -1;
    for (int64_t k = threadIdx.x; k < K; k += kPfThreads) {
        const long long pv = P[k];
        if (sl < 0 || pv > mx) { mx = pv; sl = (int)k; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const long long omx = __shfl_down_sync(0xffffffffu, mx, o);
        const int osl = __shfl_down_sync(0xffffffffu, sl, o);
        if (osl >= 0 && (sl < 0 || omx > mx || (omx == mx && osl < sl))) { mx = omx; sl = osl; }
    }
    if (lane == 0) { s_mx[warp] = mx; s_sl[warp] = sl; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kPfThreads / 32; ++w)
            if (s_sl[w] >= 0 && (sl < 0 || s_mx[w] > mx || (s_mx[w] == mx && s_sl[w] < sl))) { mx = s_mx[w]; sl = s_sl[w]; }
        summary[0] = moved; summary[1] = regained; summary[2] = sl < 0 ? 0 : mx; summary[3] = sl;
    }
}

cudaError_t launch_schedule_prefetch(int64_t K, int64_t n, const g10_migration *mig, const int64_t *start, const int64_t *bytes,
                                     uint64_t gpu_capacity_bytes, int64_t *P, int32_t *order, int32_t *new_last, int64_t *new_issue,
                                     int64_t *summary, cudaStream_t s)
{
    const int64_t cap = gpu_capacity_bytes >= ((uint64_t)1 << 63) ? INT64_MAX : (int64_t)gpu_capacity_bytes;
    k_schedule_prefetch<<<1, kPfThreads, 0, s>>>(K, n, mig, start, bytes, cap, P, order, new_last, new_issue, summary);
    return cudaGetLastError();
}

}  // namespace g10

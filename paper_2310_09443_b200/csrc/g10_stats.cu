// Workload characterisation (Section 3, Figures 2-4) from the vitality results of a trace:
//   active_bytes[k]  bytes of the tensors kernel k uses (the working set of Figure 2),
//   len_hist         inactive periods by floor(log2(length in ns))            (Figure 3),
//   size_len_hist    periods by floor(log2 size) x floor(log2 length)         (Figure 4),
//   hide             periods long enough for a round trip to the SSD / the host memory, 2 t <= L.
// The per-kernel sums go through the per-tensor use lists (already free of duplicates), one 64-bit atomic per
// (kernel, tensor) incidence; the histograms are counted in shared memory and flushed once per block.
#include "g10_device.cuh"
#include "g10_internal.h"

namespace g10 {

constexpr int kStatThreads = 256;
constexpr int kLenBins = 64, kSizeBins = 41, kLen2Bins = 45;

__global__ void __launch_bounds__(kStatThreads) k_active_bytes(int64_t N, const int64_t *__restrict__ use_ptr, const int32_t *__restrict__ uses,
                                                               const int64_t *__restrict__ bytes, ull *active)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kStatThreads + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * kStatThreads) >> 5;
    for (int64_t base = warp0 * 32; base < N; base += nwarps * 32) {
        const int64_t i = base + lane;
        int64_t lo = 0, hi = 0;
        ull s = 0;
        if (i < N) { lo = use_ptr[i]; hi = use_ptr[i + 1]; s = (ull)bytes[i]; }
        const bool heavy = hi - lo > 64;
        if (!heavy) for (int64_t j = lo; j < hi; ++j) atomicAdd(&active[uses[j]], s);
        unsigned m = __ballot_sync(0xffffffffu, heavy);
        while (m) {                                   // a tensor with a long use list: the warp shares it
            const int src = __ffs(m) - 1;
            m &= m - 1;
            const int64_t l2 = __shfl_sync(0xffffffffu, lo, src), h2 = __shfl_sync(0xffffffffu, hi, src);
            const ull s2 = __shfl_sync(0xffffffffu, s, src);
            for (int64_t j = l2 + lane; j < h2; j += 32) atomicAdd(&active[uses[j]], s2);
        }
    }
}

__device__ __forceinline__ int floor_log2(long long x) { return x > 1 ? 63 - __clzll(x) : 0; }

__global__ void __launch_bounds__(kStatThreads) k_period_hist(int64_t Pn, const int64_t *__restrict__ start, const int64_t *__restrict__ bytes,
                                                              const int32_t *__restrict__ per_t, const int32_t *__restrict__ per_u,
                                                              const int32_t *__restrict__ per_v, uint64_t host_bw, uint64_t ssd_bw,
                                                              ull *len_hist, ull *size_len_hist, ull *hide)
{
    __shared__ unsigned s_len[kLenBins];
    __shared__ unsigned s_sl[kSizeBins * kLen2Bins];
    __shared__ unsigned s_hide[2];
    for (int b = threadIdx.x; b < kLenBins; b += kStatThreads) s_len[b] = 0;
    for (int b = threadIdx.x; b < kSizeBins * kLen2Bins; b += kStatThreads) s_sl[b] = 0;
    if (threadIdx.x < 2) s_hide[threadIdx.x] = 0;
    __syncthreads();
    unsigned h0 = 0, h1 = 0;
    for (int64_t p = (int64_t)blockIdx.x * kStatThreads + threadIdx.x; p < Pn; p += (int64_t)gridDim.x * kStatThreads) {
        const long long L = start[per_v[p]] - start[per_u[p] + 1];
        const long long s = bytes[per_t[p]];
        const int bl = floor_log2(L), bs = floor_log2(s);
        atomicAdd(&s_len[bl], 1u);
        atomicAdd(&s_sl[min(bs, kSizeBins - 1) * kLen2Bins + min(bl, kLen2Bins - 1)], 1u);
        // ceil(s * 1e9 / bw) <= L / 2  <=>  s * 1e9 <= (L / 2) * bw
        const u128 need = (u128)(ull)s * (u128)1000000000ull, half = (u128)(ull)(L / 2);
        h0 += need <= half * (u128)ssd_bw;
        h1 += need <= half * (u128)host_bw;
    }
    h0 = __reduce_add_sync(0xffffffffu, h0);
    h1 = __reduce_add_sync(0xffffffffu, h1);
    if ((threadIdx.x & 31) == 0) { if (h0) atomicAdd(&s_hide[0], h0); if (h1) atomicAdd(&s_hide[1], h1); }
    __syncthreads();
    for (int b = threadIdx.x; b < kLenBins; b += kStatThreads) if (s_len[b]) atomicAdd(&len_hist[b], (ull)s_len[b]);
    for (int b = threadIdx.x; b < kSizeBins * kLen2Bins; b += kStatThreads) if (s_sl[b]) atomicAdd(&size_len_hist[b], (ull)s_sl[b]);
    if (threadIdx.x < 2 && s_hide[threadIdx.x]) atomicAdd(&hide[threadIdx.x], (ull)s_hide[threadIdx.x]);
}

// summary[0] = max active bytes; summary[1] primed for the arg-min pass (or -1 for an empty trace)
__global__ void __launch_bounds__(kStatThreads) k_active_max(int64_t K, const long long *__restrict__ active, long long *summary)
{
    __shared__ long long s_mx[kStatThreads / 32];
    long long mx = 0;
    for (int64_t k = (int64_t)blockIdx.x * kStatThreads + threadIdx.x; k < K; k += (int64_t)gridDim.x * kStatThreads) mx = max(mx, active[k]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_down_sync(0xffffffffu, mx, o));
    if ((threadIdx.x & 31) == 0) s_mx[threadIdx.x >> 5] = mx;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kStatThreads / 32; ++w) mx = max(mx, s_mx[w]);
        if (mx > 0) atomicMax(&summary[0], mx);
        if (blockIdx.x == 0) summary[1] = K > 0 ? 0x7fffffffffffffffll : -1ll;
    }
}

__global__ void __launch_bounds__(kStatThreads) k_active_argmax(int64_t K, const long long *__restrict__ active, long long *summary)
{
    const long long mx = summary[0];
    long long best = 0x7fffffffffffffffll;
    for (int64_t k = (int64_t)blockIdx.x * kStatThreads + threadIdx.x; k < K; k += (int64_t)gridDim.x * kStatThreads)
        if (active[k] == mx) { best = k; break; }       // the first hit of a thread is its lowest
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_down_sync(0xffffffffu, best, o));
    if ((threadIdx.x & 31) == 0 && best != 0x7fffffffffffffffll) atomicMin(&summary[1], best);
}

static int stat_grid(int64_t items, int per_block)
{
    int64_t g = (items + per_block - 1) / per_block;
    const int64_t cap = 148 * 8;
    return (int)(g < 1 ? 1 : (g > cap ? cap : g));
}

cudaError_t launch_characterize(int64_t K, int64_t N, const int64_t *use_ptr, const int32_t *uses, const int64_t *bytes, const int64_t *start,
                                int64_t Pn, const int32_t *per_t, const int32_t *per_u, const int32_t *per_v, uint64_t host_bw, uint64_t ssd_bw,
                                int64_t *active, int64_t *len_hist, int64_t *size_len_hist, int64_t *hide, int64_t *summary, cudaStream_t s)
{
    cudaError_t e;
    if (K > 0 && (e = cudaMemsetAsync(active, 0, (size_t)K * 8, s)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(len_hist, 0, kLenBins * 8, s)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(size_len_hist, 0, kSizeBins * kLen2Bins * 8, s)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(hide, 0, 16, s)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(summary, 0, 16, s)) != cudaSuccess) return e;
    if (N > 0 && K > 0) { k_active_bytes<<<stat_grid(N, kStatThreads), kStatThreads, 0, s>>>(N, use_ptr, uses, bytes, (ull *)active); count_launch(); }
    if (Pn > 0) {
        k_period_hist<<<stat_grid(Pn, kStatThreads * 4), kStatThreads, 0, s>>>(Pn, start, bytes, per_t, per_u, per_v, host_bw, ssd_bw,
                                                                               (ull *)len_hist, (ull *)size_len_hist, (ull *)hide); count_launch();
    }
    k_active_max<<<stat_grid(K, kStatThreads * 4), kStatThreads, 0, s>>>(K, (const long long *)active, (long long *)summary); count_launch();
    if (K > 0) { k_active_argmax<<<stat_grid(K, kStatThreads * 4), kStatThreads, 0, s>>>(K, (const long long *)active, (long long *)summary); count_launch(); }
    return cudaGetLastError();
}

}  // namespace g10

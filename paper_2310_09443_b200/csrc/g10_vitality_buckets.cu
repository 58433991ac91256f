// Tensor vitality (Section 4.2: born / dead / inactive periods) in three kernels that keep the random
// accesses on chip.  Tensors are cut into buckets of `bt` consecutive ids (a power of two, chosen so that a
// bucket holds a few thousand trace events):
//   1. k_bk_hist     counts the events of every bucket (shared-memory histogram per block);
//   2. k_bk_scatter  partitions the events by bucket: each event becomes one 64-bit key
//                    (tensor id inside the bucket << 32 | kernel) written into its bucket's slice;
//   3. k_bk_emit     takes one bucket at a time: sorts its keys in shared memory (bitonic network), after which
//                    the sorted distinct kernels of every tensor are adjacent -- first / last use, the use lists
//                    (repeats of a tensor inside one kernel collapse) and the inactive periods (consecutive
//                    distinct uses at least two kernels apart) all follow from comparing neighbours and from
//                    prefix counts; the offsets of a bucket in `uses` and in the period arrays are the sums of
//                    the totals of all earlier buckets, exchanged through tagged 64-bit words.
// Everything random happens in shared memory (atomics included); HBM sees the events twice, the keys once each
// way and the outputs once, all in coalesced runs.  A bucket whose keys do not fit in shared memory (a tensor
// listed by a great many kernels) is sorted in place in global memory by the same block: slower, same result.
#include "g10_device.cuh"
#include "g10_internal.h"

namespace g10 {

constexpr int kBkThreads = 512;
constexpr int kBkItems = 8;
constexpr int kBkTile = kBkThreads * kBkItems;     // events per partition tile
constexpr int kBkCap = 4096;                       // keys sorted in shared memory
constexpr int kBkPtrStage = 2048;                  // kernel_ptr entries staged per tile

struct BucketArgs {
    int64_t N, E, K;
    int shift;                 // log2(bt)
    int bt;                    // tensors per bucket
    int nb;                    // number of buckets
    unsigned *bucket_count;    // [nb] events per bucket
    unsigned *bucket_cursor;   // [nb] scatter cursors (start at zero)
    ull *pairs;                // [E] keys, bucket after bucket
    ull *words;                // [2 * nb] tagged totals of each bucket: distinct uses, periods
    unsigned *ticket;
    ull *status;
};

// exclusive scan of cnt[0..n) into out[0..n] (out[n] = total), n <= kBkMaxBuckets, whole block
__device__ __forceinline__ void block_scan_counts(const unsigned *cnt, int n, int *out, int *s_warp /* [32] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    int carry = 0;
    for (int base = 0; base < n; base += blockDim.x) {
        const int j = base + threadIdx.x;
        const int v = j < n ? (int)cnt[j] : 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
        __syncthreads();
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        int wpre = 0, tot = 0;
        for (int w = 0; w < nw; ++w) { const int x = s_warp[w]; if (w < warp) wpre += x; tot += x; }
        if (j < n) out[j] = carry + wpre + incl - v;
        carry += tot;
    }
    __syncthreads();
    if (threadIdx.x == 0) out[n] = carry;
    __syncthreads();
}

// last k in [lo, hi] with kptr[k] <= e
__device__ __forceinline__ int bk_kernel_of_event(const int64_t *kptr, int lo, int hi, int64_t e)
{
    while (lo < hi) {
        const int mid = lo + (hi - lo + 1) / 2;
        if (kptr[mid] <= e) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// ---------------------------------------------------------------------------------------------
// 1. events per bucket
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kBkThreads) k_bk_hist(BucketArgs B, const int32_t *__restrict__ kt)
{
    extern __shared__ unsigned s_hist[];
    for (int b = threadIdx.x; b < B.nb; b += kBkThreads) s_hist[b] = 0;
    __syncthreads();
    ull bad = 0;
    const int64_t tiles = (B.E + kBkTile - 1) / kBkTile;
    for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const int64_t base = tile * kBkTile;
        int32_t id[kBkItems];
#pragma unroll
        for (int j = 0; j < kBkItems; ++j) {
            const int64_t e = base + (int64_t)j * kBkThreads + threadIdx.x;
            id[j] = e < B.E ? kt[e] : -2;
        }
#pragma unroll
        for (int j = 0; j < kBkItems; ++j) {
            if (id[j] == -2) continue;
            if (id[j] < 0 || id[j] >= B.N) bad = G10_DEV_BAD_TENSOR_ID;
            else atomicAdd(&s_hist[id[j] >> B.shift], 1u);
        }
    }
    if (bad) raise_status(B.status, bad);
    __syncthreads();
    for (int b = threadIdx.x; b < B.nb; b += kBkThreads)
        if (s_hist[b]) atomicAdd(&B.bucket_count[b], s_hist[b]);
}

// ---------------------------------------------------------------------------------------------
// 2. partition the events by bucket
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kBkThreads) k_bk_scatter(BucketArgs B, const int64_t *__restrict__ kptr, const int32_t *__restrict__ kt)
{
    extern __shared__ int s_mem[];
    int *s_base = s_mem;                          // [nb + 1] first key of each bucket
    unsigned *s_cnt = (unsigned *)(s_base + B.nb + 1);   // [nb] events of this tile per bucket
    unsigned *s_off = s_cnt + B.nb;               // [nb] where this tile's events start inside the bucket
    __shared__ int s_warp[32];
    __shared__ int64_t s_ptr[kBkPtrStage];
    __shared__ int s_lohi[2];
    block_scan_counts(B.bucket_count, B.nb, s_base, s_warp);
    const int64_t tiles = (B.E + kBkTile - 1) / kBkTile;
    for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const int64_t base = tile * kBkTile;
        for (int b = threadIdx.x; b < B.nb; b += kBkThreads) s_cnt[b] = 0;
        if (threadIdx.x == 0) {
            const int64_t last = (base + kBkTile <= B.E ? base + kBkTile : B.E) - 1;
            s_lohi[0] = bk_kernel_of_event(kptr, 0, (int)B.K - 1, base);
            s_lohi[1] = bk_kernel_of_event(kptr, s_lohi[0], (int)B.K - 1, last);
        }
        __syncthreads();
        int lo = s_lohi[0], hi = s_lohi[1], shift_k = 0;
        const int64_t *sp = kptr;
        if (hi - lo + 2 <= kBkPtrStage) {
            for (int j = threadIdx.x; j <= hi - lo + 1; j += kBkThreads) s_ptr[j] = kptr[lo + j];
            shift_k = lo; hi -= lo; lo = 0; sp = s_ptr;
        }
        __syncthreads();
        int bucket[kBkItems];
        unsigned rank[kBkItems];
        ull key[kBkItems];
#pragma unroll
        for (int j = 0; j < kBkItems; ++j) {
            const int64_t e = base + (int64_t)j * kBkThreads + threadIdx.x;
            bucket[j] = -1;
            if (e < B.E) {
                const int32_t i = kt[e];
                if (i >= 0 && i < B.N) {
                    const int k = bk_kernel_of_event(sp, lo, hi, e) + shift_k;
                    bucket[j] = i >> B.shift;
                    key[j] = ((ull)(unsigned)(i & (B.bt - 1)) << 32) | (unsigned)k;
                    rank[j] = atomicAdd(&s_cnt[bucket[j]], 1u);
                }
            }
        }
        __syncthreads();
        for (int b = threadIdx.x; b < B.nb; b += kBkThreads)
            if (s_cnt[b]) s_off[b] = atomicAdd(&B.bucket_cursor[b], s_cnt[b]);
        __syncthreads();
#pragma unroll
        for (int j = 0; j < kBkItems; ++j)
            if (bucket[j] >= 0) {
                const int64_t pos = (int64_t)s_base[bucket[j]] + s_off[bucket[j]] + rank[j];
                if (pos < B.E) B.pairs[pos] = key[j];
            }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------
// 3. one bucket at a time: sort, compare neighbours, count, emit
// ---------------------------------------------------------------------------------------------
__device__ void bk_bitonic_sort(ull *a, int n)          // arbitrary n: the network only ever moves values up
{
    int n2 = 1;
    while (n2 < n) n2 <<= 1;
    for (int k = 2; k <= n2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            const bool mirror = (j == (k >> 1));
            for (int t = threadIdx.x; t < n2 / 2; t += blockDim.x) {
                const int blk = t / j, off = t % j;
                const int i = blk * 2 * j + off;
                const int p = mirror ? (blk * 2 * j + 2 * j - 1 - off) : (i + j);
                if (p < n) {
                    const ull x = a[i], y = a[p];
                    if (x > y) { a[i] = y; a[p] = x; }
                }
            }
            __syncthreads();
        }
    }
}

struct BkFlags {
    bool head, tail, dist, per;
    int tl, k, kprev;
};

__device__ __forceinline__ BkFlags bk_flags(const ull *kp, int j, int n)
{
    BkFlags f;
    const ull cur = kp[j];
    f.tl = (int)(cur >> 32); f.k = (int)(unsigned)cur;
    f.head = true; f.kprev = 0;
    if (j > 0) {
        const ull prev = kp[j - 1];
        f.head = (int)(prev >> 32) != f.tl;
        f.kprev = (int)(unsigned)prev;
    }
    f.dist = f.head || f.kprev != f.k;
    f.per = f.dist && !f.head && (f.k - f.kprev >= 2);
    f.tail = (j == n - 1) || ((int)(kp[j + 1] >> 32) != f.tl);
    return f;
}

__device__ __forceinline__ ull bk_pack(long long v) { return (1ull << 62) | ((ull)v & ((1ull << 62) - 1)); }

__global__ void __launch_bounds__(kBkThreads) k_bk_emit(BucketArgs B, VitalityBuffers out)
{
    extern __shared__ int s_mem[];
    int *s_base = s_mem;                                   // [nb + 1]
    int *t_first = s_base + B.nb + 1;                      // [bt] per-tensor results of the current bucket
    int *t_last = t_first + B.bt;
    int *t_nuse = t_last + B.bt;                           // counts, then exclusive offsets (bt + 1 entries)
    int *t_nper = t_nuse + B.bt + 1;                       // counts, then exclusive offsets (bt + 1 entries)
    ull *s_keys = (ull *)(((uintptr_t)(t_nper + B.bt + 1) + 7) & ~(uintptr_t)7);   // [kBkCap]
    __shared__ int s_warp[32];
    __shared__ int s_wa[kBkThreads / 32], s_wb[kBkThreads / 32];
    __shared__ int s_bucket;
    __shared__ long long s_pre[2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    block_scan_counts(B.bucket_count, B.nb, s_base, s_warp);
    for (;;) {
        __syncthreads();
        if (threadIdx.x == 0) s_bucket = (int)atomicAdd(B.ticket, 1u);
        __syncthreads();
        const int b = s_bucket;
        if (b >= B.nb) break;
        const int n = s_base[b + 1] - s_base[b];
        const int64_t t0 = (int64_t)b * B.bt;
        const int bt_eff = (int)((B.N - t0) < B.bt ? (B.N - t0) : B.bt);
        ull *gk = B.pairs + s_base[b];
        const ull *kp;
        // ---- sort the bucket's keys
        if (n <= kBkCap) {
            for (int j = threadIdx.x; j < n; j += kBkThreads) s_keys[j] = gk[j];
            __syncthreads();
            bk_bitonic_sort(s_keys, n);
            kp = s_keys;
        } else {
            __syncthreads();
            bk_bitonic_sort(gk, n);
            __threadfence_block();
            kp = gk;
        }
        for (int tl = threadIdx.x; tl <= bt_eff; tl += kBkThreads) {
            if (tl < bt_eff) { t_first[tl] = -1; t_last[tl] = -1; }
            t_nuse[tl] = 0; t_nper[tl] = 0;
        }
        __syncthreads();
        // ---- pass A: per-tensor first / last / counts
        for (int j = threadIdx.x; j < n; j += kBkThreads) {
            const BkFlags f = bk_flags(kp, j, n);
            if (f.head) t_first[f.tl] = f.k;
            if (f.tail) t_last[f.tl] = f.k;
            if (f.dist) atomicAdd(&t_nuse[f.tl], 1);
            if (f.per) atomicAdd(&t_nper[f.tl], 1);
        }
        __syncthreads();
        // in-place exclusive scans over the tensors of the bucket: [bt_eff] becomes the bucket total
        {
            int ca = 0, cb = 0;
            for (int base = 0; base < bt_eff; base += kBkThreads) {
                const int tl = base + threadIdx.x;
                const int va = tl < bt_eff ? t_nuse[tl] : 0, vb = tl < bt_eff ? t_nper[tl] : 0;
                int ia = va, ib = vb;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int ya = __shfl_up_sync(0xffffffffu, ia, o), yb = __shfl_up_sync(0xffffffffu, ib, o);
                    if (lane >= o) { ia += ya; ib += yb; }
                }
                __syncthreads();
                if (lane == 31) { s_wa[warp] = ia; s_wb[warp] = ib; }
                __syncthreads();
                int pa = 0, pb = 0, ta = 0, tb = 0;
                for (int w = 0; w < kBkThreads / 32; ++w) {
                    if (w < warp) { pa += s_wa[w]; pb += s_wb[w]; }
                    ta += s_wa[w]; tb += s_wb[w];
                }
                if (tl < bt_eff) { t_nuse[tl] = ca + pa + ia - va; t_nper[tl] = cb + pb + ib - vb; }
                ca += ta; cb += tb;
            }
            __syncthreads();
            if (threadIdx.x == 0) { t_nuse[bt_eff] = ca; t_nper[bt_eff] = cb; }
            __syncthreads();
        }
        const long long D = t_nuse[bt_eff], PC = t_nper[bt_eff];
        // ---- offsets of this bucket in the global arrays: totals of all earlier buckets
        if (threadIdx.x == 0) {
            asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(&B.words[2 * b]), "l"(bk_pack(D)) : "memory");
            asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(&B.words[2 * b + 1]), "l"(bk_pack(PC)) : "memory");
        }
        long long pu = 0, pp = 0;
        for (int j = threadIdx.x; j < 2 * b; j += kBkThreads) {
            ull w;
            unsigned polls = 0;
            for (;;) {
                asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(w) : "l"(&B.words[j]) : "memory");
                if (w >> 62) break;
                if (++polls > kSpinLimit) { raise_status(B.status, G10_DEV_TIMEOUT); w = 0; break; }
                __nanosleep(64);
            }
            const long long v = (long long)(w & ((1ull << 62) - 1));
            if (j & 1) pp += v; else pu += v;
        }
        pu = warp_sum_i64(pu); pp = warp_sum_i64(pp);
        __shared__ long long s_pu[kBkThreads / 32], s_pp[kBkThreads / 32];
        if (lane == 0) { s_pu[warp] = pu; s_pp[warp] = pp; }
        __syncthreads();
        if (threadIdx.x == 0) {
            long long a = 0, c2 = 0;
            for (int w = 0; w < kBkThreads / 32; ++w) { a += s_pu[w]; c2 += s_pp[w]; }
            s_pre[0] = a; s_pre[1] = c2;
        }
        __syncthreads();
        const long long U = s_pre[0], PB = s_pre[1];
        ull bad = 0;
        if (U + D > out.uses_cap) bad |= G10_DEV_USES_OVERFLOW;
        if (PB + PC > out.periods_cap) bad |= G10_DEV_PERIODS_OVERFLOW;
        if (bad && threadIdx.x == 0) raise_status(B.status, bad);
        // ---- per-tensor outputs, coalesced
        for (int tl = threadIdx.x; tl < bt_eff; tl += kBkThreads) {
            const int64_t t = t0 + tl;
            out.first_use[t] = t_first[tl];
            out.last_use[t] = t_last[tl];
            out.num_uses[t] = t_nuse[tl + 1] - t_nuse[tl];
            out.use_ptr[t] = U + t_nuse[tl];
            out.period_ptr[t] = PB + t_nper[tl];
        }
        if (b == B.nb - 1 && threadIdx.x == 0) {
            out.use_ptr[B.N] = U + D; out.period_ptr[B.N] = PB + PC;
            out.counts[0] = U + D; out.counts[1] = PB + PC;
        }
        // ---- pass B: sorted distinct uses and periods; positions are prefix counts of the flags
        {
            int ca = 0, cb = 0;
            for (int base = 0; base < n; base += kBkThreads) {
                const int j = base + threadIdx.x;
                BkFlags f;
                f.dist = false; f.per = false; f.tl = 0; f.k = 0; f.kprev = 0;
                if (j < n) f = bk_flags(kp, j, n);
                const unsigned md = __ballot_sync(0xffffffffu, f.dist), mp = __ballot_sync(0xffffffffu, f.per);
                __syncthreads();
                if (lane == 0) { s_wa[warp] = __popc(md); s_wb[warp] = __popc(mp); }
                __syncthreads();
                int pa = 0, pb = 0, ta = 0, tb = 0;
                for (int w = 0; w < kBkThreads / 32; ++w) {
                    if (w < warp) { pa += s_wa[w]; pb += s_wb[w]; }
                    ta += s_wa[w]; tb += s_wb[w];
                }
                const unsigned below = (1u << lane) - 1u;
                if (f.dist) {
                    const long long pos = U + ca + pa + __popc(md & below);
                    if (pos < out.uses_cap) out.uses[pos] = f.k;
                }
                if (f.per) {
                    const long long pos = PB + cb + pb + __popc(mp & below);
                    if (pos < out.periods_cap) {
                        out.period_tensor[pos] = (int32_t)(t0 + f.tl);
                        out.period_prev_use[pos] = f.kprev;
                        out.period_next_use[pos] = f.k;
                    }
                }
                ca += ta; cb += tb;
            }
        }
    }
}

// Picks the bucket width for a trace; false if the trace is outside what the bucket path handles.
static bool choose_buckets(int64_t N, int64_t E, int *shift, int *bt, int *nb)
{
    if (N <= 0) return false;
    int64_t want = E > 0 ? (2500 * N) / E : 4096;        // tensors per bucket for about 2500 events
    int s = 6;
    while (s < 12 && ((int64_t)1 << (s + 1)) <= want) ++s;
    while (s < 12 && ((N + ((int64_t)1 << s) - 1) >> s) > 4096) ++s;
    const int64_t buckets = (N + ((int64_t)1 << s) - 1) >> s;
    if (buckets > 4096) return false;
    *shift = s; *bt = 1 << s; *nb = (int)buckets;
    return true;
}

bool vitality_buckets_supported(int64_t N, int64_t E)
{
    int a, b, c;
    return choose_buckets(N, E, &a, &b, &c);
}

cudaError_t launch_vitality_buckets(const DeviceTrace &t, const Workspace &w, const VitalityBuffers &out, cudaStream_t s)
{
    BucketArgs B;
    B.N = t.N; B.E = t.E; B.K = t.K;
    if (!choose_buckets(t.N, t.E, &B.shift, &B.bt, &B.nb)) return cudaErrorInvalidValue;
    B.bucket_count = w.bk_count; B.bucket_cursor = w.bk_cursor; B.pairs = w.bk_pairs; B.words = w.bk_words;
    B.ticket = w.emit_scan.ticket; B.status = w.status;
    static int sms = 0;
    if (sms == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
            sms = 0;
            return cudaErrorInvalidDevice;
        }
    }
    const int64_t tiles = (t.E + kBkTile - 1) / kBkTile;
    if (t.E > 0 && t.K > 0) {
        const int g = (int)(tiles < 2 * (int64_t)sms ? tiles : 2 * (int64_t)sms);
        k_bk_hist<<<g, kBkThreads, sizeof(unsigned) * (size_t)B.nb, s>>>(B, t.kernel_tensors);
        const size_t sm2 = sizeof(int) * (size_t)(3 * B.nb + 1);
        cudaError_t e = cudaFuncSetAttribute(k_bk_scatter, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm2);
        if (e != cudaSuccess) return e;
        k_bk_scatter<<<g, kBkThreads, sm2, s>>>(B, t.kernel_ptr, t.kernel_tensors);
    }
    const size_t sm3 = sizeof(int) * (size_t)(B.nb + 1 + 4 * B.bt + 2) + 8 + sizeof(ull) * kBkCap;
    cudaError_t e = cudaFuncSetAttribute(k_bk_emit, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm3);
    if (e != cudaSuccess) return e;
    const int g3 = B.nb < 2 * sms ? B.nb : 2 * sms;
    k_bk_emit<<<g3, kBkThreads, sm3, s>>>(B, out);
    return cudaGetLastError();
}

}  // namespace g10

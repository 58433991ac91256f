// The memory-pressure timeline call (Section 4.3: pressure at a kernel = bytes of the tensors alive there) in two
// kernels, without first / last-use arrays ever leaving the chip's caches as separate passes:
//
//   k_tl_init      one streaming pass: checks tensor_bytes and kernel_ptr, clears the difference array and gives
//                  every tensor an 8-byte record {first, last} (Section 4.2: born at its first use, dead after its
//                  last), both encoded so that "no use yet" is 0 and later events can only raise them.
//   k_timeline     a persistent grid.  Phase 1 walks the trace events.  Two neighbouring lanes share an event: one
//                  raises the tensor's `first` word, the other its `last` word, with returning atomic maxima (both
//                  words lie in one 32-byte sector, so the pair costs the L2 one request).  A lane that raised a
//                  word moves the tensor's birth (or death) to its own kernel: it adds the tensor's size to the
//                  difference array there and takes back what the previous holder had added.  The sums telescope,
//                  so whatever order the events arrive in, the array ends as  D[first] += size, D[last + 1] -= size.
//                  Entries of the block's own run of kernels are kept in shared memory and flushed once.
//                  Phase 2, after one grid barrier, scans kernel_ns into the slot clock and the difference array
//                  into the pressure in the same sweep (each block one contiguous segment, the segment sums exchanged
//                  through tagged words) and reduces the peak and its lowest slot.
//
// A tensor flagged global is alive in every slot if it is used at all (Section 4.2: allocated when the program
// starts): its record starts with `first` saturated (no event can raise it: no birth is booked) and `last` at a
// marker that the first event to arrive swaps for "used", adding the size to D[0]; no death is booked.
#include <climits>
#ifdef G10_TL_CLOCKS
#include <cstdio>
#define TLC(i) do { if (threadIdx.x == 0) { const ull n_ = global_timer_ns(); tacc[i] += n_ - tlast; tlast = n_; } } while (0)
#else
#define TLC(i)
#endif

#include "g10_device.cuh"
#include "g10_internal.h"

namespace g10 {

constexpr int kTlThreads = 512;
constexpr int kTlWarps = kTlThreads / 32;
constexpr int kTlItems = 16;                            // half-events per thread and round
constexpr int kTlRound = kTlItems * kTlThreads / 2;     // events per round (4096)
constexpr int kTlWide = 64;                             // a kernel with more events is expanded by its whole warp
constexpr int kTlMaxTileKernels = 2048;                 // kernels per tile, at most (their difference entries sit in shared memory)
constexpr int kTlScanItems = 8;
constexpr int kTlChunk = kTlThreads * kTlScanItems;
constexpr int kGlobalSaturated = 0x7fffffff;            // `first` of a global tensor; `last` of a global tensor that is used
constexpr int kGlobalUnused = 0x7ffffff0;               // `last` of a global tensor no event has reached yet

struct TlArgs {
    int64_t K, N, E;
    const int64_t *kptr;
    const int32_t *kt;
    const int64_t *bytes;
    const int64_t *dur;
    const uint8_t *glob;
    int *pair;                 // [2 * N] first (as K - k), last (as k + 1); 0 = no use yet
    ull *diff;                 // [K + 1]
    int64_t *start;            // [K + 1]
    int64_t *P;                // [K]
    int64_t *peak_bytes;
    int32_t *peak_slot;
    ull *words;                // [2 * grid] tagged segment sums: slot clock, pressure
    int64_t *blk_max;          // [grid]
    int32_t *blk_slot;         // [grid]
    unsigned *done;
    GridBarrier *bar;
    ull *status;
    int tile_kernels;
    int vec_ok;                // tensor_bytes is 16-byte aligned and tensor_global 2-byte aligned: k_tl_init takes tensors two at a time
};

// ---------------------------------------------------------------------------------------------
// k_tl_init
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_tl_init(TlArgs A)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    ull bad = 0;
    // tensors two at a time (16-byte loads and stores, when the launcher found the pointers aligned), four pairs per thread in flight
    const int64_t N2 = A.vec_ok ? A.N / 2 : 0;
    const longlong2 *bytes2 = reinterpret_cast<const longlong2 *>(A.bytes);
    const uchar2 *glob2 = reinterpret_cast<const uchar2 *>(A.glob);
    int4 *pair2 = reinterpret_cast<int4 *>(A.pair);
    for (int64_t i0 = t0; i0 < N2; i0 += 4 * stride) {
        longlong2 b[4];
        uchar2 g[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t i = i0 + j * stride;
            b[j] = i < N2 ? bytes2[i] : make_longlong2(1, 1);
            g[j] = (i < N2 && glob2 != nullptr) ? glob2[i] : make_uchar2(0, 0);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t i = i0 + j * stride;
            if (b[j].x < 1 || b[j].x >= ((long long)1 << 40) || b[j].y < 1 || b[j].y >= ((long long)1 << 40)) bad |= G10_DEV_BAD_BYTES;
            if (i < N2) pair2[i] = make_int4(g[j].x ? kGlobalSaturated : 0, g[j].x ? kGlobalUnused : 0, g[j].y ? kGlobalSaturated : 0, g[j].y ? kGlobalUnused : 0);
        }
    }
    for (int64_t i = 2 * N2 + t0; i < A.N; i += stride) {               // the odd tensor at the end; every tensor when a pointer is not 16-byte aligned
        const long long b = A.bytes[i];
        if (b < 1 || b >= ((long long)1 << 40)) bad |= G10_DEV_BAD_BYTES;
        const bool g = A.glob != nullptr && A.glob[i] != 0;
        reinterpret_cast<int2 *>(A.pair)[i] = g ? make_int2(kGlobalSaturated, kGlobalUnused) : make_int2(0, 0);
    }
    for (int64_t k0 = t0; k0 <= A.K; k0 += 4 * stride) {
        int64_t p0[4], p1[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t k = k0 + j * stride;
            p0[j] = k < A.K ? A.kptr[k] : 0;
            p1[j] = k < A.K ? A.kptr[k + 1] : 0;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t k = k0 + j * stride;
            if (k <= A.K) A.diff[k] = 0;
            if (k < A.K && (p0[j] > p1[j] || p0[j] < 0 || p1[j] > A.E || (k == 0 && p0[j] != 0) || (k == A.K - 1 && p1[j] != A.E)))
                bad |= G10_DEV_BAD_KERNEL_PTR;
        }
    }
    if (bad) raise_status(A.status, bad);
}

// ---------------------------------------------------------------------------------------------
// k_timeline
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ ull tl_pack(long long v) { return (1ull << 62) | ((ull)v & ((1ull << 62) - 1)); }
__device__ __forceinline__ long long tl_unpack(ull w) { return (long long)(w << 2) >> 2; }     // sign-extend 62 bits

// sum over the block's warps of one value per warp (s_w written by the lanes 0 before a barrier); also the sum over
// the warps before this one
__device__ __forceinline__ long long tl_warp_totals(const long long *s_w, int lane, int warp, long long *before)
{
    const long long x = lane < kTlWarps ? s_w[lane] : 0;
    long long incl = x;
#pragma unroll
    for (int o = 1; o < kTlWarps; o <<= 1) {
        const long long y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    *before = __shfl_sync(0xffffffffu, incl - x, warp);
    return __shfl_sync(0xffffffffu, incl, kTlWarps - 1);
}

__global__ void __launch_bounds__(kTlThreads, 2) k_timeline(TlArgs A)
{
    __shared__ unsigned short s_krel[kTlRound];            // kernel of every event of the round, relative to the tile
    // bytes born at / dead before every kernel of the tile (and the one after it), each a 64-bit sum kept as two 32-bit
    // halves: native shared-memory atomics, the low half's carry handed to the high half (exact: adds to a word are serial)
    __shared__ unsigned s_pos_lo[kTlMaxTileKernels + 2], s_pos_hi[kTlMaxTileKernels + 2], s_neg_lo[kTlMaxTileKernels + 2], s_neg_hi[kTlMaxTileKernels + 2];
    __shared__ long long s_w[2][kTlWarps];
    __shared__ int s_sl[kTlWarps];
    __shared__ bool s_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int G = gridDim.x;
    const int64_t K = A.K;
#ifdef G10_TL_CLOCKS
    ull tacc[10] = {0,0,0,0,0,0,0,0,0,0}, tlast = global_timer_ns(); const ull tbeg = tlast; int nrounds = 0;
#endif
    unsigned gen = 0;
    // (launched with programmatic stream serialisation behind k_tl_init: the blocks are placed while it drains)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const bool walk = A.E > 0 && !(*(volatile ull *)A.status & G10_DEV_BAD_KERNEL_PTR);   // (else: every tensor comes out unused)
    // ------------------------------------------------------------------ phase 1: the events
    // (all trace dimensions are below 2^31: 32-bit indices throughout)
    if (walk) {
        const int Ki = (int)K, Ni = (int)A.N;
        const int TK = A.tile_kernels;
        const int tiles = (Ki + TK - 1) / TK;
        const int half = threadIdx.x & 1, qt = threadIdx.x >> 1;
        // a `first` lane books births at its kernel, a `last` lane deaths at the kernel after; taking a booking back adds to the other table
        unsigned *own_lo = half ? s_neg_lo + 1 : s_pos_lo, *own_hi = half ? s_neg_hi + 1 : s_pos_hi;
        unsigned *oth_lo = half ? s_pos_lo : s_neg_lo, *oth_hi = half ? s_pos_hi : s_neg_hi;
        int *my_pair = A.pair + half;
        ull bad = 0;
#pragma unroll 1
        for (int tile = blockIdx.x; tile < tiles; tile += G) {
            const int tk0 = tile * TK, tk1 = tk0 + TK < Ki ? tk0 + TK : Ki;
            const int T0 = (int)A.kptr[tk0], T1 = (int)A.kptr[tk1];
            for (int x = threadIdx.x; x <= tk1 - tk0 + 1; x += kTlThreads) { s_pos_lo[x] = 0; s_pos_hi[x] = 0; s_neg_lo[x] = 0; s_neg_hi[x] = 0; }
#pragma unroll 1
            for (int eb = T0; eb < T1; eb += kTlRound) {
                const int ee = eb + kTlRound < T1 ? eb + kTlRound : T1;
                const int n_round = ee - eb;
                // (a) kernel of every event of the round: a lane per kernel writes its number over its events' positions
#pragma unroll 1
                for (int k00 = tk0 + warp * 32; k00 < tk1; k00 += 2 * kTlThreads) {
                    int pa[2], pb[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {                              // two sweeps' loads in flight together
                        const int k = k00 + u * kTlThreads + lane;
                        pa[u] = (int)A.kptr[k < tk1 ? k : tk1];
                        pb[u] = (int)A.kptr[k + 1 < tk1 ? k + 1 : tk1];
                    }
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int k0 = k00 + u * kTlThreads;
                        if (k0 >= tk1) break;                                  // (uniform in the warp)
                        const int a = max(min(pa[u], ee), eb) - eb, b = max(min(pb[u], ee), eb) - eb;
                        const bool wide = b - a > kTlWide;
                        const unsigned short rel = (unsigned short)(k0 + lane - tk0);
                        if (!wide)
                            for (int p = a; p < b; ++p) s_krel[p] = rel;
                        unsigned m = __ballot_sync(0xffffffffu, wide);
#pragma unroll 1
                        while (m) {
                            const int src = __ffs(m) - 1;
                            m &= m - 1;
                            const int wa = __shfl_sync(0xffffffffu, a, src), wb = __shfl_sync(0xffffffffu, b, src);
                            const unsigned short wrel = (unsigned short)(k0 + src - tk0);
                            for (int p = wa + lane; p < wb; p += 32) s_krel[p] = wrel;
                        }
                    }
                }
                __syncthreads();
                TLC(0);
#ifdef G10_TL_CLOCKS
                ++nrounds;
#endif
                // (b) the events, two lanes each.  All tensor ids of the round first; then, eight items at a time: the
                // returning maxima (all in flight together), the sizes of the lanes that raised a word, their bookings.
                int32_t id[kTlItems];
                unsigned live = 0;                                                 // items of this lane that still have work
                const int32_t *kt = A.kt + eb;
#pragma unroll
                for (int j = 0; j < kTlItems; ++j) {
                    const int q = j * (kTlThreads / 2) + qt;
                    id[j] = 0;
                    if (q < n_round) { id[j] = kt[q]; live |= 1u << j; }
                }
#pragma unroll
                for (int j = 0; j < kTlItems; ++j)
                    if ((live >> j & 1u) && (unsigned)id[j] >= (unsigned)Ni) { bad |= G10_DEV_BAD_TENSOR_ID; live &= ~(1u << j); }
                TLC(1);
#pragma unroll
                for (int h = 0; h < kTlItems; h += 8) {
                    int old[8], rel[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        old[j] = 0;
                        rel[j] = s_krel[(h + j) * (kTlThreads / 2) + qt];
                        if (live >> (h + j) & 1u) old[j] = atomicMax(my_pair + 2 * (size_t)(unsigned)id[h + j], half ? tk0 + rel[j] + 1 : Ki - tk0 - rel[j]);
                    }
                    long long sz[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        sz[j] = 0;
                        const int val = half ? tk0 + rel[j] + 1 : Ki - tk0 - rel[j];
                        if ((live >> (h + j) & 1u) && (old[j] < val || old[j] == kGlobalUnused)) sz[j] = A.bytes[(unsigned)id[h + j]];
                        else old[j] = -1;                                          // nothing to book for this lane
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int o = old[j];
                        if (o < 0) continue;
                        const unsigned lo = (unsigned)(ull)sz[j], hi = (unsigned)((ull)sz[j] >> 32);
                        if (o == kGlobalUnused) {                              // (only a `last` lane can see this marker)
                            if (atomicMax(&A.pair[2 * (size_t)id[h + j] + 1], kGlobalSaturated) == kGlobalUnused) atomicAdd(&A.diff[0], (ull)sz[j]);
                            continue;
                        }
                        // born at this kernel (first lane) / dead after it (last lane): this lane's own table, always inside the tile
                        const unsigned was = atomicAdd(&own_lo[rel[j]], lo);
                        if (hi | (unsigned)(was + lo < was)) atomicAdd(&own_hi[rel[j]], hi + (was + lo < was ? 1u : 0u));
                        if (o != 0) {
                            // ... and not where the earlier holder had booked it: the same amount into the other table there
                            const int x = half ? o : Ki - o;
                            const unsigned xr = (unsigned)(x - tk0);
                            if (xr <= (unsigned)(tk1 - tk0)) {
                                const unsigned w2 = atomicAdd(&oth_lo[xr], lo);
                                if (hi | (unsigned)(w2 + lo < w2)) atomicAdd(&oth_hi[xr], hi + (w2 + lo < w2 ? 1u : 0u));
                            } else atomicAdd(&A.diff[x], half ? (ull)sz[j] : (ull)(-sz[j]));
                        }
                    }
                }
                TLC(2);
                __syncthreads();
                TLC(3);
            }
            // the tile's entries go to the difference array (other blocks may have added to the same entries)
            for (int x = threadIdx.x; x <= tk1 - tk0; x += kTlThreads) {
                const ull v = (((ull)s_pos_hi[x] << 32) | s_pos_lo[x]) - (((ull)s_neg_hi[x] << 32) | s_neg_lo[x]);
                if (v) atomicAdd(&A.diff[tk0 + x], v);
            }
            __syncthreads();
        }
        if (bad) raise_status(A.status, bad);
    }
    TLC(4);
    if (!grid_barrier(A.bar, (unsigned)G, gen)) { if (threadIdx.x == 0) raise_status(A.status, G10_DEV_TIMEOUT); return; }
    TLC(5);
    // ------------------------------------------------------------------ phase 2: both scans over this block's segment
    const int g = blockIdx.x;
    const int64_t seg = ((K + G - 1) / G + kTlChunk - 1) / kTlChunk * kTlChunk;
    const int64_t lo = (int64_t)g * seg < K ? (int64_t)g * seg : K, hi = lo + seg < K ? lo + seg : K;
    long long sum_c = 0, sum_p = 0;
    ull bad = 0;
    // A segment of one chunk (the usual case: up to kTlChunk kernels per block) is loaded once, each thread its
    // kTlScanItems consecutive kernels, and stays in registers for the scan; a longer one is summed here and read again.
    const bool single = hi - lo <= kTlChunk;
    long long rc[kTlScanItems], rd[kTlScanItems];
    if (single) {
        const int64_t base = lo + (int64_t)threadIdx.x * kTlScanItems;
#pragma unroll
        for (int j = 0; j < kTlScanItems; ++j) {
            const int64_t k = base + j;
            rc[j] = k < hi ? A.dur[k] : 0;
            rd[j] = k < hi ? (long long)__ldcg(&A.diff[k]) : 0;
        }
#pragma unroll
        for (int j = 0; j < kTlScanItems; ++j) {
            if (base + j < hi && (rc[j] < 1 || rc[j] >= ((long long)1 << 44))) { bad |= G10_DEV_BAD_DURATION; rc[j] = 1; }
            sum_c += rc[j]; sum_p += rd[j];
        }
    } else
    for (int64_t k0 = lo + threadIdx.x; k0 < hi; k0 += 4 * kTlThreads) {
        long long c[4], d[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t k = k0 + (int64_t)j * kTlThreads;
            c[j] = k < hi ? A.dur[k] : 1;
            d[j] = k < hi ? (long long)__ldcg(&A.diff[k]) : 0;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t k = k0 + (int64_t)j * kTlThreads;
            if (k < hi) {
                if (c[j] < 1 || c[j] >= ((long long)1 << 44)) { bad |= G10_DEV_BAD_DURATION; c[j] = 1; }
                sum_c += c[j]; sum_p += d[j];
            }
        }
    }
    if (bad) raise_status(A.status, bad);
    sum_c = warp_sum_i64(sum_c); sum_p = warp_sum_i64(sum_p);
    if (lane == 0) { s_w[0][warp] = sum_c; s_w[1][warp] = sum_p; }
    __syncthreads();
    long long unused;
    const long long tot_c = tl_warp_totals(s_w[0], lane, warp, &unused), tot_p = tl_warp_totals(s_w[1], lane, warp, &unused);
    if (threadIdx.x == 0) {
        asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(&A.words[2 * g]), "l"(tl_pack(tot_c)) : "memory");
        asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(&A.words[2 * g + 1]), "l"(tl_pack(tot_p)) : "memory");
    }
    // prefix of the segment: the sums of all segments before it
    long long pre_c = 0, pre_p = 0;
    for (int j = threadIdx.x; j < 2 * g; j += kTlThreads) {
        ull w;
        unsigned polls = 0;
        for (;;) {
            asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(w) : "l"(&A.words[j]) : "memory");
            if (w >> 62) break;
            if (++polls > kSpinLimit) { raise_status(A.status, G10_DEV_TIMEOUT); w = 0; break; }
            __nanosleep(64);
        }
        if (j & 1) pre_p += tl_unpack(w); else pre_c += tl_unpack(w);
    }
    pre_c = warp_sum_i64(pre_c); pre_p = warp_sum_i64(pre_p);
    __syncthreads();                                       // s_w has been read by every warp
    if (lane == 0) { s_w[0][warp] = pre_c; s_w[1][warp] = pre_p; }
    __syncthreads();
    long long carry_c = tl_warp_totals(s_w[0], lane, warp, &unused), carry_p = tl_warp_totals(s_w[1], lane, warp, &unused);
    long long mx = 0;
    int sl = -1;
    for (int64_t c0 = lo; c0 < hi; c0 += kTlChunk) {
        const int64_t base = c0 + (int64_t)threadIdx.x * kTlScanItems;
        long long c[kTlScanItems], d[kTlScanItems];
        long long tc = 0, tp = 0;
#pragma unroll
        for (int j = 0; j < kTlScanItems; ++j) {
            const int64_t k = base + j;
            if (single) { c[j] = rc[j]; d[j] = rd[j]; }
            else {
                c[j] = k < hi ? A.dur[k] : 0;
                d[j] = k < hi ? (long long)__ldcg(&A.diff[k]) : 0;
                if (k < hi && (c[j] < 1 || c[j] >= ((long long)1 << 44))) c[j] = 1;
            }
            tc += c[j]; tp += d[j];
        }
        const long long ic = warp_inclusive_scan_i64(tc, lane), ip = warp_inclusive_scan_i64(tp, lane);
        __syncthreads();                                   // s_w has been read by every warp
        if (lane == 31) { s_w[0][warp] = ic; s_w[1][warp] = ip; }
        __syncthreads();
        long long wc, wp;
        const long long ctot = tl_warp_totals(s_w[0], lane, warp, &wc), ptot = tl_warp_totals(s_w[1], lane, warp, &wp);
        long long run_c = carry_c + wc + ic - tc, run_p = carry_p + wp + ip - tp;
#pragma unroll
        for (int j = 0; j < kTlScanItems; ++j) {
            const int64_t k = base + j;
            if (k < hi) {
                A.start[k] = run_c;
                run_c += c[j];
                run_p += d[j];
                A.P[k] = run_p;
                if (sl < 0 || run_p > mx) { mx = run_p; sl = (int)k; }
            }
        }
        carry_c += ctot; carry_p += ptot;
    }
    if (hi == K && (lo < K || g == 0) && threadIdx.x == 0) {       // the block whose segment ends the trace (block 0 when K = 0)
        A.start[K] = carry_c;
        if (carry_c >= ((long long)1 << 44)) raise_status(A.status, G10_DEV_BAD_DURATION);
    }
    TLC(6);
#ifdef G10_TL_CLOCKS
    if (threadIdx.x == 0 && (blockIdx.x == 0 || blockIdx.x == 100 || blockIdx.x == 295)) printf("blk %d rounds %d ns: walk %llu atom %llu book %llu sync %llu flush+tail %llu barrier %llu phase2 %llu total %llu\n", blockIdx.x, nrounds, tacc[0], tacc[1], tacc[2], tacc[3], tacc[4], tacc[5], tacc[6], global_timer_ns() - tbeg);
#endif
    // block maximum (ties to the lowest slot), then the last block to finish reduces the per-block results
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const long long omx = __shfl_down_sync(0xffffffffu, mx, o);
        const int osl = __shfl_down_sync(0xffffffffu, sl, o);
        if (osl >= 0 && (sl < 0 || omx > mx || (omx == mx && osl < sl))) { mx = omx; sl = osl; }
    }
    __syncthreads();
    if (lane == 0) { s_w[0][warp] = mx; s_sl[warp] = sl; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kTlWarps; ++w)
            if (s_sl[w] >= 0 && (sl < 0 || s_w[0][w] > mx || (s_w[0][w] == mx && s_sl[w] < sl))) { mx = s_w[0][w]; sl = s_sl[w]; }
        A.blk_max[g] = mx;
        A.blk_slot[g] = sl;
        unsigned arrived;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(arrived) : "l"(A.done) : "memory");
        s_last = (arrived == (unsigned)G - 1u);
    }
    __syncthreads();
    if (s_last) {
        long long bm = 0;
        int bs = -1;
        for (int t = threadIdx.x; t < G; t += kTlThreads) {
            const long long m = __ldcg(&A.blk_max[t]);
            const int s2 = __ldcg(&A.blk_slot[t]);
            if (s2 >= 0 && (bs < 0 || m > bm || (m == bm && s2 < bs))) { bm = m; bs = s2; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const long long omx = __shfl_down_sync(0xffffffffu, bm, o);
            const int osl = __shfl_down_sync(0xffffffffu, bs, o);
            if (osl >= 0 && (bs < 0 || omx > bm || (omx == bm && osl < bs))) { bm = omx; bs = osl; }
        }
        __syncthreads();
        if (lane == 0) { s_w[0][warp] = bm; s_sl[warp] = bs; }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < kTlWarps; ++w)
                if (s_sl[w] >= 0 && (bs < 0 || s_w[0][w] > bm || (s_w[0][w] == bm && s_sl[w] < bs))) { bm = s_w[0][w]; bs = s_sl[w]; }
            *A.peak_bytes = bs < 0 ? 0 : bm;
            *A.peak_slot = bs;
        }
    }
}

// Number of blocks of the persistent grid: all of them must be resident at once (grid barrier).
static int timeline_blocks(int64_t K, int64_t E)
{
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_timeline, kTlThreads, 0) != cudaSuccess || per_sm < 1) return 0;
    if (per_sm > 2) per_sm = 2;
    int64_t g = (int64_t)sms * per_sm;
    int64_t by_work = (K + kTlChunk - 1) / kTlChunk;                    // no point in scan segments without a full chunk ...
    const int64_t by_events = (E + kTlRound - 1) / kTlRound;           // ... unless the events ask for more blocks
    if (by_events > by_work) by_work = by_events;
    if (g > by_work) g = by_work;
    if (g > kTlMaxBlocks) g = kTlMaxBlocks;
    return g < 1 ? 1 : (int)g;
}

cudaError_t launch_timeline(const DeviceTrace &t, const Workspace &w, int64_t *start, int64_t *pressure, int64_t *peak_bytes,
                            int32_t *peak_slot, cudaStream_t s)
{
    TlArgs A;
    A.K = t.K; A.N = t.N; A.E = t.E;
    A.kptr = t.kernel_ptr; A.kt = t.kernel_tensors; A.bytes = t.tensor_bytes; A.dur = t.kernel_ns; A.glob = t.tensor_global;
    A.pair = w.tl_pair; A.diff = (ull *)w.diff; A.start = start; A.P = pressure; A.peak_bytes = peak_bytes; A.peak_slot = peak_slot;
    A.words = w.tl_words; A.blk_max = w.tl_blk_max; A.blk_slot = w.tl_blk_slot; A.done = w.pressure_scan.done;
    A.bar = (GridBarrier *)w.barrier; A.status = w.status;
    const int G = timeline_blocks(t.K, t.E);
    if (G < 1) return cudaErrorLaunchFailure;
    // kernels per tile: about one round of events, evened out so that every block gets the same number of tiles
    int64_t tk = t.E > 0 ? ((int64_t)kTlRound * 9 / 10) * t.K / t.E : kTlMaxTileKernels;
    tk = tk < 32 ? 32 : (tk > kTlMaxTileKernels ? kTlMaxTileKernels : tk);
    if (t.K > 0) {
        const int64_t per_block = (t.K + tk * G - 1) / (tk * G);
        tk = (t.K + per_block * G - 1) / (per_block * G);
        tk = tk > kTlMaxTileKernels ? kTlMaxTileKernels : tk;
    }
    A.tile_kernels = (int)tk;
    A.vec_ok = (((uintptr_t)t.tensor_bytes & 15) == 0 && ((uintptr_t)t.tensor_global & 1) == 0) ? 1 : 0;
    {
        const int64_t work = (t.N > t.K + 1 ? t.N : t.K + 1);
        int64_t blocks = (work + 256 * 4 - 1) / (256 * 4);
        const int sms = current_sm_count();
        if (blocks > 8 * (int64_t)sms) blocks = 8 * (int64_t)sms;
        if (blocks < 1) blocks = 1;
        k_tl_init<<<(unsigned)blocks, 256, 0, s>>>(A);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    // cooperative launch (all blocks resident: grid barrier) with programmatic stream serialisation
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)G);
    cfg.blockDim = dim3(kTlThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, k_timeline, A);
    if (e == cudaErrorInvalidValue || e == cudaErrorNotSupported) {     // (a driver that does not combine the two attributes)
        (void)cudaGetLastError();
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, k_timeline, A);
    }
    return e;
}

}  // namespace g10

// Tensor vitality (Section 4.2: born / dead / inactive periods) in three kernels that keep the random
// accesses on chip.  Tensors are cut into buckets of `bt` consecutive ids (chosen so that a bucket holds a few
// thousand trace events and the buckets come to whole rounds of the last kernel's grid):
//   1. k_bk_hist     counts the events of every bucket (shared-memory histogram per block);
//   2. k_bk_scatter  partitions the events by bucket: each event becomes one 64-bit key
//                    (tensor id inside the bucket << 32 | kernel) written into its bucket's slice; the events are
//                    walked kernel by kernel, one lane per kernel, so no event has to look its kernel up;
//   3. k_bk_emit     takes one bucket at a time, entirely in shared memory: counts the events of each tensor,
//                    scans the counts, scatters the kernels into per-tensor segments, lets one thread sort and
//                    de-duplicate each (short) segment -- a tensor listed by more than 32 kernels is sorted by the
//                    whole block -- and counts the inactive periods (consecutive distinct uses at least two kernels
//                    apart); the offsets of a bucket in `uses` and in the period arrays are the sums of the totals
//                    of all earlier buckets, exchanged through tagged 64-bit words; then everything is written out
//                    in coalesced runs.
// Everything random happens in shared memory (atomics included); HBM sees the events twice, the keys once each
// way and the outputs once.  A bucket with more events than fit in shared memory (a tensor listed by a great many
// kernels) keeps its segments in global memory instead: slower, same result.
#include "g10_device.cuh"
#include "g10_internal.h"

namespace g10 {

constexpr int kBkThreads = 512;
constexpr int kBkItems = 8;
constexpr int kBkTile = kBkThreads * kBkItems;     // events per partition tile (4096)
constexpr int kBkCap = 10240;                      // events of a bucket kept in shared memory
constexpr int kBkWide = 64;                        // a kernel with more events is walked by its whole warp in the partition
constexpr int kBkHeavy = 32;                       // longer segments are sorted by the whole block

// A trace with more tensors than 4096 buckets of 4096 hold is taken in passes over the events, each for a run of
// consecutive tensor ids (t_begin, N of them): events of other tensors are skipped, tensor numbers inside a pass are
// relative to t_begin, and the totals of the earlier passes come in through `carry_in`.
struct BucketArgs {
    int64_t N, E, K;           // N: tensors of this pass
    int64_t t_begin, N_total;  // first tensor id of the pass; tensors of the trace
    int last_pass;
    const long long *carry_in; // [2] distinct uses and periods of all tensors before the pass (nullptr: none)
    long long *carry_out;      // [2] the same after the pass
    ull magic;                 // ceil(2^40 / bt): (x * magic) >> 40 == x / bt for every tensor number x of a pass (bk_bucket)
    int bt;                    // tensors per bucket
    int nb;                    // number of buckets
    int tile_kernels;          // kernels per partition tile (at most 32768)
    int tile_cap;              // events of a tile that go through shared memory in one round (a multiple of kBkThreads)
    unsigned *bucket_count;    // [nb] events per bucket
    unsigned *bucket_cursor;   // [nb] scatter cursors (start at zero)
    ull *pairs;                // [E] keys, bucket after bucket
    ull *words;                // [2 * nb] tagged totals of each bucket: distinct uses, periods
    int32_t *spill;            // [E] per-tensor segments of buckets too large for shared memory
    unsigned *ticket;
    int64_t *zero_diff, *zero_point;   // timeline wanted from the same call: difference array [K + 1] and point masses [K] that
                                       // the counting kernel of the first pass clears on its way (nullptr: nothing to clear)
    unsigned *done;            // blocks of the last kernel that have finished (starts at zero)
    int64_t *status_out;       // receives the status word when the last of them finishes the last pass (nullptr: nobody asked)
    ull *status;
};

// Bucket of tensor number x (inside a pass: 0 <= x < 2^24) for buckets of bt tensors, 64 <= bt <= 4096, without a division:
// with magic = ceil(2^40 / bt) the product x * magic / 2^40 exceeds x / bt by less than 2^-16, and x / bt is at least
// 1 / bt >= 2^-12 short of the next integer.
__device__ __forceinline__ int bk_bucket(int x, ull magic) { return (int)(((ull)(unsigned)x * magic) >> 40); }

// Block-wide exclusive scans over at most kBkThreads * 8 = 4096 entries, eight consecutive entries per thread.
// in[0..n) -> out[0..n), out[n] = total (in == out allowed).  NA = 1 or 2 arrays scanned together.
template <int NA>
__device__ __forceinline__ void bk_block_scan(const int *in0, int *out0, const int *in1, int *out1, int n, int *s_w /* [NA][kBkThreads/32 + 1] */)
{
    // The arrays start on 16-byte boundaries and are padded to a multiple of four entries (bk_pad), so a thread's
    // eight entries move as two 128-bit accesses (eight 32-bit ones at a stride of eight words would meet in the
    // same banks eight at a time).  Entries at or past n are read (they lie inside the padding or the next array)
    // but never used or written.
    constexpr int W = kBkThreads / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int base = threadIdx.x * 8;
    int v[NA][8], tot[NA];
#pragma unroll
    for (int a = 0; a < NA; ++a) {
        const int *in = a == 0 ? in0 : in1;
        int4 x = make_int4(0, 0, 0, 0), y = make_int4(0, 0, 0, 0);
        if (base < n) x = *reinterpret_cast<const int4 *>(in + base);
        if (base + 4 < n) y = *reinterpret_cast<const int4 *>(in + base + 4);
        v[a][0] = x.x; v[a][1] = x.y; v[a][2] = x.z; v[a][3] = x.w; v[a][4] = y.x; v[a][5] = y.y; v[a][6] = y.z; v[a][7] = y.w;
        tot[a] = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { if (base + j >= n) v[a][j] = 0; tot[a] += v[a][j]; }
    }
    int incl[NA];
#pragma unroll
    for (int a = 0; a < NA; ++a) {
        incl[a] = tot[a];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl[a], o); if (lane >= o) incl[a] += y; }
    }
    __syncthreads();                                      // all inputs read (in == out), scratch free
#pragma unroll
    for (int a = 0; a < NA; ++a) if (lane == 31) s_w[a * (W + 1) + warp] = incl[a];
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int a = 0; a < NA; ++a) {
            const int x = lane < W ? s_w[a * (W + 1) + lane] : 0;
            int xi = x;
#pragma unroll
            for (int o = 1; o < W; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, xi, o); if (lane >= o) xi += y; }
            if (lane < W) s_w[a * (W + 1) + lane] = xi - x;
            if (lane == W - 1) s_w[a * (W + 1) + W] = xi;
        }
    }
    __syncthreads();
#pragma unroll
    for (int a = 0; a < NA; ++a) {
        int *out = a == 0 ? out0 : out1;
        int run = s_w[a * (W + 1) + warp] + incl[a] - tot[a];
        int r[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) { r[j] = run; run += v[a][j]; }
        if (base + 8 <= n) {
            *reinterpret_cast<int4 *>(out + base) = make_int4(r[0], r[1], r[2], r[3]);
            *reinterpret_cast<int4 *>(out + base + 4) = make_int4(r[4], r[5], r[6], r[7]);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) if (base + j < n) out[base + j] = r[j];
        }
        if (threadIdx.x == 0) out[n] = s_w[a * (W + 1) + W];
    }
    __syncthreads();
}

// entries of a shared-memory array of n + 1 ints, padded so that the next array starts on a 16-byte boundary
__host__ __device__ inline int bk_pad(int n) { return (n + 1 + 3) & ~3; }

__device__ __forceinline__ void block_scan_counts(const unsigned *cnt, int n, int *out, int *s_w)
{
    bk_block_scan<1>((const int *)cnt, out, nullptr, nullptr, n, s_w);
}


// ---------------------------------------------------------------------------------------------
// 1. events per bucket
// ---------------------------------------------------------------------------------------------
// (kMulti: the trace is taken in several passes; with one pass the tensor ids are used as they are)
template <bool kMulti>
__global__ void __launch_bounds__(kBkThreads) k_bk_hist(BucketArgs B, const int64_t *__restrict__ kptr, const int32_t *__restrict__ kt)
{
    extern __shared__ unsigned s_hist[];
    for (int b = threadIdx.x; b < B.nb; b += kBkThreads) s_hist[b] = 0;
    if (B.zero_diff != nullptr)
        for (int64_t k = (int64_t)blockIdx.x * kBkThreads + threadIdx.x; k <= B.K; k += (int64_t)gridDim.x * kBkThreads) {
            B.zero_diff[k] = 0;
            if (k < B.K) B.zero_point[k] = 0;
        }
    __syncthreads();
    ull bad = 0;
    // the partition walks the events kernel by kernel: kernel_ptr has to be a monotone map onto [0, E]
    // (both walks are short chains of memory latencies: four steps of the first and two tiles of the second have their loads
    // in flight together)
    for (int64_t k0 = (int64_t)blockIdx.x * kBkThreads + threadIdx.x; k0 < B.K; k0 += 4 * (int64_t)gridDim.x * kBkThreads) {
        int64_t p0[4], p1[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int64_t k = k0 + q * (int64_t)gridDim.x * kBkThreads;
            p0[q] = k < B.K ? kptr[k] : 0; p1[q] = k < B.K ? kptr[k + 1] : 0;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int64_t k = k0 + q * (int64_t)gridDim.x * kBkThreads;
            if (k < B.K && (p0[q] > p1[q] || p0[q] < 0 || p1[q] > B.E || (k == 0 && p0[q] != 0) || (k == B.K - 1 && p1[q] != B.E)))
                bad |= G10_DEV_BAD_KERNEL_PTR;
        }
    }
    const int64_t tiles = (B.E + kBkTile - 1) / kBkTile;
    constexpr int kHistItems = 2 * kBkItems;
    for (int64_t tile = blockIdx.x; tile < tiles; tile += 2 * (int64_t)gridDim.x) {
        int32_t id[kHistItems];
#pragma unroll
        for (int j = 0; j < kHistItems; ++j) {
            const int64_t t2 = tile + (j / kBkItems) * (int64_t)gridDim.x;
            const int64_t e = t2 * kBkTile + (int64_t)(j % kBkItems) * kBkThreads + threadIdx.x;
            id[j] = (t2 < tiles && e < B.E) ? kt[e] : -2;
        }
#pragma unroll
        for (int j = 0; j < kHistItems; ++j) {
            if (id[j] == -2) continue;
            if (!kMulti) {
                if (id[j] < 0 || id[j] >= B.N) bad |= G10_DEV_BAD_TENSOR_ID;
                else atomicAdd(&s_hist[bk_bucket(id[j], B.magic)], 1u);
            } else if (id[j] < 0 || id[j] >= B.N_total) { if (B.t_begin == 0) bad |= G10_DEV_BAD_TENSOR_ID; }
            else {
                const int64_t rel = (int64_t)id[j] - B.t_begin;
                if (rel >= 0 && rel < B.N) atomicAdd(&s_hist[bk_bucket((int)rel, B.magic)], 1u);
            }
        }
    }
    if (bad) raise_status(B.status, bad);
    __syncthreads();
    for (int b = threadIdx.x; b < B.nb; b += kBkThreads)
        if (s_hist[b]) atomicAdd(&B.bucket_count[b], s_hist[b]);
    // (when this kernel was allowed to start beside its predecessor in the stream: its completion must imply that one's)
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------
// 2. partition the events by bucket
// ---------------------------------------------------------------------------------------------
// A tile is a run of consecutive kernels; its events [T0, T1) go through the block in rounds of at most B.tile_cap.
// Per round: (a) the kernels of the tile write their number (relative to the tile) over the positions of their
// events in shared memory -- a lane per kernel, a whole warp for a kernel with more than kBkWide events; stores
// only, nothing is loaded inside the walk; (b) the events are read coalesced, each looks its kernel up at its own
// position and takes its rank inside (round, bucket) from a shared-memory counter; ids and ranks stay in
// registers; (c) the counters are scanned and the round's room in every bucket it touches is reserved with one
// global atomic per bucket; (d) the keys are staged in bucket order in shared memory and (e) written out in
// coalesced runs.
constexpr int kPtMaxItems = 18;                     // events per thread and round, at most (tile_cap <= 18 * kBkThreads)

template <bool kMulti>
__global__ void __launch_bounds__(kBkThreads, 2) k_bk_scatter(BucketArgs B, const int64_t *__restrict__ kptr, const int32_t *__restrict__ kt)
{
    extern __shared__ __align__(16) int s_mem[];
    int *s_base = s_mem;                                   // [nb + 1] first key of each bucket
    int *s_cnt = s_base + bk_pad(B.nb);                      // [nb + 1] events of this round per bucket, then their scan
    int *s_off = s_cnt + bk_pad(B.nb);                      // [nb] global position of the round's first key of the bucket minus its slot
    ull *s_key = (ull *)(((uintptr_t)(s_off + B.nb) + 7) & ~(uintptr_t)7);   // [tile_cap] keys of the round in bucket order, the bucket in bits 48..59
    unsigned short *s_krel = (unsigned short *)(s_key + B.tile_cap);         // [tile_cap] kernel of every event of the round, relative to the tile
    __shared__ int s_warp[2 * (kBkThreads / 32 + 1)];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // (launched with programmatic stream serialisation: the blocks are placed while k_bk_hist drains and wait here
    // until it has finished and its counts are visible; no effect on an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (*(volatile ull *)B.status & G10_DEV_BAD_KERNEL_PTR) return;          // (found by k_bk_hist: nothing is partitioned)
    block_scan_counts(B.bucket_count, B.nb, s_base, s_warp);
    const int64_t TK = B.tile_kernels;
    const int64_t tiles = (B.K + TK - 1) / TK;
    const int cap = B.tile_cap;
#pragma unroll 1
    for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const int64_t tk0 = tile * TK, tk1 = tk0 + TK < B.K ? tk0 + TK : B.K;
        const int64_t T0 = kptr[tk0], T1 = kptr[tk1];
#pragma unroll 1
        for (int64_t eb = T0; eb < T1; eb += cap) {
            const int64_t ee = eb + cap < T1 ? eb + cap : T1;
            const int n_round = (int)(ee - eb);
            for (int b = threadIdx.x; b <= B.nb; b += kBkThreads) s_cnt[b] = 0;
            // (a) kernel of every event of the round
#pragma unroll 1
            for (int64_t k0 = tk0 + warp * 32; k0 < tk1; k0 += kBkThreads) {
                const int64_t k = k0 + lane;
                int64_t a = kptr[k < tk1 ? k : tk1], b = kptr[k + 1 < tk1 ? k + 1 : tk1];
                a = a > eb ? a : eb; a = a < ee ? a : ee;
                b = b > eb ? b : eb; b = b < ee ? b : ee;
                const bool wide = b - a > kBkWide;
                const unsigned short rel = (unsigned short)(k - tk0);
                if (!wide)
                    for (int p = (int)(a - eb), q = (int)(b - eb); p < q; ++p) s_krel[p] = rel;
                unsigned m = __ballot_sync(0xffffffffu, wide);
#pragma unroll 1
                while (m) {
                    const int src = __ffs(m) - 1;
                    m &= m - 1;
                    const int wa = (int)(__shfl_sync(0xffffffffu, a, src) - eb), wb = (int)(__shfl_sync(0xffffffffu, b, src) - eb);
                    const unsigned short wrel = (unsigned short)(k0 + src - tk0);
                    for (int p = wa + lane; p < wb; p += 32) s_krel[p] = wrel;
                }
            }
            __syncthreads();
            // (b) events, coalesced: bucket and rank inside (round, bucket)
            int32_t id[kPtMaxItems];
            int rank[kPtMaxItems];
#pragma unroll
            for (int j = 0; j < kPtMaxItems; ++j) {
                const int p = j * kBkThreads + threadIdx.x;
                id[j] = p < n_round ? kt[eb + p] : -1;
            }
#pragma unroll
            for (int j = 0; j < kPtMaxItems; ++j) {
                rank[j] = 0;
                if (!kMulti) {
                    if (id[j] >= 0 && id[j] < B.N) rank[j] = atomicAdd(&s_cnt[bk_bucket(id[j], B.magic)], 1);
                    else id[j] = -1;
                } else {
                    const int64_t rel = (int64_t)id[j] - B.t_begin;          // (the tensor's number inside the pass from here on)
                    if (id[j] >= 0 && rel >= 0 && rel < B.N) { id[j] = (int)rel; rank[j] = atomicAdd(&s_cnt[bk_bucket(id[j], B.magic)], 1); }
                    else id[j] = -1;
                }
            }
            __syncthreads();
            // (c) reserve this round's room in every bucket it touches, then turn the counts into offsets inside the round
            // (the global cursors answer while the block scans: their results stay in registers until after the scan)
            int cur[8];                                            // nb <= 4096 = 8 * kBkThreads
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int b = j * kBkThreads + threadIdx.x;
                cur[j] = (b < B.nb && s_cnt[b]) ? (int)atomicAdd(&B.bucket_cursor[b], (unsigned)s_cnt[b]) : 0;
            }
            block_scan_counts((const unsigned *)s_cnt, B.nb, s_cnt, s_warp);      // in place: s_cnt[b] = first slot of bucket b in the round
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int b = j * kBkThreads + threadIdx.x;
                if (b < B.nb) s_off[b] = cur[j] + s_base[b] - s_cnt[b];
            }
            // (d) keys in bucket order
#pragma unroll
            for (int j = 0; j < kPtMaxItems; ++j) {
                if (id[j] >= 0) {
                    const int p = j * kBkThreads + threadIdx.x;
                    const int b = bk_bucket(id[j], B.magic);
                    const unsigned k = (unsigned)(tk0 + s_krel[p]);
                    s_key[s_cnt[b] + rank[j]] = ((ull)(unsigned)b << 48) | ((ull)(unsigned)(id[j] - b * B.bt) << 32) | k;
                }
            }
            __syncthreads();
            // (e) out, coalesced
            const int n_valid = s_cnt[B.nb];
            for (int slot = threadIdx.x; slot < n_valid; slot += kBkThreads) {
                const ull key = s_key[slot];                       // bits 48..59: the bucket (staging only)
                const int64_t pos = (int64_t)s_off[(int)(key >> 48)] + slot;
                if (pos >= 0 && pos < B.E) B.pairs[pos] = key & 0x0000ffffffffffffull;
            }
            __syncthreads();
        }
    }
}

// ---------------------------------------------------------------------------------------------
// 3. one bucket at a time: count, scan, scatter, sort the short segments, count, emit
// ---------------------------------------------------------------------------------------------
__device__ void bk_bitonic_sort_i32(int32_t *a, int n)    // arbitrary n: the network only ever moves values up
{
    int n2 = 1;
    while (n2 < n) n2 <<= 1;
    for (int k = 2; k <= n2; k <<= 1) {
        for (int j = k >> 1, lj = 31 - __clz(k >> 1); j > 0; j >>= 1, --lj) {
            const bool mirror = (j == (k >> 1));
            for (int t = threadIdx.x; t < n2 / 2; t += blockDim.x) {
                const int blk = t >> lj, off = t & (j - 1);
                const int i = blk * 2 * j + off;
                const int p = mirror ? (blk * 2 * j + 2 * j - 1 - off) : (i + j);
                if (p < n) {
                    const int32_t x = a[i], y = a[p];
                    if (x > y) { a[i] = y; a[p] = x; }
                }
            }
            __syncthreads();
        }
    }
}

__device__ __forceinline__ ull bk_pack(long long v) { return (1ull << 62) | ((ull)v & ((1ull << 62) - 1)); }


// (kTimeline: the call also wants the pressure timeline; the kernel then books every tensor's size itself, see VitalityBuffers.
// Two blocks share an SM -- shared memory is sized for that -- so the kernel must stay within 64 registers.)
template <bool kTimeline>
__global__ void __launch_bounds__(kBkThreads, 2) k_bk_emit(BucketArgs B, VitalityBuffers out)
{
    extern __shared__ __align__(16) int s_mem[];
    int *s_base = s_mem;                       // [nb + 1] first key of each bucket
    int *t_off = s_base + bk_pad(B.nb);          // [bt + 1] raw events per tensor, then segment offsets
    int *t_d = t_off + bk_pad(B.bt);             // [bt + 1] scatter cursor, then distinct uses, then their offsets
    int *t_np = t_d + bk_pad(B.bt);             // [bt + 1] periods per tensor, then their offsets
    int32_t *s_ks = t_np + bk_pad(B.bt);         // [kBkCap] kernels, tensor segment after tensor segment
    unsigned short *s_mid = (unsigned short *)(s_ks + kBkCap);   // [bt] tensors of the bucket with three to kBkHeavy raw uses
    __shared__ int s_scan[2 * (kBkThreads / 32 + 1)];
    __shared__ int s_wa[kBkThreads / 32], s_wb[kBkThreads / 32];
    __shared__ long long s_pu[kBkThreads / 32], s_pp[kBkThreads / 32];
    __shared__ int s_bucket, s_nheavy, s_nmid, s_total, s_periods;
    __shared__ int s_heavy[64];
    __shared__ long long s_pre[2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.wait;" ::: "memory");             // (as in k_bk_scatter: the partition is complete)
    block_scan_counts(B.bucket_count, B.nb, s_base, s_scan);
    if (*(volatile ull *)B.status & G10_DEV_BAD_KERNEL_PTR) {      // nothing was partitioned: every tensor comes out unused
        for (int b = threadIdx.x; b <= B.nb; b += kBkThreads) s_base[b] = 0;
        __syncthreads();
    }
    long long tl_gsum = 0;                     // (timeline wanted too: bytes of the global tensors this thread met)
    bool tl_bad = false;
    for (;;) {
        __syncthreads();
        // (the number is taken when the work starts, not earlier: a later bucket waits for the totals of all earlier
        // ones, which are then certain to be under way)
        if (threadIdx.x == 0) { s_bucket = (int)atomicAdd(B.ticket, 1u); s_nheavy = 0; s_nmid = 0; }
        __syncthreads();
        const int b = s_bucket;
        if (b >= B.nb) break;
        const int n = s_base[b + 1] - s_base[b];
        const int64_t t0 = B.t_begin + (int64_t)b * B.bt;        // first tensor id of the bucket
        const int bt_eff = (int)((B.N - (int64_t)b * B.bt) < B.bt ? (B.N - (int64_t)b * B.bt) : B.bt);
        const ull *gk = B.pairs + s_base[b];
        int32_t *ks = n <= kBkCap ? s_ks : B.spill + s_base[b];
        for (int tl = threadIdx.x; tl <= bt_eff; tl += kBkThreads) { t_off[tl] = 0; t_d[tl] = 0; }
        __syncthreads();
        // ---- raw events per tensor, segment offsets, scatter.  The first keys of the bucket stay in registers between the
        // counting and the scatter; the rest is read again (from L2).  Eight per thread, about a usual bucket's share: with
        // twelve the kernel needs more than the 64 registers that let two blocks share an SM, and spills.
        constexpr int kRegKeys = 8;
        ull rk[kRegKeys];
#pragma unroll
        for (int q = 0; q < kRegKeys; ++q) {
            const int j = q * kBkThreads + threadIdx.x;
            rk[q] = j < n ? gk[j] : ~0ull;
        }
#pragma unroll
        for (int q = 0; q < kRegKeys; ++q)
            if (rk[q] != ~0ull) atomicAdd(&t_off[(int)(rk[q] >> 32)], 1);
        for (int j = kRegKeys * kBkThreads + threadIdx.x; j < n; j += kBkThreads) atomicAdd(&t_off[(int)(gk[j] >> 32)], 1);
        __syncthreads();
        bk_block_scan<1>(t_off, t_off, nullptr, nullptr, bt_eff, s_scan);
#pragma unroll
        for (int q = 0; q < kRegKeys; ++q)
            if (rk[q] != ~0ull) {
                const int tl = (int)(rk[q] >> 32);
                ks[t_off[tl] + atomicAdd(&t_d[tl], 1)] = (int32_t)(unsigned)rk[q];
            }
        for (int j = kRegKeys * kBkThreads + threadIdx.x; j < n; j += kBkThreads) {
            const ull key = gk[j];
            const int tl = (int)(key >> 32);
            ks[t_off[tl] + atomicAdd(&t_d[tl], 1)] = (int32_t)(unsigned)key;
        }
        __syncthreads();
        // ---- short segments: one or two raw uses are settled on the spot; three to kBkHeavy go to a list that the
        // threads then take one tensor each from (one thread sorts, removes repeats in place and counts the periods),
        // so that a warp is not held up eight times over by its longest segment
        int my_d = 0, my_p = 0;                 // this thread's share of the bucket totals
        for (int tl = threadIdx.x; tl < bt_eff; tl += kBkThreads) {
            const int o = t_off[tl], m = t_off[tl + 1] - o;
            int dd = 0, pp = 0;
            if (m == 1) dd = 1;
            else if (m == 2) {
                const int32_t x = ks[o], y = ks[o + 1];
                const int32_t lo = x < y ? x : y, hi = x < y ? y : x;
                if (lo == hi) dd = 1;
                else { ks[o] = lo; ks[o + 1] = hi; dd = 2; pp = hi - lo >= 2 ? 1 : 0; }
            } else if (m > kBkHeavy) {
                const int q = atomicAdd(&s_nheavy, 1);
                if (q < 64) s_heavy[q] = tl;
            } else if (m > 2) s_mid[atomicAdd(&s_nmid, 1)] = (unsigned short)tl;
            t_d[tl] = dd; t_np[tl] = pp;
            my_d += dd; my_p += pp;
        }
        __syncthreads();
        for (int q = threadIdx.x; q < s_nmid; q += kBkThreads) {
            const int tl = s_mid[q];
            const int m = t_off[tl + 1] - t_off[tl];
            int32_t *seg = ks + t_off[tl];
            int dd = 1, pp = 0;
            if (m <= 8) {
                // up to eight raw uses (nearly all of the list): loaded together, put in order by a 19-comparator network in
                // registers (the padding sorts to the end), then de-duplicated on the way back -- one round trip to shared
                // memory instead of an insertion sort's chain of them
                int32_t v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = j < m ? seg[j] : 0x7fffffff;
#define G10_CE(a, b) { const int32_t lo = min(v[a], v[b]), hi = max(v[a], v[b]); v[a] = lo; v[b] = hi; }
                G10_CE(0, 1) G10_CE(2, 3) G10_CE(4, 5) G10_CE(6, 7) G10_CE(0, 2) G10_CE(1, 3) G10_CE(4, 6) G10_CE(5, 7) G10_CE(1, 2) G10_CE(5, 6)
                G10_CE(0, 4) G10_CE(1, 5) G10_CE(2, 6) G10_CE(3, 7) G10_CE(2, 4) G10_CE(3, 5) G10_CE(1, 2) G10_CE(3, 4) G10_CE(5, 6)
#undef G10_CE
                int32_t prev = v[0];
                seg[0] = prev;
#pragma unroll
                for (int a = 1; a < 8; ++a) {
                    const int32_t x = v[a];
                    if (a < m && x != prev) { if (x - prev >= 2) ++pp; seg[dd++] = x; prev = x; }
                }
            } else {
                for (int a = 1; a < m; ++a) {
                    const int32_t x = seg[a];
                    int c = a - 1;
                    while (c >= 0 && seg[c] > x) { seg[c + 1] = seg[c]; --c; }
                    seg[c + 1] = x;
                }
                int32_t prev = seg[0];
                for (int a = 1; a < m; ++a) {
                    const int32_t x = seg[a];
                    if (x != prev) { if (x - prev >= 2) ++pp; seg[dd++] = x; prev = x; }
                }
            }
            t_d[tl] = dd; t_np[tl] = pp;
            my_d += dd; my_p += pp;
        }
        __syncthreads();
        // ---- long segments: the whole block sorts, compacts and counts, one tensor after the other
        const int nheavy = s_nheavy;
        for (int hq = 0; hq < (nheavy <= 64 ? nheavy : bt_eff); ++hq) {
            const int tl = nheavy <= 64 ? s_heavy[hq] : hq;
            const int m = t_off[tl + 1] - t_off[tl];
            if (m <= kBkHeavy) continue;                       // (only when the list overflowed: uniform test)
            int32_t *seg = ks + t_off[tl];
            bk_bitonic_sort_i32(seg, m);
            if (threadIdx.x == 0) { s_total = 0; s_periods = 0; }
            __syncthreads();
            for (int c0 = 0; c0 < m; c0 += kBkThreads) {
                const int t = c0 + threadIdx.x;
                int32_t x = 0, prev = 0;
                bool keep = false, per = false;
                if (t < m) {
                    x = seg[t];
                    if (t > 0) prev = seg[t - 1];
                    keep = (t == 0) || (x != prev);
                    per = keep && t > 0 && (x - prev >= 2);
                }
                const unsigned mk = __ballot_sync(0xffffffffu, keep), mp = __ballot_sync(0xffffffffu, per);
                if (lane == 0) s_wa[warp] = __popc(mk);
                __syncthreads();
                int off = s_total, chunk_total = 0;
                for (int w = 0; w < kBkThreads / 32; ++w) { if (w < warp) off += s_wa[w]; chunk_total += s_wa[w]; }
                off += __popc(mk & ((1u << lane) - 1u));
                __syncthreads();                               // every seg[t], seg[t-1] of this chunk has been read
                if (keep) seg[off] = x;                        // off <= t: never overtakes an unread element
                if (lane == 0 && mp) atomicAdd(&s_periods, __popc(mp));
                if (threadIdx.x == 0) s_total += chunk_total;
                __syncthreads();
            }
            if (threadIdx.x == 0) { t_d[tl] = s_total; t_np[tl] = s_periods; my_d += s_total; my_p += s_periods; }
            __syncthreads();
        }
        // ---- the bucket's totals go out first (later buckets wait for them), then the offsets of every tensor's
        // distinct uses and periods inside the bucket
        {
            const int wd = __reduce_add_sync(0xffffffffu, my_d), wp = __reduce_add_sync(0xffffffffu, my_p);
            if (lane == 0) { s_wa[warp] = wd; s_wb[warp] = wp; }
            __syncthreads();
            if (threadIdx.x == 0) {
                long long td = 0, tp = 0;
                for (int w = 0; w < kBkThreads / 32; ++w) { td += s_wa[w]; tp += s_wb[w]; }
                asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(&B.words[2 * b]), "l"(bk_pack(td)) : "memory");
                asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(&B.words[2 * b + 1]), "l"(bk_pack(tp)) : "memory");
            }
        }
        // ---- the pressure timeline is wanted from the same call: every tensor's size is booked where it is born and where it
        // dies (a tensor of one kernel in that slot's point mass; a global tensor in slot 0, summed per thread first).  First
        // and last use are known since the segments were sorted.  Done here, in a loop of their own behind the publication of
        // the totals, the reductions go out while the totals of the earlier buckets come in; inside the outputs loop their
        // requests to the L2 came on top of that loop's stores, and the loop's registers cost the kernel its keys in registers.
        if (kTimeline) {
            constexpr int kBook = 4;                           // (tensors of a thread whose loads are in flight together; 2, 3 and 8 were slower)
            for (int tl0 = threadIdx.x; tl0 < bt_eff; tl0 += kBook * kBkThreads) {
                long long bz4[kBook];
                int dd4[kBook], of4[kBook];
#pragma unroll
                for (int q = 0; q < kBook; ++q) {
                    const int tl = tl0 + q * kBkThreads;
                    bz4[q] = 1; dd4[q] = -1; of4[q] = 0;
                    if (tl < bt_eff) {
                        bz4[q] = out.tl_bytes[t0 + tl]; dd4[q] = t_d[tl]; of4[q] = t_off[tl];
                        if (out.tl_glob != nullptr && out.tl_glob[t0 + tl]) dd4[q] = -2 - dd4[q];   // (a global tensor: -2 - its uses)
                    }
                }
#pragma unroll
                for (int q = 0; q < kBook; ++q) {
                    if (dd4[q] == -1) continue;
                    const long long bsz = bz4[q];
                    if (bsz < 1 || bsz >= ((long long)1 << 40)) tl_bad = true;
                    if (dd4[q] < -2) tl_gsum += bsz;                   // (global and used)
                    else if (dd4[q] > 0) {
                        const int64_t f = ks[of4[q]], l = ks[of4[q] + dd4[q] - 1];
                        if (f == l) atomicAdd(&out.tl_point[f], (ull)bsz);
                        else {
                            atomicAdd(&out.tl_diff[f], (ull)bsz);
                            if (l + 1 < out.tl_K) atomicAdd(&out.tl_diff[l + 1], (ull)(-bsz));
                        }
                    }
                }
            }
            // (no barrier: the scan below writes t_d only behind a barrier of its own, which every thread reaches after this loop)
        }
        bk_block_scan<2>(t_d, t_d, t_np, t_np, bt_eff, s_scan);
        const long long D = t_d[bt_eff], PC = t_np[bt_eff];
        long long pu = 0, pq = 0;
        for (int j0 = threadIdx.x; j0 < 2 * b; j0 += 4 * kBkThreads) {
            ull w[4];
            bool pending = true;
            unsigned polls = 0;
            while (pending) {                                  // up to four words per thread in flight
                pending = false;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int j = j0 + q * kBkThreads;
                    w[q] = 1ull << 62;
                    if (j < 2 * b) asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(w[q]) : "l"(&B.words[j]) : "memory");
                    if (!(w[q] >> 62)) pending = true;
                }
                if (pending) {
                    if (++polls > kSpinLimit) { raise_status(B.status, G10_DEV_TIMEOUT); break; }
                    __nanosleep(100);
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int j = j0 + q * kBkThreads;
                if (j < 2 * b) { const long long v = (long long)(w[q] & ((1ull << 62) - 1)); if (j & 1) pq += v; else pu += v; }
            }
        }
        pu = warp_sum_i64(pu); pq = warp_sum_i64(pq);
        if (lane == 0) { s_pu[warp] = pu; s_pp[warp] = pq; }
        __syncthreads();
        if (threadIdx.x == 0) {
            long long a = 0, c2 = 0;
            for (int w = 0; w < kBkThreads / 32; ++w) { a += s_pu[w]; c2 += s_pp[w]; }
            if (B.carry_in != nullptr) { a += B.carry_in[0]; c2 += B.carry_in[1]; }    // (the tensors of the earlier passes)
            s_pre[0] = a; s_pre[1] = c2;
        }
        __syncthreads();
        const long long U = s_pre[0], PB = s_pre[1];
        ull bad = 0;
        if (U + D > out.uses_cap) bad |= G10_DEV_USES_OVERFLOW;
        if (PB + PC > out.periods_cap) bad |= G10_DEV_PERIODS_OVERFLOW;
        if (bad && threadIdx.x == 0) raise_status(B.status, bad);
        // ---- outputs.  Without repeats anywhere in the bucket (the usual case) the segments are already the use
        // lists, back to back in tensor order: they go out as one coalesced copy.
        const bool dense = D == n;
        if (dense)
            for (int j = threadIdx.x; j < n; j += kBkThreads)
                if (U + j < out.uses_cap) out.uses[U + j] = ks[j];
        // (two tensors of the thread at a time: their table entries, then their first and last use, are loaded together --
        // the loop is a chain of dependent shared-memory reads otherwise)
        for (int tl0 = threadIdx.x; tl0 < bt_eff; tl0 += 2 * kBkThreads) {
            int d04[2], dd4[2], of4[2], np4[2];
            int32_t f4[2], l4[2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int tl = tl0 + q * kBkThreads;
                d04[q] = 0; dd4[q] = -1; of4[q] = 0; np4[q] = 0;
                if (tl < bt_eff) { d04[q] = t_d[tl]; dd4[q] = t_d[tl + 1] - d04[q]; of4[q] = t_off[tl]; np4[q] = t_np[tl]; }
            }
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                f4[q] = -1; l4[q] = -1;
                if (dd4[q] > 0) { f4[q] = ks[of4[q]]; l4[q] = ks[of4[q] + dd4[q] - 1]; }
            }
#pragma unroll
            for (int q = 0; q < 2; ++q) {
            const int tl = tl0 + q * kBkThreads;
            if (dd4[q] < 0) continue;
            const int64_t t = t0 + tl;
            const int dd = dd4[q];
            const int32_t *seg = ks + of4[q];
            out.first_use[t] = f4[q];
            out.last_use[t] = l4[q];
            out.num_uses[t] = dd;
            out.use_ptr[t] = U + d04[q];
            out.period_ptr[t] = PB + np4[q];
            long long uo = U + d04[q], po = PB + np4[q];
            for (int a = dense ? 1 : 0; a < dd; ++a) {
                const int32_t x = seg[a];
                if (!dense && uo + a < out.uses_cap) out.uses[uo + a] = x;
                if (a > 0 && x - seg[a - 1] >= 2) {
                    if (po < out.periods_cap) {
                        out.period_tensor[po] = (int32_t)t;
                        out.period_prev_use[po] = seg[a - 1];
                        out.period_next_use[po] = x;
                    }
                    ++po;
                }
            }
            }
        }
        if (b == B.nb - 1 && threadIdx.x == 0) {
            B.carry_out[0] = U + D; B.carry_out[1] = PB + PC;
            if (B.last_pass) {
                out.use_ptr[B.N_total] = U + D; out.period_ptr[B.N_total] = PB + PC;
                out.counts[0] = U + D; out.counts[1] = PB + PC;
            }
        }
    }
    if (kTimeline) {
        if (tl_bad) raise_status(B.status, G10_DEV_BAD_BYTES);
        tl_gsum = warp_sum_i64(tl_gsum);
        if (lane == 0 && tl_gsum != 0) atomicAdd(&out.tl_diff[0], (ull)tl_gsum);
    }
    // the last block out, on the last pass, hands the status word over (every block's bits are in: acquire-release count)
    if (threadIdx.x == 0 && B.last_pass && B.status_out != nullptr) {
        unsigned arrived;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(arrived) : "l"(B.done) : "memory");
        if (arrived == gridDim.x - 1u) *B.status_out = (int64_t)*(volatile ull *)B.status;
    }
}

// Picks the bucket width for (a pass over) N tensors with about E events; false if that is outside what the bucket path handles.
static bool choose_buckets(int64_t N, int64_t E, int sms, int *bt, int *nb, ull *magic)
{
    if (N <= 0) return false;
    int64_t want = E > 0 ? (6000 * N) / E : 4096;        // tensors per bucket for about 4000-6000 events
    int s = 6;
    while (s < 12 && ((int64_t)1 << (s + 1)) <= want) ++s;
    while (s < 12 && ((N + ((int64_t)1 << s) - 1) >> s) > 4096) ++s;
    int64_t width = (int64_t)1 << s;
    int64_t buckets = (N + width - 1) / width;
    if (buckets > 4096) return false;
    // k_bk_emit takes the buckets one per block at a time with two blocks per SM, and what a bucket costs depends little on
    // its width: when there are more buckets than blocks, somewhat narrower buckets that come to whole rounds of the grid
    // finish sooner than a last round that a quarter of the blocks take part in.
    const int64_t G = 2 * (int64_t)sms;
    if (buckets > G) {
        const int64_t target = (buckets + G - 1) / G * G;
        const int64_t narrower = (N + target - 1) / target;
        if (target <= 4096 && narrower >= 64) { width = narrower; buckets = (N + width - 1) / width; }
    }
    *bt = (int)width; *nb = (int)buckets;
    *magic = (((ull)1 << 40) + (ull)width - 1) / (ull)width;
    return true;
}

constexpr int64_t kBkPassTensors = (int64_t)4096 * 4096;       // tensors one pass can take (4096 buckets of 4096)
constexpr int64_t kBkMaxPasses = 16;                           // (every pass reads all events: beyond this the plain formulation is used)

bool vitality_buckets_supported(int64_t N, int64_t E)
{
    (void)E;
    return N > 0 && N <= kBkMaxPasses * kBkPassTensors;
}

// One pass: the three kernels for tensors [B.t_begin, B.t_begin + B.N).
static cudaError_t launch_bucket_pass(BucketArgs B, const DeviceTrace &t, const VitalityBuffers &out, int sms, bool multi, bool pdl_first, cudaStream_t s)
{
    const int64_t tiles = (t.E + kBkTile - 1) / kBkTile;
    // the second and third kernel are launched with programmatic stream serialisation (they wait for their
    // predecessor themselves): launch and block placement overlap its tail
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kBkThreads);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (t.E > 0 && t.K > 0) {
        const int g = (int)(tiles < 2 * (int64_t)sms ? tiles : 2 * (int64_t)sms);
        {
            cudaLaunchConfig_t c1 = cfg;
            c1.gridDim = dim3((unsigned)g);
            c1.dynamicSmemBytes = sizeof(unsigned) * (size_t)B.nb;
            c1.numAttrs = pdl_first ? 1 : 0;
            const int64_t *kp = t.kernel_ptr;
            const int32_t *kt = t.kernel_tensors;
            const cudaError_t e1 = multi ? cudaLaunchKernelEx(&c1, k_bk_hist<true>, B, kp, kt) : cudaLaunchKernelEx(&c1, k_bk_hist<false>, B, kp, kt);
            if (e1 != cudaSuccess) return e1;
        }
        // Shared memory of the partition kernel: three bucket tables and ten bytes per staged event; two blocks per SM.
        const size_t tables = sizeof(int) * (size_t)(3 * bk_pad(B.nb)) + 8;
        int64_t cap = ((int64_t)(108 << 10) - (int64_t)tables) / 10 / kBkThreads * kBkThreads;
        cap = cap < kBkThreads ? kBkThreads : (cap > (int64_t)kPtMaxItems * kBkThreads ? (int64_t)kPtMaxItems * kBkThreads : cap);
        B.tile_cap = (int)cap;
        // Kernels per tile: as many as fill 92 % of a round on average (so that few tiles need a second round; a round has costs
        // of its own, so few full rounds beat many light ones: config 4 takes two rounds per block this way, not three),
        // then evened out so that every block of the grid gets the same number of tiles.
        const int g2max = 2 * sms;
        int64_t tk = (cap * 92 / 100) * t.K / t.E;
        tk = tk < 32 ? 32 : (tk > 32768 ? 32768 : tk);
        const int64_t per_block = (t.K + tk * g2max - 1) / (tk * g2max);
        tk = (t.K + per_block * g2max - 1) / (per_block * g2max);
        tk = (tk + 31) / 32 * 32;
        tk = tk > 32768 ? 32768 : tk;
        B.tile_kernels = (int)tk;
        const int64_t ktiles = (t.K + tk - 1) / tk;
        const int g2 = (int)(ktiles < g2max ? ktiles : g2max);
        const size_t sm2 = tables + (sizeof(ull) + sizeof(unsigned short)) * (size_t)cap;
        cudaError_t e = multi ? cudaFuncSetAttribute(k_bk_scatter<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm2)
                              : cudaFuncSetAttribute(k_bk_scatter<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm2);
        if (e != cudaSuccess) return e;
        cfg.gridDim = dim3((unsigned)g2);
        cfg.dynamicSmemBytes = sm2;
        const int64_t *kp = t.kernel_ptr;
        const int32_t *kt = t.kernel_tensors;
        e = multi ? cudaLaunchKernelEx(&cfg, k_bk_scatter<true>, B, kp, kt) : cudaLaunchKernelEx(&cfg, k_bk_scatter<false>, B, kp, kt);
        if (e != cudaSuccess) return e;
    }
    const size_t sm3 = sizeof(int) * (size_t)(bk_pad(B.nb) + 3 * bk_pad(B.bt) + kBkCap) + sizeof(unsigned short) * (size_t)B.bt;
    const bool fused = out.tl_diff != nullptr;
    cudaError_t e = fused ? cudaFuncSetAttribute(k_bk_emit<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm3)
                          : cudaFuncSetAttribute(k_bk_emit<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm3);
    if (e != cudaSuccess) return e;
    const int g3 = B.nb < 2 * sms ? B.nb : 2 * sms;
    cfg.gridDim = dim3((unsigned)g3);
    cfg.dynamicSmemBytes = sm3;
    e = fused ? cudaLaunchKernelEx(&cfg, k_bk_emit<true>, B, out) : cudaLaunchKernelEx(&cfg, k_bk_emit<false>, B, out);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

cudaError_t launch_vitality_buckets(const DeviceTrace &t, const Workspace &w, const VitalityBuffers &out, cudaStream_t s, int64_t *status_out, bool pdl_first)
{
    if (!vitality_buckets_supported(t.N, t.E)) return cudaErrorInvalidValue;
    const int sms = current_sm_count();
    if (sms <= 0) return cudaErrorInvalidDevice;
    const int64_t passes = (t.N + kBkPassTensors - 1) / kBkPassTensors;
    for (int64_t p = 0; p < passes; ++p) {
        BucketArgs B;
        B.t_begin = p * kBkPassTensors;
        B.N_total = t.N;
        B.N = t.N - B.t_begin < kBkPassTensors ? t.N - B.t_begin : kBkPassTensors;
        B.E = t.E; B.K = t.K; B.tile_kernels = kBkThreads; B.tile_cap = kBkThreads;
        B.last_pass = p == passes - 1 ? 1 : 0;
        B.carry_in = p > 0 ? w.bk_carry + 2 * ((p - 1) & 1) : nullptr;
        B.carry_out = w.bk_carry + 2 * (p & 1);
        // (bucket width from the pass's share of the events, taken as proportional to its share of the tensors)
        const int64_t e_share = passes > 1 ? (int64_t)((double)t.E * (double)B.N / (double)t.N) : t.E;
        if (!choose_buckets(B.N, e_share, sms, &B.bt, &B.nb, &B.magic)) return cudaErrorInvalidValue;
        B.bucket_count = w.bk_count; B.bucket_cursor = w.bk_cursor; B.pairs = w.bk_pairs; B.words = w.bk_words;
        B.ticket = w.emit_scan.ticket; B.done = w.emit_scan.done; B.status_out = status_out; B.status = w.status; B.spill = w.raw_uses;
        B.zero_diff = nullptr; B.zero_point = nullptr;
        if (p == 0 && out.tl_diff != nullptr && !out.tl_cleared) {
            if (t.E > 0 && t.K > 0) { B.zero_diff = (int64_t *)out.tl_diff; B.zero_point = (int64_t *)out.tl_point; }
            else {                                     // (no counting kernel will run: clear them here)
                cudaError_t e0;
                if ((e0 = cudaMemsetAsync(out.tl_diff, 0, sizeof(int64_t) * (size_t)(t.K + 1), s)) != cudaSuccess) return e0;
                if (t.K > 0 && (e0 = cudaMemsetAsync(out.tl_point, 0, sizeof(int64_t) * (size_t)t.K, s)) != cudaSuccess) return e0;
            }
        }
        if (p > 0) {                                   // what the call's opening memset cleared for the first pass
            cudaError_t e;
            if ((e = cudaMemsetAsync(w.bk_count, 0, sizeof(unsigned) * 4096, s)) != cudaSuccess) return e;
            if ((e = cudaMemsetAsync(w.bk_cursor, 0, sizeof(unsigned) * 4096, s)) != cudaSuccess) return e;
            if ((e = cudaMemsetAsync(w.bk_words, 0, sizeof(ull) * 2 * 4096, s)) != cudaSuccess) return e;
            if ((e = cudaMemsetAsync(w.emit_scan.ticket, 0, sizeof(unsigned), s)) != cudaSuccess) return e;
        }
        const cudaError_t e = launch_bucket_pass(B, t, out, sms, passes > 1, pdl_first && p == 0, s);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace g10

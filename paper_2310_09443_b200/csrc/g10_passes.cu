// The HBM-bound passes: slot clock (Section 4.2: kernel times measure the inactive periods), tensor
// vitality (Section 4.2: born / dead / inactive periods), memory-pressure timeline (Section 4.3) and
// candidate geometry (Algorithm 1's t = size / BW; Section 4.4's latest safe prefetch time).
#include <climits>

#include "g10_device.cuh"
#include "g10_internal.h"

namespace g10 {

// =============================================================================================
// Segmented single-kernel scan for the two timeline-sized scans (slot clock, pressure).  A grid of a few
// hundred blocks -- all resident at once, launched in one wave -- gives every block one contiguous
// segment.  Pass 1 sums the segment and publishes the sum in one 64-bit word (2 state bits + 62 value
// bits, so no fence is needed); every block then adds up the words of ALL its predecessors (a few
// hundred loads spread over the block, no dependency chain between blocks) and pass 2 rescans the
// segment, now L2-resident, with that prefix.  Segment numbers come from a ticket, so a predecessor
// has always started.
// =============================================================================================
constexpr int kSegThreads = 512;
constexpr int kSegWarps = kSegThreads / 32;
constexpr int kSegItems = 8;
constexpr int kSegChunk = kSegThreads * kSegItems;
constexpr int kSegMaxBlocks = 512;
// Every block's word sits in a 128-byte line of its own: a few hundred blocks each read all their predecessors' words at the
// same moment, and words packed into a few lines would all be served by the same one or two L2 slices, one after the other.
constexpr int kSegWordStride = 16;

__device__ __forceinline__ ull seg_pack(long long v) { return (1ull << 62) | ((ull)v & ((1ull << 62) - 1)); }
__device__ __forceinline__ long long seg_unpack(ull w) { return (long long)(w << 2) >> 2; }     // sign-extend 62 bits

// Sum of one value per warp (s_w[kSegWarps], written by the lanes 0 before a barrier): every warp adds them up
// for itself with shuffles.  Also returns the sum over the warps before this one.
__device__ __forceinline__ long long seg_warp_totals(const long long *s_w, int lane, int warp, long long *before)
{
    const long long x = lane < kSegWarps ? s_w[lane] : 0;
    long long incl = x;
#pragma unroll
    for (int o = 1; o < kSegWarps; o <<= 1) {
        const long long y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    *before = __shfl_sync(0xffffffffu, incl - x, warp);
    return __shfl_sync(0xffffffffu, incl, kSegWarps - 1);
}

// kind 0: exclusive scan of kernel_ns into start[0..K] with validation of kernel_ns and kernel_ptr
// kind 1: inclusive scan of the difference array into the pressure, plus peak and lowest peak slot; `kptr`, if not null, holds
//         for every slot the bytes of the tensors that are alive in that slot alone (added to the scan's result, not carried on)
template <int kind>
__global__ void __launch_bounds__(kSegThreads, 2) k_seg_scan(int64_t n, int64_t E, const int64_t *__restrict__ in, const int64_t *__restrict__ kptr,
                                                             int64_t *__restrict__ out, unsigned *ticket, unsigned *done, ull *words,
                                                             int64_t *blk_max, int32_t *blk_slot, int64_t *peak_bytes, int32_t *peak_slot, ull *status,
                                                             int64_t *status_out, int64_t *zero_a = nullptr, int64_t *zero_b = nullptr)
{
    __shared__ long long s_w[kSegWarps];
    __shared__ int s_sl[kSegWarps];
    __shared__ bool s_last;
    const int G = gridDim.x;
    // Nothing later in a call reads the slot clock, so a kernel launched behind this one with programmatic stream
    // serialisation may start as soon as every block of this grid is running (no effect on ordinary launches).
    if (kind == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // (the segment number comes from a counter that the call's opening memset cleared, before any kernel: it can be taken
    // while the predecessor still runs)
    const int g = next_tile(ticket);
    if (kind != 0) asm volatile("griddepcontrol.wait;" ::: "memory");   // (the difference array is complete; see k_diff_scatter)
    // (kind 0, when the same call goes on to the pressure timeline: this kernel, the lighter of the two that open the call
    // side by side, clears the difference array [n + 1] and the point masses [n] on its way)
    if (kind == 0 && zero_a != nullptr)
        for (int64_t k = (int64_t)blockIdx.x * kSegThreads + threadIdx.x; k <= n; k += (int64_t)G * kSegThreads) {
            zero_a[k] = 0;
            if (k < n) zero_b[k] = 0;
        }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t seg = ((n + G - 1) / G + kSegChunk - 1) / kSegChunk * kSegChunk;
    const int64_t lo = (int64_t)g * seg, hi = lo + seg < n ? lo + seg : n;
    // ---- pass 1: segment sum
    long long sum = 0;
    ull bad = 0;
    for (int64_t k0 = lo + threadIdx.x; k0 < hi; k0 += 4 * kSegThreads) {
        long long v[4], p0[4], p1[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {                      // all loads of the batch in flight together
            const int64_t k = k0 + (int64_t)j * kSegThreads;
            v[j] = k < hi ? in[k] : (kind == 0 ? 1 : 0);
            if (kind == 0 && kptr != nullptr) { p0[j] = k < hi ? kptr[k] : 0; p1[j] = k < hi ? kptr[k + 1] : 0; }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t k = k0 + (int64_t)j * kSegThreads;
            if (k < hi) {
                if (kind == 0) {
                    if (v[j] < 1 || v[j] >= ((long long)1 << 44)) { bad |= G10_DEV_BAD_DURATION; v[j] = 1; }
                    if (kptr != nullptr && (p0[j] > p1[j] || p0[j] < 0 || p1[j] > E || (k == 0 && p0[j] != 0) || (k == n - 1 && p1[j] != E)))
                        bad |= G10_DEV_BAD_KERNEL_PTR;
                }
                sum += v[j];
            }
        }
    }
    if (bad) raise_status(status, bad);
    sum = warp_sum_i64(sum);
    if (lane == 0) s_w[warp] = sum;
    __syncthreads();
    long long unused;
    const long long seg_total = seg_warp_totals(s_w, lane, warp, &unused);
    if (threadIdx.x == 0)
        asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(&words[(size_t)g * kSegWordStride]), "l"(seg_pack(seg_total)) : "memory");
    // ---- prefix of the segment: all predecessors' sums
    long long pre = 0;
    for (int j = threadIdx.x; j < g; j += kSegThreads) {
        ull w;
        unsigned polls = 0;
        for (;;) {
            asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(w) : "l"(&words[(size_t)j * kSegWordStride]) : "memory");
            if (w >> 62) break;
            if (++polls > kSpinLimit) { raise_status(status, G10_DEV_TIMEOUT); w = 0; break; }
            __nanosleep(64);
        }
        pre += seg_unpack(w);
    }
    pre = warp_sum_i64(pre);
    __syncthreads();                                       // s_w has been read by every warp
    if (lane == 0) s_w[warp] = pre;
    __syncthreads();
    long long carry = seg_warp_totals(s_w, lane, warp, &unused);
    // ---- pass 2: scan the segment chunk by chunk.  A warp takes 32 * kSegItems consecutive elements as kSegItems rows of 32,
    // lane l the l-th of each row: every load and store of a warp is one contiguous 256-byte run (a thread with kSegItems
    // consecutive elements of its own would touch each 32-byte sector four times, and the stores reach the L2 one by one).
    long long mx = 0;
    int sl = -1;
    for (int64_t c0 = lo; c0 < hi; c0 += kSegChunk) {
        const int64_t base = c0 + (int64_t)warp * (32 * kSegItems) + lane;
        long long v[kSegItems], inc[kSegItems], pt[kSegItems];
#pragma unroll
        for (int j = 0; j < kSegItems; ++j) {
            const int64_t k = base + j * 32;
            v[j] = k < hi ? in[k] : 0;
            if (kind == 0 && k < hi && (v[j] < 1 || v[j] >= ((long long)1 << 44))) v[j] = 1;
            pt[j] = (kind == 1 && kptr != nullptr && k < hi) ? kptr[k] : 0;   // (kind 1: kptr = bytes alive in slot k only, or null)
        }
        long long rows = 0;                                // the rows before row j, then the warp's total
#pragma unroll
        for (int j = 0; j < kSegItems; ++j) {
            inc[j] = warp_inclusive_scan_i64(v[j], lane) + rows;
            rows = __shfl_sync(0xffffffffu, inc[j], 31);
        }
        __syncthreads();                                   // s_w has been read by every warp
        if (lane == 0) s_w[warp] = rows;
        __syncthreads();
        long long wpre;
        const long long ctot = seg_warp_totals(s_w, lane, warp, &wpre);
        const long long before = carry + wpre;
#pragma unroll
        for (int j = 0; j < kSegItems; ++j) {
            const int64_t k = base + j * 32;
            if (k < hi) {
                if (kind == 0) out[k] = before + inc[j] - v[j];
                else {
                    const long long p = before + inc[j] + pt[j];
                    out[k] = p;
                    if (sl < 0 || p > mx) { mx = p; sl = (int)k; }
                }
            }
        }
        carry += ctot;
    }
    if constexpr (kind == 0) {
        // after its own segment the last block's carry is the sum of everything
        if (g == G - 1 && threadIdx.x == 0) {
            out[n] = carry;
            if (carry >= ((long long)1 << 44)) raise_status(status, G10_DEV_BAD_DURATION);
        }
    } else {
    // ---- kind 1: block maximum (ties to the lowest slot), then the last block reduces the per-block results
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const long long omx = __shfl_down_sync(0xffffffffu, mx, o);
        const int osl = __shfl_down_sync(0xffffffffu, sl, o);
        if (osl >= 0 && (sl < 0 || omx > mx || (omx == mx && osl < sl))) { mx = omx; sl = osl; }
    }
    __syncthreads();
    if (lane == 0) { s_w[warp] = mx; s_sl[warp] = sl; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kSegWarps; ++w)
            if (s_sl[w] >= 0 && (sl < 0 || s_w[w] > mx || (s_w[w] == mx && s_sl[w] < sl))) { mx = s_w[w]; sl = s_sl[w]; }
        blk_max[g] = mx;
        blk_slot[g] = sl;
        // (acquire-release add: publishes this block's result; the last block to arrive has acquired everyone's)
        unsigned arrived;
        asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(arrived) : "l"(done) : "memory");
        s_last = (arrived == (unsigned)G - 1u);
    }
    __syncthreads();
    if (s_last) {
        long long bm = 0;
        int bs = -1;
        for (int t = threadIdx.x; t < G; t += kSegThreads) {
            const long long m = __ldcg(&blk_max[t]);
            const int s2 = __ldcg(&blk_slot[t]);
            if (s2 >= 0 && (bs < 0 || m > bm || (m == bm && s2 < bs))) { bm = m; bs = s2; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const long long omx = __shfl_down_sync(0xffffffffu, bm, o);
            const int osl = __shfl_down_sync(0xffffffffu, bs, o);
            if (osl >= 0 && (bs < 0 || omx > bm || (omx == bm && osl < bs))) { bm = omx; bs = osl; }
        }
        __syncthreads();
        if (lane == 0) { s_w[warp] = bm; s_sl[warp] = bs; }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < kSegWarps; ++w)
                if (s_sl[w] >= 0 && (bs < 0 || s_w[w] > bm || (s_w[w] == bm && s_sl[w] < bs))) { bm = s_w[w]; bs = s_sl[w]; }
            *peak_bytes = bs < 0 ? 0 : bm;
            *peak_slot = bs;
            // (kind 1, the last kernel of a timeline call: every block of this grid has arrived, every earlier kernel of the
            // call has completed, so the status word is final)
            if (status_out != nullptr) *status_out = (int64_t)*(volatile ull *)status;
        }
    }
    }
}

static int seg_scan_blocks(int64_t n)
{
    const int sms = current_sm_count();
    if (sms <= 0) return 1;
    int64_t g = 2 * (int64_t)sms;
    const int64_t by_work = (n + kSegChunk - 1) / kSegChunk;        // no point in blocks without a full chunk
    if (g > by_work) g = by_work;
    if (g > kSegMaxBlocks) g = kSegMaxBlocks;
    return g < 1 ? 1 : (int)g;
}

cudaError_t launch_slot_clock(const DeviceTrace &t, const Workspace &w, int64_t *start, cudaStream_t s, bool check_kernel_ptr, int64_t *zero_diff,
                              int64_t *zero_point)
{
    const int G = seg_scan_blocks(t.K);
    // (check_kernel_ptr false: another kernel of the same call makes the same check of kernel_ptr; this one then reads a third)
    k_seg_scan<0><<<G, kSegThreads, 0, s>>>(t.K, t.E, t.kernel_ns, check_kernel_ptr ? t.kernel_ptr : nullptr, start, w.clock_scan.ticket, w.clock_scan.done,
                                          w.seg_words, nullptr, nullptr, nullptr, nullptr, w.status, nullptr, zero_diff, zero_point); count_launch();
    return cudaGetLastError();
}

// =============================================================================================
// Event passes.  An event is one (kernel, tensor) entry of the CSR.  In the plain vitality kernels a
// block takes 2048 consecutive events and finds the kernel of an event by binary search in kernel_ptr,
// bracketed once per block; the first / last pass of the timeline call walks the events kernel by kernel.
// =============================================================================================
constexpr int kEvThreads = 256;
constexpr int kEvItems = 8;
constexpr int kEvTile = kEvThreads * kEvItems;

// last k in [lo, hi] with kptr[k] <= e  (kptr nondecreasing; lo is known to satisfy it)
__device__ __forceinline__ int kernel_of_event(const int64_t *kptr, int lo, int hi, int64_t e)
{
    while (lo < hi) {
        const int mid = lo + (hi - lo + 1) / 2;
        if (kptr[mid] <= e) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// raw use count per tensor (a tensor listed twice by one kernel counts twice here; collapsed later)
__global__ void __launch_bounds__(kEvThreads) k_count_events(int64_t E, int64_t N, const int32_t *__restrict__ kt,
                                                             int32_t *__restrict__ cnt, ull *status)
{
    const int64_t base = (int64_t)blockIdx.x * kEvTile;
    ull bad = 0;
#pragma unroll
    for (int j = 0; j < kEvItems; ++j) {
        const int64_t e = base + (int64_t)j * kEvThreads + threadIdx.x;
        if (e < E) {
            const int32_t i = kt[e];
            if (i < 0 || i >= N) bad = G10_DEV_BAD_TENSOR_ID;
            else atomicAdd(&cnt[i], 1);
        }
    }
    if (bad) raise_status(status, bad);
}

// raw_ptr = exclusive scan of the raw counts; tensors with more than kHeavyThreshold raw uses are
// queued for the block-wide sort.
__global__ void __launch_bounds__(kScanThreads) k_scan_counts(int64_t N, const int32_t *__restrict__ cnt, int32_t *__restrict__ raw_ptr,
                                                              int32_t *__restrict__ heavy_list, unsigned *heavy_count,
                                                              TileState<1> st, int tiles, ull *status)
{
    const int tile = next_tile(st.ticket);
    if (tile >= tiles) return;
    const int64_t base = (int64_t)tile * kScanTile + (int64_t)threadIdx.x * kScanItems;
    int v[kScanItems];
    Sums<1> mine;
    mine.v[0] = 0;
#pragma unroll
    for (int j = 0; j < kScanItems; ++j) {
        const int64_t i = base + j;
        v[j] = i < N ? cnt[i] : 0;
        mine.v[0] += v[j];
        if (v[j] > kHeavyThreshold) heavy_list[atomicAdd(heavy_count, 1u)] = (int32_t)i;
    }
    Sums<1> total;
    Sums<1> ex = block_exclusive_with_lookback<1>(st, tile, mine, status, &total);
    long long run = ex.v[0];
#pragma unroll
    for (int j = 0; j < kScanItems; ++j) {
        const int64_t i = base + j;
        if (i < N) raw_ptr[i] = (int32_t)run;
        run += v[j];
    }
    if (tile == tiles - 1 && threadIdx.x == 0) raw_ptr[N] = (int32_t)total.v[0];
}

// scatter every event's kernel index into its tensor's segment (order inside a segment is arbitrary)
__global__ void __launch_bounds__(kEvThreads) k_scatter_events(int64_t E, int64_t N, int64_t K, const int64_t *__restrict__ kptr,
                                                               const int32_t *__restrict__ kt, const int32_t *__restrict__ raw_ptr,
                                                               int32_t *__restrict__ cursor, int32_t *__restrict__ raw_uses)
{
    __shared__ int s_lo, s_hi;
    const int64_t base = (int64_t)blockIdx.x * kEvTile;
    if (threadIdx.x == 0) {
        const int64_t last = (base + kEvTile <= E ? base + kEvTile : E) - 1;
        s_lo = kernel_of_event(kptr, 0, (int)K - 1, base);
        s_hi = kernel_of_event(kptr, s_lo, (int)K - 1, last);
    }
    __syncthreads();
    const int lo = s_lo, hi = s_hi;
#pragma unroll
    for (int j = 0; j < kEvItems; ++j) {
        const int64_t e = base + (int64_t)j * kEvThreads + threadIdx.x;
        if (e < E) {
            const int32_t i = kt[e];
            if (i >= 0 && i < N) {
                const int k = kernel_of_event(kptr, lo, hi, e);
                const int old = atomicSub(&cursor[i], 1);          // counts back down to zero
                const int64_t pos = (int64_t)raw_ptr[i] + old - 1;
                if (old >= 1 && pos < E) raw_uses[pos] = k;
            }
        }
    }
}

// first / last use by atomic maxima (the timeline call alone does not need the sorted use lists); the results stay
// encoded (see below) and are decoded by the difference-array pass.
// One thread per kernel, a warp per 32 consecutive kernels: the warp walks the events of its kernels 32 at a time
// and finds the kernel of an event by a search over the lanes' kernel_ptr values (five shuffles), so nothing is
// searched in memory.  The kernel may run beside the pass that validates kernel_ptr, so it bounds its own work:
// a block books the events between its first and last kernel_ptr entry against a call-wide budget of E events
// (a valid kernel_ptr hands every event to exactly one block) and its warps stay inside that range.
constexpr int kFlThreads = 256;
__global__ void __launch_bounds__(kFlThreads) k_first_last_events(int64_t E, int64_t N, int64_t K, const int64_t *__restrict__ kptr,
                                                                  const int32_t *__restrict__ kt, int32_t *__restrict__ first_enc,
                                                                  int32_t *__restrict__ last_enc, ull *budget, ull *status)
{
    // both arrays start at zero: first_enc holds max(K - k) (0 = unused), last_enc holds max(k + 1)
    __shared__ int64_t s_span[2];
    const int lane = threadIdx.x & 31;
    const int64_t kb0 = (int64_t)blockIdx.x * kFlThreads;
    if (threadIdx.x == 0) {
        const int64_t kb1 = kb0 + kFlThreads < K ? kb0 + kFlThreads : K;
        int64_t b0 = kptr[kb0], b1 = kptr[kb1];
        b0 = b0 < 0 ? 0 : (b0 > E ? E : b0);
        b1 = b1 < 0 ? 0 : (b1 > E ? E : b1);
        if (b1 < b0) b1 = b0;
        if (b1 > b0 && atomicAdd(budget, (ull)(b1 - b0)) + (ull)(b1 - b0) > (ull)E) {
            raise_status(status, G10_DEV_BAD_KERNEL_PTR);
            b1 = b0;
        }
        s_span[0] = b0; s_span[1] = b1;
    }
    __syncthreads();
    const int64_t b0 = s_span[0], b1 = s_span[1];
    const int64_t k = kb0 + threadIdx.x, k0 = k - lane;
    if (k0 >= K || b1 == b0) return;
    int64_t mine = kptr[k < K ? k : K];                          // lanes past the last kernel hold kernel_ptr[K]
    int64_t span1 = kptr[k0 + 32 < K ? k0 + 32 : K];
    mine = mine < b0 ? b0 : (mine > b1 ? b1 : mine);
    span1 = span1 < b0 ? b0 : (span1 > b1 ? b1 : span1);
    const int64_t span0 = __shfl_sync(0xffffffffu, mine, 0);
    ull bad = 0;
#pragma unroll 1
    for (int64_t base = span0; base < span1; base += 32) {
        const int64_t e = base + lane;
        int lo = 0;                                              // last lane whose kernel starts at or before e
#pragma unroll
        for (int st = 16; st > 0; st >>= 1) {
            const int64_t p = __shfl_sync(0xffffffffu, mine, (lo + st) & 31);
            if (p <= e) lo += st;
        }
        if (e < span1) {
            const int32_t i = kt[e];
            if (i < 0 || i >= N) bad = G10_DEV_BAD_TENSOR_ID;
            else {
                const int kq = (int)(k0 + lo);
                atomicMax(&first_enc[i], (int)K - kq);
                atomicMax(&last_enc[i], kq + 1);
            }
        }
    }
    if (bad) raise_status(status, bad);
}

// The same pass for the timeline call, on an interleaved array pair[2 i] = max(K - k), pair[2 i + 1] = max(k + 1): lanes l and
// l + 16 of a warp share an event, one raises the tensor's first word, the other its last word.  Both words lie in one
// 32-byte sector, so the two reductions reach the L2 as one request; the L2 serves such scattered requests at a fixed
// rate per sector whatever they carry (about 170 G/s on this part), which is what bounds this pass.
__global__ void __launch_bounds__(kFlThreads) k_first_last_pairs(int64_t E, int64_t N, int64_t K, const int64_t *__restrict__ kptr,
                                                                 const int32_t *__restrict__ kt, int32_t *__restrict__ pair, ull *budget, ull *status,
                                                                 int64_t *zero_diff, int64_t *zero_point)
{
    __shared__ int64_t s_span[2];
    const int lane = threadIdx.x & 31, half = lane >> 4, l16 = lane & 15;
    const int64_t kb0 = (int64_t)blockIdx.x * kFlThreads;
    // the difference array [K + 1] and the point masses [K], which the NEXT kernel adds into, are cleared here (the grid has
    // a thread per kernel): 16 bytes per thread instead of a third of the call's opening memset
    if (zero_diff != nullptr) {
        const int64_t z = kb0 + threadIdx.x;
        if (z < K) { zero_diff[z] = 0; zero_point[z] = 0; }
        if (z == 0) zero_diff[K] = 0;
    }
    if (threadIdx.x == 0) {
        const int64_t kb1 = kb0 + kFlThreads < K ? kb0 + kFlThreads : K;
        int64_t b0 = kptr[kb0], b1 = kptr[kb1];
        b0 = b0 < 0 ? 0 : (b0 > E ? E : b0);
        b1 = b1 < 0 ? 0 : (b1 > E ? E : b1);
        if (b1 < b0) b1 = b0;
        if (b1 > b0 && atomicAdd(budget, (ull)(b1 - b0)) + (ull)(b1 - b0) > (ull)E) {
            raise_status(status, G10_DEV_BAD_KERNEL_PTR);
            b1 = b0;
        }
        s_span[0] = b0; s_span[1] = b1;
    }
    __syncthreads();
    const int64_t b0 = s_span[0], b1 = s_span[1];
    const int64_t k = kb0 + threadIdx.x, k0 = k - lane;
    const bool idle = k0 >= K || b1 == b0;                       // (uniform in the warp)
    int64_t mine = idle ? 0 : kptr[k < K ? k : K];               // lanes past the last kernel hold kernel_ptr[K]
    int64_t span1 = idle ? 0 : kptr[k0 + 32 < K ? k0 + 32 : K];
    mine = mine < b0 ? b0 : (mine > b1 ? b1 : mine);
    span1 = span1 < b0 ? b0 : (span1 > b1 ? b1 : span1);
    const int64_t span0 = __shfl_sync(0xffffffffu, mine, 0);
    if (idle) span1 = span0;
    ull bad = 0;
#pragma unroll 1
    for (int64_t base = span0; base < span1; base += 32) {       // two rows of sixteen events per step: both rows' loads in flight
        int32_t id[2];
        int kq[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int64_t e = base + 16 * r + l16;
            int lo = 0;                                          // last lane whose kernel starts at or before e
#pragma unroll
            for (int st = 16; st > 0; st >>= 1) {
                const int64_t p = __shfl_sync(0xffffffffu, mine, (lo + st) & 31);
                if (p <= e) lo += st;
            }
            kq[r] = (int)(k0 + lo);
            id[r] = e < span1 ? kt[e] : INT32_MIN;
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            if (id[r] == INT32_MIN) continue;
            if (id[r] < 0 || id[r] >= N) bad = G10_DEV_BAD_TENSOR_ID;
            else atomicMax(&pair[2 * (size_t)id[r] + half], half ? kq[r] + 1 : (int)K - kq[r]);
        }
    }
    if (bad) raise_status(status, bad);
    // Launched with programmatic stream serialisation behind the slot-clock scan, which lets its dependents start early: this
    // grid reads nothing of the scan's, but it must not complete before the scan has (the kernels behind it wait for this
    // grid only, and the call's status word and slot clock have to be final by then).
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

cudaError_t launch_first_last(const DeviceTrace &t, const Workspace &w, int32_t *first_use, int32_t *last_use, cudaStream_t s)
{
    if (t.N == 0) return cudaSuccess;
    cudaError_t e = cudaMemsetAsync(first_use, 0, sizeof(int32_t) * (size_t)t.N, s);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(last_use, 0, sizeof(int32_t) * (size_t)t.N, s);
    if (e != cudaSuccess) return e;
    if (t.E > 0 && t.K > 0) {
        const int blocks = (int)tiles_of(t.K, kFlThreads);
        k_first_last_events<<<blocks, kFlThreads, 0, s>>>(t.E, t.N, t.K, t.kernel_ptr, t.kernel_tensors, first_use, last_use, w.event_budget, w.status); count_launch();
    }
    return cudaGetLastError();
}

// =============================================================================================
// Heavy tensors: one block sorts the segment (bitonic network that only ever moves values up, so an
// arbitrary length works by skipping partners beyond the end), removes repeats in place and counts
// the periods.  cnt[tensor] receives the tensor's slot in heavy_info.
// =============================================================================================
constexpr int kHeavyThreads = 256;
constexpr int kHeavySmem = 8192;   // ints sorted in shared memory; longer segments are sorted in global memory

__device__ void block_bitonic_sort(int32_t *a, int n)
{
    int n2 = 1;
    while (n2 < n) n2 <<= 1;
    for (int k = 2; k <= n2; k <<= 1) {
        // first stage of each merge mirrors the upper half, the others are plain half-cleaners
        for (int j = k >> 1; j > 0; j >>= 1) {
            const bool mirror = (j == (k >> 1));
            for (int t = threadIdx.x; t < n2 / 2; t += blockDim.x) {
                const int blk = t / j, off = t % j;
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

__global__ void __launch_bounds__(kHeavyThreads) k_sort_heavy(const unsigned *heavy_count, const int32_t *__restrict__ heavy_list,
                                                              const int32_t *__restrict__ raw_ptr, int32_t *__restrict__ raw_uses,
                                                              int32_t *__restrict__ cnt, int32_t *__restrict__ heavy_info)
{
    __shared__ int32_t s_buf[kHeavySmem];
    __shared__ int s_wcount[kHeavyThreads / 32];
    __shared__ int s_total, s_periods;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned nh = *heavy_count;
    for (unsigned h = blockIdx.x; h < nh; h += gridDim.x) {
        const int32_t i = heavy_list[h];
        const int beg = raw_ptr[i], n = raw_ptr[i + 1] - beg;
        int32_t *seg = raw_uses + beg;
        int32_t *a = n <= kHeavySmem ? s_buf : seg;
        if (n <= kHeavySmem) {
            for (int t = threadIdx.x; t < n; t += blockDim.x) s_buf[t] = seg[t];
        }
        __syncthreads();
        block_bitonic_sort(a, n);
        // in-place compaction of the distinct values, chunk by chunk, in order (read chunk, sync, write)
        if (threadIdx.x == 0) { s_total = 0; s_periods = 0; }
        __syncthreads();
        for (int c0 = 0; c0 < n; c0 += blockDim.x) {
            const int t = c0 + threadIdx.x;
            int32_t x = 0, prev = 0;
            bool keep = false, per = false;
            if (t < n) {
                x = a[t];
                if (t > 0) prev = a[t - 1];
                keep = (t == 0) || (x != prev);
                per = keep && t > 0 && (x - prev >= 2);
            }
            const unsigned mk = __ballot_sync(0xffffffffu, keep);
            const unsigned mp = __ballot_sync(0xffffffffu, per);
            if (lane == 0) s_wcount[warp] = __popc(mk);
            __syncthreads();
            int off = s_total;
            for (int w = 0; w < warp; ++w) off += s_wcount[w];
            off += __popc(mk & ((1u << lane) - 1u));
            int chunk_total = 0;
            for (int w = 0; w < kHeavyThreads / 32; ++w) chunk_total += s_wcount[w];
            __syncthreads();                                   // every a[t], a[t-1] of this chunk has been read
            if (keep) seg[off] = x;                            // off <= t: never overtakes an unread element
            if (lane == 0 && mp) atomicAdd(&s_periods, __popc(mp));
            if (threadIdx.x == 0) s_total += chunk_total;
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            heavy_info[2 * h] = s_total;
            heavy_info[2 * h + 1] = s_periods;
            cnt[i] = (int32_t)h;
        }
        __syncthreads();
    }
}

// =============================================================================================
// Vitality emit: per tensor sort its (few) raw uses, drop repeats, count periods; one fused
// two-sum look-back scan gives every tensor its offsets into `uses` and into the period arrays;
// then first / last / count / CSR pointers / sorted uses / periods are written in a single pass.
// =============================================================================================
constexpr int kEmThreads = kScanThreads;
constexpr int kEmItems = 4;
constexpr int kEmTile = kEmThreads * kEmItems;

__global__ void __launch_bounds__(kEmThreads) k_vitality_emit(int64_t N, const int32_t *__restrict__ raw_ptr, int32_t *__restrict__ raw_uses,
                                                              const int32_t *__restrict__ cnt, const int32_t *__restrict__ heavy_info,
                                                              VitalityBuffers out, TileState<2> st, int tiles, ull *status)
{
    __shared__ int s_heavy_n;
    __shared__ int s_heavy_tensor[kEmTile];
    __shared__ int s_wcount[kEmThreads / 32];
    __shared__ int s_chunk_base;
    const int tile = next_tile(st.ticket);
    if (tile >= tiles) return;
    if (threadIdx.x == 0) s_heavy_n = 0;
    const int64_t base = (int64_t)tile * kEmTile + (int64_t)threadIdx.x * kEmItems;
    int beg[kEmItems], d[kEmItems], pc[kEmItems];
    bool heavy[kEmItems];
    Sums<2> mine;
    mine.v[0] = 0; mine.v[1] = 0;
#pragma unroll
    for (int j = 0; j < kEmItems; ++j) {
        const int64_t i = base + j;
        beg[j] = 0; d[j] = 0; pc[j] = 0; heavy[j] = false;
        if (i < N) {
            beg[j] = raw_ptr[i];
            const int n = raw_ptr[i + 1] - beg[j];
            if (n > kHeavyThreshold) {
                const int h = cnt[i];
                heavy[j] = true;
                d[j] = heavy_info[2 * h];
                pc[j] = heavy_info[2 * h + 1];
            } else if (n > 0) {
                int32_t *seg = raw_uses + beg[j];
                for (int a = 1; a < n; ++a) {               // insertion sort, n <= 32
                    const int32_t x = seg[a];
                    int b = a - 1;
                    while (b >= 0 && seg[b] > x) { seg[b + 1] = seg[b]; --b; }
                    seg[b + 1] = x;
                }
                int32_t prev = seg[0];
                int dd = 1, pp = 0;
                for (int a = 1; a < n; ++a) {
                    const int32_t x = seg[a];
                    if (x != prev) { if (x - prev >= 2) ++pp; seg[dd++] = x; prev = x; }
                }
                d[j] = dd; pc[j] = pp;
            }
        }
        mine.v[0] += d[j];
        mine.v[1] += pc[j];
    }
    Sums<2> total;
    Sums<2> ex = block_exclusive_with_lookback<2>(st, tile, mine, status, &total);
    long long uoff = ex.v[0], poff = ex.v[1];
    ull bad = 0;
#pragma unroll
    for (int j = 0; j < kEmItems; ++j) {
        const int64_t i = base + j;
        if (i < N) {
            const int32_t *seg = raw_uses + beg[j];
            out.num_uses[i] = d[j];
            out.use_ptr[i] = uoff;
            out.period_ptr[i] = poff;
            out.first_use[i] = d[j] > 0 ? seg[0] : -1;
            out.last_use[i] = d[j] > 0 ? seg[d[j] - 1] : -1;
            if (uoff + d[j] > out.uses_cap) bad |= G10_DEV_USES_OVERFLOW;
            if (poff + pc[j] > out.periods_cap) bad |= G10_DEV_PERIODS_OVERFLOW;
            if (heavy[j]) {
                s_heavy_tensor[atomicAdd(&s_heavy_n, 1)] = (int)i;
            } else {
                long long po = poff;
                for (int a = 0; a < d[j]; ++a) {
                    const int32_t x = seg[a];
                    if (uoff + a < out.uses_cap) out.uses[uoff + a] = x;
                    if (a > 0 && x - seg[a - 1] >= 2) {
                        if (po < out.periods_cap) {
                            out.period_tensor[po] = (int32_t)i;
                            out.period_prev_use[po] = seg[a - 1];
                            out.period_next_use[po] = x;
                        }
                        ++po;
                    }
                }
            }
        }
        uoff += d[j];
        poff += pc[j];
    }
    if (bad) raise_status(status, bad);
    if (tile == tiles - 1 && threadIdx.x == 0) {
        out.use_ptr[N] = total.v[0];
        out.period_ptr[N] = total.v[1];
        out.counts[0] = total.v[0];
        out.counts[1] = total.v[1];
    }
    __syncthreads();
    // heavy tensors of this tile, one after the other, with the whole block
    const int nh = s_heavy_n;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int q = 0; q < nh; ++q) {
        // offsets and counts were written to global memory by the owning thread before the barrier above
        const int tensor = s_heavy_tensor[q];
        const int32_t *seg = raw_uses + raw_ptr[tensor];
        const int dd = out.num_uses[tensor];
        const long long uo = out.use_ptr[tensor], po = out.period_ptr[tensor];
        if (threadIdx.x == 0) s_chunk_base = 0;
        __syncthreads();
        for (int t = threadIdx.x; t < dd; t += blockDim.x)
            if (uo + t < out.uses_cap) out.uses[uo + t] = seg[t];
        for (int c0 = 1; c0 < dd; c0 += blockDim.x) {
            const int t = c0 + threadIdx.x;
            bool per = false;
            int32_t x = 0, prev = 0;
            if (t < dd) { x = seg[t]; prev = seg[t - 1]; per = (x - prev >= 2); }
            const unsigned mp = __ballot_sync(0xffffffffu, per);
            if (lane == 0) s_wcount[warp] = __popc(mp);
            __syncthreads();
            int off = s_chunk_base;
            for (int w = 0; w < warp; ++w) off += s_wcount[w];
            off += __popc(mp & ((1u << lane) - 1u));
            if (per && po + off < out.periods_cap) {
                out.period_tensor[po + off] = tensor;
                out.period_prev_use[po + off] = prev;
                out.period_next_use[po + off] = x;
            }
            __syncthreads();
            if (threadIdx.x == 0) { int tot = 0; for (int w = 0; w < kEmThreads / 32; ++w) tot += s_wcount[w]; s_chunk_base += tot; }
            __syncthreads();
        }
        __syncthreads();
    }
}

cudaError_t launch_vitality(const DeviceTrace &t, const Workspace &w, const VitalityBuffers &out, cudaStream_t s)
{
    if (t.E > 0 && t.N > 0) {
        k_count_events<<<(unsigned)tiles_of(t.E, kEvTile), kEvThreads, 0, s>>>(t.E, t.N, t.kernel_tensors, w.cnt, w.status); count_launch();
    }
    {
        const int tiles = (int)tiles_of(t.N, kScanTile);
        TileState<1> st{w.count_scan.ticket, w.count_scan.flag, w.count_scan.agg, w.count_scan.incl};
        k_scan_counts<<<tiles, kScanThreads, 0, s>>>(t.N, w.cnt, w.raw_ptr, w.heavy_list, w.heavy_count, st, tiles, w.status); count_launch();
    }
    if (t.E > 0 && t.N > 0 && t.K > 0) {
        k_scatter_events<<<(unsigned)tiles_of(t.E, kEvTile), kEvThreads, 0, s>>>(t.E, t.N, t.K, t.kernel_ptr, t.kernel_tensors,
                                                                                 w.raw_ptr, w.cnt, w.raw_uses); count_launch();
        k_sort_heavy<<<64, kHeavyThreads, 0, s>>>(w.heavy_count, w.heavy_list, w.raw_ptr, w.raw_uses, w.cnt, w.heavy_info); count_launch();
    }
    {
        const int tiles = (int)tiles_of(t.N, kEmTile);
        TileState<2> st{w.emit_scan.ticket, w.emit_scan.flag, w.emit_scan.agg, w.emit_scan.incl};
        k_vitality_emit<<<tiles, kEmThreads, 0, s>>>(t.N, w.raw_ptr, w.raw_uses, w.cnt, w.heavy_info, out, st, tiles, w.status); count_launch();
    }
    return cudaGetLastError();
}

// =============================================================================================
// Pressure timeline: D[first] += size, D[last + 1] -= size (a global tensor that is used at all is
// alive in every slot: its size goes to D[0] only), then P = inclusive scan of D, peak and its
// lowest slot.
// =============================================================================================
// kEncoded: first / last come straight from k_first_last_events (first as K - k, 0 = unused; last as k + 1).
template <bool kEncoded>
__global__ void __launch_bounds__(256) k_diff_scatter(int64_t N, int64_t K, const int64_t *__restrict__ bytes, const uint8_t *__restrict__ glob,
                                                      const int32_t *__restrict__ first, const int32_t *__restrict__ last,
                                                      ull *__restrict__ diff, ull *status)
{
    __shared__ long long s_part[8];
    // (launched with programmatic stream serialisation: its blocks may be placed while the kernel before it drains;
    // nothing is read before that kernel has finished and its writes are visible.  No effect on an ordinary launch.)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    long long gsum = 0;
    if (i < N) {
        const long long b = bytes[i];
        if (b < 1 || b >= ((long long)1 << 40)) raise_status(status, G10_DEV_BAD_BYTES);
        int f = first[i];
        if (kEncoded) f = f == 0 ? -1 : (int)K - f;
        if (f >= 0 && f < K) {
            if (glob != nullptr && glob[i]) gsum = b;
            else {
                atomicAdd(&diff[f], (ull)b);
                const int l = kEncoded ? last[i] - 1 : last[i];
                if (l + 1 < K) atomicAdd(&diff[l + 1], (ull)(-b));
            }
        }
    }
    // global tensors all land on D[0]: one atomic per block instead of one per tensor
    gsum = warp_sum_i64(gsum);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = gsum;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long tot = 0;
        for (int w = 0; w < 8; ++w) tot += s_part[w];
        if (tot != 0) atomicAdd(&diff[0], (ull)tot);
    }
}
// The same from the interleaved pair array of k_first_last_pairs.  A tensor that a single kernel uses (most tensors of a
// trace) is alive in that slot alone: instead of a birth and a death next to each other in the difference array it is
// booked once, in `point`, which the pressure scan adds to its result slot by slot.
__global__ void __launch_bounds__(256) k_diff_scatter_pairs(int64_t N, int64_t K, const int64_t *__restrict__ bytes, const uint8_t *__restrict__ glob,
                                                            const int2 *__restrict__ pair, ull *__restrict__ diff, ull *__restrict__ point, ull *status)
{
    __shared__ long long s_part[8];
    asm volatile("griddepcontrol.wait;" ::: "memory");     // (see k_diff_scatter)
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    long long gsum = 0;
    if (i < N) {
        const long long b = bytes[i];
        if (b < 1 || b >= ((long long)1 << 40)) raise_status(status, G10_DEV_BAD_BYTES);
        const int2 enc = pair[i];                                // K - first, last + 1; 0 = unused
        if (enc.x > 0 && enc.x <= K && enc.y > 0 && enc.y <= K) {
            const int64_t f = K - enc.x, l = (int64_t)enc.y - 1;
            if (glob != nullptr && glob[i]) gsum = b;
            else if (f == l) atomicAdd(&point[f], (ull)b);
            else {
                atomicAdd(&diff[f], (ull)b);
                if (l + 1 < K) atomicAdd(&diff[l + 1], (ull)(-b));
            }
        }
    }
    gsum = warp_sum_i64(gsum);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = gsum;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long tot = 0;
        for (int w = 0; w < 8; ++w) tot += s_part[w];
        if (tot != 0) atomicAdd(&diff[0], (ull)tot);
    }
}

// The same from first / last use as the vitality analysis reports them (-1 = unused), handed over by the caller.
__global__ void __launch_bounds__(256) k_diff_scatter_given(int64_t N, int64_t K, const int64_t *__restrict__ bytes, const uint8_t *__restrict__ glob,
                                                            const int32_t *__restrict__ first_use, const int32_t *__restrict__ last_use,
                                                            ull *__restrict__ diff, ull *__restrict__ point, ull *status)
{
    __shared__ long long s_part[8];
    asm volatile("griddepcontrol.wait;" ::: "memory");     // (see k_diff_scatter)
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    long long gsum = 0;
    if (i < N) {
        const long long b = bytes[i];
        if (b < 1 || b >= ((long long)1 << 40)) raise_status(status, G10_DEV_BAD_BYTES);
        const int64_t f = first_use[i], l = last_use[i];
        if (f >= 0) {
            if (l < f || l >= K) raise_status(status, G10_DEV_BAD_FIRST_LAST);
            else if (glob != nullptr && glob[i]) gsum = b;
            else if (f == l) atomicAdd(&point[f], (ull)b);
            else {
                atomicAdd(&diff[f], (ull)b);
                if (l + 1 < K) atomicAdd(&diff[l + 1], (ull)(-b));
            }
        }
    }
    gsum = warp_sum_i64(gsum);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = gsum;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long tot = 0;
        for (int w = 0; w < 8; ++w) tot += s_part[w];
        if (tot != 0) atomicAdd(&diff[0], (ull)tot);
    }
}

cudaError_t launch_pressure(const DeviceTrace &t, const Workspace &w, const int32_t *first_use, const int32_t *last_use, bool encoded,
                            int64_t *pressure, int64_t *peak_bytes, int32_t *peak_slot, cudaStream_t s)
{
    // Both kernels are launched with programmatic stream serialisation and wait for their predecessor themselves
    // (griddepcontrol.wait at their start): the launch and the placement of their blocks overlap its tail.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (t.N > 0 && t.K > 0) {
        cfg.gridDim = dim3((unsigned)((t.N + 255) / 256));
        cfg.blockDim = dim3(256);
        const int64_t *bytes = t.tensor_bytes;
        const uint8_t *glob = t.tensor_global;
        ull *diff = (ull *)w.diff;
        if (encoded) e = cudaLaunchKernelEx(&cfg, k_diff_scatter<true>, t.N, t.K, bytes, glob, first_use, last_use, diff, w.status);
        else e = cudaLaunchKernelEx(&cfg, k_diff_scatter<false>, t.N, t.K, bytes, glob, first_use, last_use, diff, w.status);
        if (e != cudaSuccess) return e;
    }
    cfg.gridDim = dim3((unsigned)seg_scan_blocks(t.K));
    cfg.blockDim = dim3(kSegThreads);
    e = cudaLaunchKernelEx(&cfg, k_seg_scan<1>, t.K, (int64_t)0, (const int64_t *)w.diff, (const int64_t *)nullptr, pressure, w.pressure_scan.ticket,
                           w.pressure_scan.done, w.seg_words2, w.tile_max, w.tile_slot, peak_bytes, peak_slot, w.status, (int64_t *)nullptr, (int64_t *)nullptr, (int64_t *)nullptr);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

// The timeline call: slot clock beside the first / last pass (the two are independent), difference array from the pairs,
// pressure scan.  `pair` [2 N], `point` [K] and the difference array start at zero (cleared by the caller).
cudaError_t launch_timeline_pairs(const DeviceTrace &t, const Workspace &w, int64_t *start, int32_t *pair, int64_t *point, int64_t *pressure,
                                  int64_t *peak_bytes, int32_t *peak_slot, int64_t *status_out, cudaStream_t s)
{
    cudaError_t e;
    if ((e = launch_slot_clock(t, w, start, s)) != cudaSuccess) return e;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (t.N > 0 && t.E > 0 && t.K > 0) {
        cfg.gridDim = dim3((unsigned)tiles_of(t.K, kFlThreads));
        cfg.blockDim = dim3(kFlThreads);
        if ((e = cudaLaunchKernelEx(&cfg, k_first_last_pairs, t.E, t.N, t.K, t.kernel_ptr, t.kernel_tensors, pair, w.event_budget, w.status, w.diff, point)) != cudaSuccess) return e;
    } else if (t.K > 0) {
        // (no events: nothing clears the difference array and the point masses on the way)
        if ((e = cudaMemsetAsync(w.diff, 0, sizeof(int64_t) * (size_t)(t.K + 1), s)) != cudaSuccess) return e;
        if ((e = cudaMemsetAsync(point, 0, sizeof(int64_t) * (size_t)t.K, s)) != cudaSuccess) return e;
    }
    if (t.N > 0 && t.K > 0) {
        cfg.gridDim = dim3((unsigned)((t.N + 255) / 256));
        cfg.blockDim = dim3(256);
        const int64_t *bytes = t.tensor_bytes;
        const uint8_t *glob = t.tensor_global;
        const int2 *cpair = reinterpret_cast<const int2 *>(pair);
        if ((e = cudaLaunchKernelEx(&cfg, k_diff_scatter_pairs, t.N, t.K, bytes, glob, cpair, (ull *)w.diff, (ull *)point, w.status)) != cudaSuccess) return e;
    }
    cfg.gridDim = dim3((unsigned)seg_scan_blocks(t.K));
    cfg.blockDim = dim3(kSegThreads);
    return cudaLaunchKernelEx(&cfg, k_seg_scan<1>, t.K, (int64_t)0, (const int64_t *)w.diff, (const int64_t *)point, pressure, w.pressure_scan.ticket,
                              w.pressure_scan.done, w.seg_words2, w.tile_max, w.tile_slot, peak_bytes, peak_slot, w.status, status_out, (int64_t *)nullptr, (int64_t *)nullptr);
}

cudaError_t launch_pressure_scan(const DeviceTrace &t, const Workspace &w, const int64_t *point, int64_t *pressure, int64_t *peak_bytes,
                                 int32_t *peak_slot, int64_t *status_out, cudaStream_t s)
{
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3((unsigned)seg_scan_blocks(t.K));
    cfg.blockDim = dim3(kSegThreads);
    return cudaLaunchKernelEx(&cfg, k_seg_scan<1>, t.K, (int64_t)0, (const int64_t *)w.diff, point, pressure, w.pressure_scan.ticket,
                              w.pressure_scan.done, w.seg_words2, w.tile_max, w.tile_slot, peak_bytes, peak_slot, w.status, status_out, (int64_t *)nullptr, (int64_t *)nullptr);
}

// The timeline call when the caller hands first / last use over: slot clock, then (beside it) the bookings, then the scan.
// The caller has cleared w.diff [K + 1] and point [K].
cudaError_t launch_timeline_given(const DeviceTrace &t, const Workspace &w, int64_t *start, const int32_t *first_use, const int32_t *last_use,
                                  int64_t *point, int64_t *pressure, int64_t *peak_bytes, int32_t *peak_slot, int64_t *status_out, cudaStream_t s)
{
    cudaError_t e;
    if ((e = launch_slot_clock(t, w, start, s)) != cudaSuccess) return e;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (t.N > 0 && t.K > 0) {
        cfg.gridDim = dim3((unsigned)((t.N + 255) / 256));
        cfg.blockDim = dim3(256);
        const int64_t *bytes = t.tensor_bytes;
        const uint8_t *glob = t.tensor_global;
        if ((e = cudaLaunchKernelEx(&cfg, k_diff_scatter_given, t.N, t.K, bytes, glob, first_use, last_use, (ull *)w.diff, (ull *)point, w.status)) != cudaSuccess) return e;
    }
    cfg.gridDim = dim3((unsigned)seg_scan_blocks(t.K));
    cfg.blockDim = dim3(kSegThreads);
    return cudaLaunchKernelEx(&cfg, k_seg_scan<1>, t.K, (int64_t)0, (const int64_t *)w.diff, (const int64_t *)point, pressure, w.pressure_scan.ticket,
                              w.pressure_scan.done, w.seg_words2, w.tile_max, w.tile_slot, peak_bytes, peak_slot, w.status, status_out, (int64_t *)nullptr, (int64_t *)nullptr);
}

// =============================================================================================
// Candidate geometry.
// =============================================================================================
__global__ void __launch_bounds__(256) k_geometry(int64_t K, int64_t Pn_bound, const int64_t *Pn_dev, const int64_t *__restrict__ start,
                                                  const int64_t *__restrict__ bytes, const int32_t *__restrict__ per_t,
                                                  const int32_t *__restrict__ per_u, const int32_t *__restrict__ per_v,
                                                  uint64_t host_bw, uint64_t ssd_bw, int64_t stride, int64_t *__restrict__ geo_t,
                                                  int32_t *__restrict__ geo_a, int32_t *__restrict__ geo_b)
{
    const int64_t Pn = Pn_dev ? (*Pn_dev < Pn_bound ? *Pn_dev : Pn_bound) : Pn_bound;
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= Pn) return;
    const int64_t s = bytes[per_t[p]];
    const int u = per_u[p], v = per_v[p];
#pragma unroll
    for (int X = 0; X < 2; ++X) {
        int64_t t;
        int a_abs, b_abs;
        period_geometry(start, u, v, s, X == G10_DEST_SSD ? ssd_bw : host_bw, &t, &a_abs, &b_abs);
        geo_t[X * stride + p] = t;
        geo_a[X * stride + p] = a_abs;
        geo_b[X * stride + p] = b_abs;
    }
    (void)K;
}

cudaError_t launch_geometry(int64_t K, int64_t Pn_bound, const int64_t *Pn_dev, const int64_t *start, const int64_t *tensor_bytes,
                            const int32_t *per_t, const int32_t *per_u, const int32_t *per_v, uint64_t host_bw, uint64_t ssd_bw,
                            int64_t stride, int64_t *geo_t, int32_t *geo_a, int32_t *geo_b, cudaStream_t s)
{
    if (Pn_bound <= 0) return cudaSuccess;
    k_geometry<<<(unsigned)((Pn_bound + 255) / 256), 256, 0, s>>>(K, Pn_bound, Pn_dev, start, tensor_bytes, per_t, per_u, per_v,
                                                                  host_bw, ssd_bw, stride, geo_t, geo_a, geo_b); count_launch();
    return cudaGetLastError();
}

}  // namespace g10

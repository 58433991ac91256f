// Code instrumentation (Section 4.4, Figure 9): the stream of g10_alloc / g10_free / g10_pre_evict /
// g10_prefetch calls, ordered by kernel boundary, then FREE < PRE_EVICT < ALLOC < PREFETCH, then tensor id.
//
// Every instruction is one 64-bit key (boundary << 33 | opcode << 31 | tensor; unique) plus the plan record it
// came from.  The keys are sorted with the same shape as the vitality pass: boundaries are cut into buckets of
// consecutive boundaries holding a couple of thousand instructions, a histogram sizes the buckets -- kept per block of
// the counting kernel, so that the scatter kernel, whose blocks walk the same items, knows each block's own run inside
// every bucket and places its keys with shared-memory counters alone (no global cursor) --, the keys are
// scattered into their bucket's slice, and one block per bucket sorts its slice in shared memory (counting sort by
// boundary, then the few instructions of every boundary in key order by one thread; a boundary with more than 32
// by a bitonic network), which also gives the CSR pointers, and writes the records out in order.
// A bucket too large for shared memory (very many tensors allocated at one boundary) is sorted in global memory.
#include "g10_device.cuh"
#include "g10_internal.h"
#include <cstddef>

namespace g10 {

constexpr int kEmitThreads = 512;
constexpr int kEmitCap = 4096;            // instructions of a bucket sorted in shared memory
enum { kOpFree = 0, kOpPreEvict = 1, kOpAlloc = 2, kOpPrefetch = 3 };

struct EmitArgs {
    int64_t K, N, n;
    const int32_t *first_use, *last_use;
    const int64_t *bytes;
    const uint8_t *glob;
    const int64_t *start;
    const g10_migration *mig;
    const int64_t *new_issue;
    int bw, nb;                           // boundaries per bucket, buckets
    ull magic;                            // ceil(2^64 / bw) (0 when bw == 1): the bucket of boundary x is the high half of x * magic
    unsigned *bucket_count, *bucket_cursor;
    unsigned *block_count;                // [nb][G] per bucket: what each block of the counting kernel saw, then the running sums
    int G;                                // blocks of the counting and of the scatter kernel (the same items go to the same block)
    ull *keys;
    int32_t *payload;
    unsigned *ticket;
    ull *status;
};

// item -> (boundary, opcode, tensor, record); false if the item does not exist
__device__ __forceinline__ bool emit_item(const EmitArgs &A, int64_t item, int64_t *boundary, int *opcode, int *tensor, int *record)
{
    *record = -1;
    if (item < 2 * A.N) {
        const int64_t i = item < A.N ? item : item - A.N;
        const int f = A.first_use[i];
        if (f < 0) return false;
        const bool g = A.glob != nullptr && A.glob[i] != 0;
        *tensor = (int)i;
        if (item < A.N) { *opcode = kOpAlloc; *boundary = g ? 0 : f; return true; }
        if (g) return false;
        *opcode = kOpFree; *boundary = (int64_t)A.last_use[i] + 1;
        return true;
    }
    const int64_t r = item - 2 * A.N < A.n ? item - 2 * A.N : item - 2 * A.N - A.n;
    const bool evict = item - 2 * A.N < A.n;
    *record = (int)r; *tensor = A.mig[r].tensor;
    int64_t t = evict ? A.mig[r].evict_issue_ns : (A.new_issue ? A.new_issue[r] : A.mig[r].prefetch_issue_ns);
    // (a steady-state plan: the prefetch of a wrap-around period may lie in the next iteration; it stands at the same
    // moment of this one)
    if (!evict && t >= A.start[A.K]) t -= A.start[A.K];
    // last boundary b in [0, K] with start[b] <= t (for a pre-eviction start[b] == t_r exactly)
    int lo = 0, hi = (int)A.K;
    while (lo < hi) { const int mid = lo + (hi - lo + 1) / 2; if (A.start[mid] <= t) lo = mid; else hi = mid - 1; }
    *boundary = lo; *opcode = evict ? kOpPreEvict : kOpPrefetch;
    return true;
}

// Bucket of a boundary.  With magic = (2^64 + e) / bw, 0 <= e < bw, the product x * magic / 2^64 exceeds x / bw by less than
// 2^-32 for x < 2^32, and x / bw is at least 1 / bw short of the next integer: the high half is the quotient exactly.
__device__ __forceinline__ int emit_bucket(const EmitArgs &A, int64_t boundary)
{
    return A.magic ? (int)__umul64hi((ull)boundary, A.magic) : (int)boundary;
}

__device__ __forceinline__ ull emit_key(int64_t boundary, int opcode, int tensor)
{
    return ((ull)boundary << 33) | ((ull)opcode << 31) | (ull)(unsigned)tensor;
}

__global__ void __launch_bounds__(kEmitThreads) k_emit_hist(EmitArgs A)
{
    extern __shared__ unsigned s_hist[];
    for (int b = threadIdx.x; b < A.nb; b += kEmitThreads) s_hist[b] = 0;
    __syncthreads();
    const int64_t total = 2 * A.N + 2 * A.n;
    for (int64_t item = (int64_t)blockIdx.x * kEmitThreads + threadIdx.x; item < total; item += (int64_t)gridDim.x * kEmitThreads) {
        int64_t bd; int op, tn, rc;
        if (emit_item(A, item, &bd, &op, &tn, &rc)) atomicAdd(&s_hist[emit_bucket(A, bd)], 1u);
    }
    __syncthreads();
    // what this block saw of every bucket: the scatter kernel, whose blocks walk the same items, gets from it the block's own
    // run inside every bucket's slice and needs no global cursor
    for (int b = threadIdx.x; b < A.nb; b += kEmitThreads) A.block_count[(size_t)b * A.G + blockIdx.x] = s_hist[b];
}

// Per bucket: running sums over the blocks (in place) and the bucket's total.  One warp per bucket.
__global__ void __launch_bounds__(kEmitThreads) k_emit_block_offsets(EmitArgs A)
{
    const int lane = threadIdx.x & 31;
    const int b = (int)(blockIdx.x * (kEmitThreads / 32) + (threadIdx.x >> 5));
    if (b >= A.nb) return;
    unsigned *row = A.block_count + (size_t)b * A.G;
    unsigned carry = 0;
    for (int j0 = 0; j0 < A.G; j0 += 32) {
        const int j = j0 + lane;
        const unsigned v = j < A.G ? row[j] : 0u;
        unsigned incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const unsigned y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
        if (j < A.G) row[j] = carry + incl - v;
        carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) A.bucket_count[b] = carry;
}

// exclusive scan of the bucket counts (nb <= 4096) into s_base[0..nb]
__device__ __forceinline__ void emit_scan_buckets(const unsigned *cnt, int nb, long long *s_base, long long *s_w)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    long long carry = 0;
    for (int base = 0; base < nb; base += kEmitThreads) {
        const int j = base + threadIdx.x;
        const long long v = j < nb ? (long long)cnt[j] : 0;
        const long long incl = warp_inclusive_scan_i64(v, lane);
        __syncthreads();
        if (lane == 31) s_w[warp] = incl;
        __syncthreads();
        long long wpre = 0, tot = 0;
        for (int w = 0; w < kEmitThreads / 32; ++w) { const long long x = s_w[w]; if (w < warp) wpre += x; tot += x; }
        if (j < nb) s_base[j] = carry + wpre + incl - v;
        carry += tot;
    }
    __syncthreads();
    if (threadIdx.x == 0) s_base[nb] = carry;
    __syncthreads();
}

__global__ void __launch_bounds__(kEmitThreads) k_emit_scatter(EmitArgs A)
{
    extern __shared__ long long s_base[];            // [nb + 1] first slot of each bucket, then [nb] (unsigned) this block's next slot inside it
    __shared__ long long s_w[kEmitThreads / 32];
    emit_scan_buckets(A.bucket_count, A.nb, s_base, s_w);
    unsigned *s_next = (unsigned *)(s_base + A.nb + 1);
    for (int b = threadIdx.x; b < A.nb; b += kEmitThreads) s_next[b] = A.block_count[(size_t)b * A.G + blockIdx.x];
    __syncthreads();
    const int64_t total = 2 * A.N + 2 * A.n;
    for (int64_t item = (int64_t)blockIdx.x * kEmitThreads + threadIdx.x; item < total; item += (int64_t)gridDim.x * kEmitThreads) {
        int64_t bd; int op, tn, rc;
        if (emit_item(A, item, &bd, &op, &tn, &rc)) {
            const int b = emit_bucket(A, bd);
            const long long pos = s_base[b] + atomicAdd(&s_next[b], 1u);       // (shared memory: the block's own run of the bucket)
            A.keys[pos] = emit_key(bd, op, tn);
            if (rc >= 0) A.payload[pos] = rc;          // (only the few instructions that come from a plan record carry one: the
                                                       // others' payload is never read, which spares a scattered store per tensor)
        }
    }
}

// bitonic network over (key, payload) pairs; arbitrary n (values only ever move up)
__device__ void emit_bitonic(ull *k, int32_t *p, int n)
{
    int n2 = 1;
    while (n2 < n) n2 <<= 1;
    for (int kk = 2; kk <= n2; kk <<= 1) {
        for (int j = kk >> 1, lj = 31 - __clz(kk >> 1); j > 0; j >>= 1, --lj) {
            const bool mirror = (j == (kk >> 1));
            for (int t = threadIdx.x; t < n2 / 2; t += blockDim.x) {
                const int blk = t >> lj, off = t & (j - 1);
                const int i = blk * 2 * j + off;
                const int q = mirror ? (blk * 2 * j + 2 * j - 1 - off) : (i + j);
                if (q < n) {
                    const ull x = k[i], y = k[q];
                    if (x > y) { k[i] = y; k[q] = x; const int32_t px = p[i]; p[i] = p[q]; p[q] = px; }
                }
            }
            __syncthreads();
        }
    }
}

static_assert(sizeof(g10_instruction) == 32 && offsetof(g10_instruction, opcode) == 0 && offsetof(g10_instruction, tensor) == 4 &&
              offsetof(g10_instruction, target) == 8 && offsetof(g10_instruction, record) == 12 && offsetof(g10_instruction, bytes) == 16 &&
              offsetof(g10_instruction, time_ns) == 24, "k_emit_write assembles the record from four 64-bit words");
constexpr int kEmitStageStride = 36;      // (32 + 4: the four word planes of a warp's tile fall into different banks)
constexpr int kEmitRegs = kEmitCap / kEmitThreads;   // keys a thread keeps in registers between the two passes
constexpr int kEmitWide = 32;                        // a boundary with more instructions is sorted by the whole block

__global__ void __launch_bounds__(kEmitThreads, 2) k_emit_write(EmitArgs A, int64_t *inst_ptr, g10_instruction *inst, int64_t inst_cap, int64_t *counts)
{
    extern __shared__ long long s_dyn[];
    long long *s_base = s_dyn;                                   // [nb + 1]
    int *s_cnt = (int *)(s_base + A.nb + 1);                     // [bw + 1] instructions per boundary of the bucket, then their offsets
    int *s_cur = s_cnt + A.bw + 1;                               // [bw] fill cursors
    ull *s_keys = (ull *)(((uintptr_t)(s_cur + A.bw) + 7) & ~(uintptr_t)7);               // [kEmitCap]
    int32_t *s_pay = (int32_t *)(s_keys + kEmitCap);              // [kEmitCap]
    ull *s_stage = (ull *)(s_pay + kEmitCap);                     // [warps][4][kEmitStageStride] the records of a warp on their way out
    __shared__ long long s_w[kEmitThreads / 32];
    __shared__ int s_bucket, s_nwide;
    __shared__ int s_wide[64];
    const int bw = A.bw;
    emit_scan_buckets(A.bucket_count, A.nb, s_base, s_w);
    for (;;) {
        __syncthreads();
        if (threadIdx.x == 0) { s_bucket = (int)atomicAdd(A.ticket, 1u); s_nwide = 0; }
        __syncthreads();
        const int b = s_bucket;
        if (b >= A.nb) break;
        const long long base = s_base[b];
        const int n = (int)(s_base[b + 1] - base);
        ull *gk = A.keys + base;
        int32_t *gp = A.payload + base;
        const int64_t b0 = (int64_t)b * bw;
        const int bw_eff = (int)((A.K + 1 - b0) < bw ? (A.K + 1 - b0) : bw);
        for (int j = threadIdx.x; j <= bw_eff; j += kEmitThreads) { s_cnt[j] = 0; if (j < bw_eff) s_cur[j] = 0; }
        __syncthreads();
        const ull *kp; const int32_t *pp;
        if (n <= kEmitCap) {
            // Counting sort by boundary in shared memory (the keys stay in registers between the two passes), then
            // every boundary's few instructions are put in key order by one thread; the keys are unique, so this is
            // the order a sort of the whole bucket would give.
            ull rk[kEmitRegs];
#pragma unroll
            for (int q = 0; q < kEmitRegs; ++q) {
                const int j = q * kEmitThreads + threadIdx.x;
                rk[q] = j < n ? gk[j] : ~0ull;
            }
#pragma unroll
            for (int q = 0; q < kEmitRegs; ++q)
                if (rk[q] != ~0ull) atomicAdd(&s_cnt[(int)((rk[q] >> 33) - b0)], 1);
            __syncthreads();
            {   // in-place exclusive scan of s_cnt[0..bw_eff), total in s_cnt[bw_eff]
                const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
                int carry = 0;
                for (int c0 = 0; c0 < bw_eff; c0 += kEmitThreads) {
                    const int j = c0 + threadIdx.x;
                    const int v = j < bw_eff ? s_cnt[j] : 0;
                    int incl = v;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
                    __syncthreads();
                    if (lane == 31) s_w[warp] = incl;
                    __syncthreads();
                    int wpre = 0, tot = 0;
                    for (int w = 0; w < kEmitThreads / 32; ++w) { const int x = (int)s_w[w]; if (w < warp) wpre += x; tot += x; }
                    if (j < bw_eff) s_cnt[j] = carry + wpre + incl - v;
                    carry += tot;
                }
                __syncthreads();
                if (threadIdx.x == 0) s_cnt[bw_eff] = carry;
                __syncthreads();
            }
#pragma unroll
            for (int q = 0; q < kEmitRegs; ++q)
                if (rk[q] != ~0ull) {
                    const int j = q * kEmitThreads + threadIdx.x;
                    const int bd = (int)((rk[q] >> 33) - b0);
                    const int slot = s_cnt[bd] + atomicAdd(&s_cur[bd], 1);
                    s_keys[slot] = rk[q];
                    s_pay[slot] = ((rk[q] >> 31) & 1u) ? gp[j] : -1;       // (PRE_EVICT = 1 and PREFETCH = 3 come from a plan record)
                }
            __syncthreads();
            // Inside a boundary the keys go in key order.  Every thread takes back the instructions at its slots, finds for
            // each its rank among the instructions of its boundary by counting the smaller keys (a boundary holds a handful;
            // keys are unique, so ranks are too), and puts it where it belongs.  One thread sorting one boundary, as before,
            // makes the whole block wait for the boundary with the most instructions.
            {
                ull ik[kEmitRegs];
                int ip[kEmitRegs], dst[kEmitRegs];
#pragma unroll
                for (int q = 0; q < kEmitRegs; ++q) {
                    const int j = q * kEmitThreads + threadIdx.x;
                    dst[q] = -1;
                    if (j < n) {
                        ik[q] = s_keys[j]; ip[q] = s_pay[j];
                        const int bd = (int)((ik[q] >> 33) - b0);
                        const int o = s_cnt[bd], m = s_cnt[bd + 1] - o;
                        if (m <= kEmitWide) {
                            int r = 0;
                            for (int a = 0; a < m; ++a) r += s_keys[o + a] < ik[q] ? 1 : 0;
                            dst[q] = o + r;
                        } else if (j == o) { const int w2 = atomicAdd(&s_nwide, 1); if (w2 < 64) s_wide[w2] = bd; }   // (its first slot reports it)
                    }
                }
                __syncthreads();
#pragma unroll
                for (int q = 0; q < kEmitRegs; ++q)
                    if (dst[q] >= 0) { s_keys[dst[q]] = ik[q]; s_pay[dst[q]] = ip[q]; }
            }
            __syncthreads();
            const int nwide = s_nwide;
            for (int hq = 0; hq < (nwide <= 64 ? nwide : bw_eff); ++hq) {
                const int bd = nwide <= 64 ? s_wide[hq] : hq;
                const int o = s_cnt[bd], m = s_cnt[bd + 1] - o;
                if (m <= kEmitWide) continue;                      // (only when the list overflowed: uniform test)
                emit_bitonic(s_keys + o, s_pay + o, m);
            }
            kp = s_keys; pp = s_pay;
        } else {
            emit_bitonic(gk, gp, n);
            for (int j = threadIdx.x; j < n; j += kEmitThreads) atomicAdd(&s_cnt[(int)((gk[j] >> 33) - b0)], 1);
            __syncthreads();
            {   // in-place exclusive scan of s_cnt[0..bw_eff)
                const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
                int carry = 0;
                for (int c0 = 0; c0 < bw_eff; c0 += kEmitThreads) {
                    const int j = c0 + threadIdx.x;
                    const int v = j < bw_eff ? s_cnt[j] : 0;
                    int incl = v;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
                    __syncthreads();
                    if (lane == 31) s_w[warp] = incl;
                    __syncthreads();
                    int wpre = 0, tot = 0;
                    for (int w = 0; w < kEmitThreads / 32; ++w) { const int x = (int)s_w[w]; if (w < warp) wpre += x; tot += x; }
                    if (j < bw_eff) s_cnt[j] = carry + wpre + incl - v;
                    carry += tot;
                }
                __syncthreads();
            }
            kp = gk; pp = gp;
        }
        // CSR pointers of the bucket's boundaries
        for (int j = threadIdx.x; j < bw_eff; j += kEmitThreads) inst_ptr[b0 + j] = base + s_cnt[j];
        if (b == A.nb - 1 && threadIdx.x == 0) {
            inst_ptr[A.K + 1] = s_base[A.nb];
            counts[0] = s_base[A.nb];
            if (s_base[A.nb] > inst_cap) raise_status(A.status, G10_DEV_PLAN_OVERFLOW);
        }
        // the records, in order.  A thread that stored its own 32-byte record would write every 32-byte sector in four pieces
        // (four 8-byte stores at a stride of 32 bytes across the warp); the 32 records of a warp go through a small
        // shared-memory tile instead and leave as four contiguous 256-byte runs.
        {
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            ull *st = s_stage + warp * (4 * kEmitStageStride);
            for (int j0 = 0; j0 < n; j0 += kEmitThreads) {
                const int j = j0 + threadIdx.x;
                ull w0 = 0, w1 = 0, w2 = 0, w3 = 0;
                if (j < n && base + j < inst_cap) {
                    const ull key = kp[j];
                    const int64_t boundary = (int64_t)(key >> 33);
                    const int opcode = (int)((key >> 31) & 3u), tensor = (int)(key & 0x7fffffffu), record = (opcode & 1) ? pp[j] : -1;
                    int target = -1;
                    int64_t time_ns = A.start[boundary];
                    if (opcode == kOpPreEvict) { target = A.mig[record].dest; time_ns = A.mig[record].evict_issue_ns; }
                    if (opcode == kOpPrefetch) {
                        time_ns = A.new_issue ? A.new_issue[record] : A.mig[record].prefetch_issue_ns;
                        if (time_ns >= A.start[A.K]) time_ns -= A.start[A.K];      // (steady-state plans: see emit_item)
                    }
                    w0 = (ull)(unsigned)opcode | ((ull)(unsigned)tensor << 32);
                    w1 = (ull)(unsigned)target | ((ull)(unsigned)record << 32);
                    w2 = (ull)A.bytes[tensor];
                    w3 = (ull)time_ns;
                }
                st[0 * kEmitStageStride + lane] = w0; st[1 * kEmitStageStride + lane] = w1;
                st[2 * kEmitStageStride + lane] = w2; st[3 * kEmitStageStride + lane] = w3;
                __syncwarp();
                const long long first = base + j0 + warp * 32;              // the warp's first record
                long long nrec = n - (j0 + warp * 32);
                if (inst_cap - first < nrec) nrec = inst_cap - first;
                if (nrec > 32) nrec = 32;
                ull *dst = reinterpret_cast<ull *>(inst + first);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int i = q * 32 + lane;                          // 8-byte word of the warp's 1024 bytes
                    if ((i >> 2) < nrec) dst[i] = st[(i & 3) * kEmitStageStride + (i >> 2)];
                }
                __syncwarp();
            }
        }
    }
}

bool emit_choose_buckets(int64_t K, int64_t total_items, int sms, int *bw, int *nb, ull *magic)
{
    // boundaries per bucket so that a bucket holds about 3000 instructions (kEmitCap = 4096 are sorted in shared memory; a
    // fuller bucket goes the slow way); at most 4096 buckets of 4096 boundaries.  k_emit_write takes the buckets one per block
    // at a time with two blocks per SM: with more buckets than blocks they are narrowed to whole rounds of its grid (sms > 0).
    const int64_t B = K + 1;
    int64_t w = total_items > 0 ? (3000 * B) / total_items : 4096;
    w = w < 1 ? 1 : (w > 4096 ? 4096 : w);
    int64_t buckets = (B + w - 1) / w;
    if (buckets > 4096) { w = (B + 4095) / 4096; buckets = (B + w - 1) / w; }
    if (w > 4096) return false;
    const int64_t G = 2 * (int64_t)sms;
    if (G > 0 && buckets > G) {
        const int64_t target = (buckets + G - 1) / G * G;
        if (target <= 4096) { w = (B + target - 1) / target; buckets = (B + w - 1) / w; }
    }
    *bw = (int)w; *nb = (int)buckets;
    *magic = w == 1 ? 0 : ~(ull)0 / (ull)w + 1;
    return true;
}

cudaError_t launch_emit(const EmitLaunch &L, cudaStream_t s)
{
    EmitArgs A;
    A.K = L.K; A.N = L.N; A.n = L.n;
    A.first_use = L.first_use; A.last_use = L.last_use; A.bytes = L.bytes; A.glob = L.glob; A.start = L.start;
    A.mig = L.mig; A.new_issue = L.new_issue;
    A.bucket_count = L.bucket_count; A.bucket_cursor = L.bucket_cursor; A.keys = L.keys; A.payload = L.payload;
    A.ticket = L.ticket; A.status = L.status;
    const int sms = current_sm_count();
    if (sms <= 0) return cudaErrorInvalidDevice;
    if (!emit_choose_buckets(L.K, 2 * L.N + 2 * L.n, sms, &A.bw, &A.nb, &A.magic)) return cudaErrorInvalidValue;
    const int64_t total = 2 * L.N + 2 * L.n;
    int64_t g = (total + kEmitThreads - 1) / kEmitThreads;
    if (g > 4 * (int64_t)sms) g = 4 * (int64_t)sms;
    if (g > kEmitMaxBlocks) g = kEmitMaxBlocks;
    if (g < 1) g = 1;
    A.block_count = L.block_count; A.G = (int)g;
    k_emit_hist<<<(int)g, kEmitThreads, sizeof(unsigned) * (size_t)A.nb, s>>>(A); count_launch();
    k_emit_block_offsets<<<(A.nb + kEmitThreads / 32 - 1) / (kEmitThreads / 32), kEmitThreads, 0, s>>>(A); count_launch();
    const size_t sm2 = sizeof(long long) * (size_t)(A.nb + 1) + sizeof(unsigned) * (size_t)A.nb;
    cudaError_t e2 = cudaFuncSetAttribute(k_emit_scatter, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm2);
    if (e2 != cudaSuccess) return e2;
    k_emit_scatter<<<(int)g, kEmitThreads, sm2, s>>>(A); count_launch();
    const size_t sm3 = sizeof(long long) * (size_t)(A.nb + 1) + sizeof(int) * (size_t)(2 * A.bw + 2) + 8 +
                       (sizeof(ull) + sizeof(int32_t)) * kEmitCap + sizeof(ull) * (kEmitThreads / 32) * 4 * kEmitStageStride;
    cudaError_t e = cudaFuncSetAttribute(k_emit_write, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm3);
    if (e != cudaSuccess) return e;
    const int g3 = A.nb < 2 * sms ? A.nb : 2 * sms;
    k_emit_write<<<g3, kEmitThreads, sm3, s>>>(A, L.inst_ptr, L.inst, L.inst_cap, L.counts); count_launch();
    return cudaGetLastError();
}

}  // namespace g10

// Smart tensor prefetching (Section 4.4): after the eviction plan is made, the evicted periods are visited in
// the order of their latest safe prefetch time and every prefetch is moved back to the earliest slot from which
// the GPU can hold the tensor with the space that is left; the pressure curve is updated as it goes.
//
// Each move changes the pressure the next search sees, so the visits form a sequence.  Two forms:
//   - one block does the whole pass (k_schedule_prefetch: curve in shared memory; k_schedule_prefetch_tiled: curve in
//     global memory with per-tile bounds in shared memory): records ordered by a bitonic network over their indices,
//     then, record by record, a backward search and a range addition, parallel inside each record only;
//   - many blocks (k_pf_rank, k_pf_prepare, k_pf_pipe; needs the caller's workspace): the timeline is cut into one
//     slice per block and a record travels from block to block only as far as its search goes, so that records whose
//     searches lie apart proceed at the same time.  Same results as the sequence.
#include <cstdlib>

#include "g10_device.cuh"
#include "g10_internal.h"

namespace g10 {

// kPfThreads (template parameter): 256 for a timeline that fits shared memory (a block-wide barrier per search chunk
// and per record: few warps keep it cheap), 1024 for a long one in global memory (its ranges are long: width pays)
constexpr int kPfRows = 8;                       // slots a thread looks at per search chunk

// (T = length of the iteration: the prefetch of a steady-state plan's wrap-around period may lie in the next iteration; what
// orders the visits is its moment inside the iteration.  Times of an ordinary plan are all below T.)
__device__ __forceinline__ bool pf_before(const g10_migration *mig, int x, int y, int64_t T)
{
    const int64_t kx = mig[x].prefetch_issue_ns % T, ky = mig[y].prefetch_issue_ns % T;
    return kx < ky || (kx == ky && x < y);
}

// Orders the records by (latest safe prefetch time, record index) into `order`, with the whole block: a bitonic network
// over (time, record) pairs in shared memory (`scratch`: n2 * 12 bytes) when they fit, else over the indices in global memory.
__device__ void pf_order_records(int64_t n, int64_t n2, const g10_migration *__restrict__ mig, int32_t *order, long long *scratch,
                                 int sort_in_smem, int nthreads, int64_t T)
{
    if (sort_in_smem) {
        // (time, record) pairs sorted in shared memory: the network's comparisons would otherwise each cost two
        // dependent global loads
        long long *s_key = scratch;
        int *s_idx = (int *)(s_key + n2);
        for (int64_t i = threadIdx.x; i < n2; i += nthreads) {
            s_key[i] = i < n ? mig[i].prefetch_issue_ns % T : 0x7fffffffffffffffll;
            s_idx[i] = i < n ? (int)i : 0x7fffffff;
        }
        __syncthreads();
        for (int64_t k = 2; k <= n2; k <<= 1) {
            for (int64_t j = k >> 1; j > 0; j >>= 1) {
                const bool mirror = (j == (k >> 1));
                const int lj = 63 - __clzll(j);                        // (j is a power of two)
                for (int64_t t = threadIdx.x; t < n2 / 2; t += nthreads) {
                    const int64_t blk = t >> lj, off = t & (j - 1);
                    const int64_t i = blk * 2 * j + off;
                    const int64_t p = mirror ? (blk * 2 * j + 2 * j - 1 - off) : (i + j);
                    const long long kx = s_key[i], ky = s_key[p];
                    const int ix = s_idx[i], iy = s_idx[p];
                    if (ky < kx || (ky == kx && iy < ix)) { s_key[i] = ky; s_key[p] = kx; s_idx[i] = iy; s_idx[p] = ix; }
                }
                __syncthreads();
            }
        }
        for (int64_t i = threadIdx.x; i < n; i += nthreads) order[i] = s_idx[i];
        __syncthreads();
    } else {
        for (int64_t i = threadIdx.x; i < n; i += nthreads) order[i] = (int32_t)i;
        __syncthreads();
        for (int64_t k = 2; k <= n2; k <<= 1) {
            for (int64_t j = k >> 1; j > 0; j >>= 1) {
                const bool mirror = (j == (k >> 1));
                const int lj = 63 - __clzll(j);
                for (int64_t t = threadIdx.x; t < n2 / 2; t += nthreads) {
                    const int64_t blk = t >> lj, off = t & (j - 1);
                    const int64_t i = blk * 2 * j + off;
                    const int64_t p = mirror ? (blk * 2 * j + 2 * j - 1 - off) : (i + j);
                    if (p < n) {
                        const int32_t x = order[i], y = order[p];
                        if (pf_before(mig, y, x, T)) { order[i] = y; order[p] = x; }
                    }
                }
                __syncthreads();
            }
        }
    }
}

template <int kPfThreads>
__global__ void __launch_bounds__(kPfThreads) k_schedule_prefetch(int64_t K, int64_t n, const g10_migration *__restrict__ mig,
                                                                  const int64_t *__restrict__ start, const int64_t *__restrict__ bytes,
                                                                  int64_t cap, int64_t *P, int32_t *order, int32_t *new_last,
                                                                  int64_t *new_issue, int64_t *summary, int p_in_smem, int sort_in_smem)
{
    extern __shared__ long long s_dyn[];   // the pressure curve, when the launch gave it room
    __shared__ int s_wstop[2][kPfThreads / 32];   // per warp: smallest offset below hi of a slot of the current chunk that cannot take the tensor;
                                                  // two copies used in turn, so that one barrier per chunk is enough
    __shared__ int s_ra[kPfThreads], s_rb[kPfThreads], s_rj[kPfThreads];
    __shared__ long long s_rs[kPfThreads];
    long long *Pw = (long long *)P;
    if (p_in_smem) {
        Pw = s_dyn;
        for (int64_t k = threadIdx.x; k < K; k += kPfThreads) Pw[k] = P[k];
    }
    __shared__ long long s_mx[kPfThreads / 32];
    __shared__ int s_sl[kPfThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // ---- order the records by (latest safe prefetch time, record index)
    int64_t n2 = 1;
    while (n2 < n) n2 <<= 1;
    const int64_t T = K > 0 ? start[K] : 1;
    pf_order_records(n, n2, mig, order, s_dyn + (p_in_smem ? K : 0), sort_in_smem, kPfThreads, T);
    // ---- visit the records in that order, a batch of kPfThreads at a time: the batch's fields are fetched together
    // (one thread per record), the visits read them from shared memory; the pressure curve sits in shared memory
    // too when it fits (Pw), else in global memory
    long long moved = 0, regained = 0;
    int turn = 0;
    for (int64_t q0 = 0; q0 < n; q0 += kPfThreads) {
        const int nb = (int)(n - q0 < kPfThreads ? n - q0 : kPfThreads);
        __syncthreads();
        if ((int)threadIdx.x < nb) {
            const int r = order[q0 + threadIdx.x];
            s_ra[threadIdx.x] = mig[r].absent_first; s_rb[threadIdx.x] = mig[r].absent_last;
            s_rs[threadIdx.x] = bytes[mig[r].tensor];
        }
        __syncthreads();
        for (int q = 0; q < nb; ++q) {
            const int a_abs = s_ra[q], b_abs = s_rb[q];          // unrolled slots; beyond K only for a steady-state plan
            const int64_t s = s_rs[q];
            int j = a_abs - 1;                  // result: last slot that stays absent (unrolled)
            // The range as at most two runs of physical slots, the later one first: the part in the next iteration
            // (slot x stands for slot x - K), then the part in this one.
            const int Ki = (int)K;
            int seg_lo[2], seg_hi[2], seg_off[2], nseg = 0;
            if (b_abs >= Ki) { seg_lo[nseg] = (a_abs > Ki ? a_abs : Ki) - Ki; seg_hi[nseg] = b_abs - Ki; seg_off[nseg] = Ki; ++nseg; }
            if (a_abs < Ki) { seg_lo[nseg] = a_abs; seg_hi[nseg] = b_abs < Ki ? b_abs : Ki - 1; seg_off[nseg] = 0; ++nseg; }
            bool stopped = false;
            for (int g = 0; g < nseg && !stopped; ++g) {
              const int lo_p = seg_lo[g];
              int hi = seg_hi[g];                 // slots (.., seg_hi] above hi are known to take the tensor
              while (hi >= lo_p) {
                // a chunk of kPfRows rows of kPfThreads slots, from hi downwards: row r, thread t looks at slot
                // hi - (r * kPfThreads + t); all loads of a thread are in flight together.  The highest slot that
                // cannot take the tensor is the failing one with the smallest offset r * kPfThreads + t.
                const int span = hi - lo_p + 1;                      // slots still to look at
                int first = 0x7fffffff;                             // this warp's smallest failing offset
                long long pv[kPfRows];
#pragma unroll
                for (int r = 0; r < kPfRows; ++r) {
                    const int off = r * kPfThreads + (int)threadIdx.x;
                    pv[r] = off < span ? Pw[hi - off] : 0;
                }
#pragma unroll
                for (int r = 0; r < kPfRows; ++r) {
                    const int off = r * kPfThreads + (int)threadIdx.x;
                    const unsigned fail = __ballot_sync(0xffffffffu, off < span && pv[r] > cap - s);
                    if (fail && first == 0x7fffffff) first = r * kPfThreads + warp * 32 + __ffs(fail) - 1;
                }
                if (lane == 0) s_wstop[turn][warp] = first;
                __syncthreads();
                const int mine = lane < kPfThreads / 32 ? s_wstop[turn][lane] : 0x7fffffff;      // one warp result per lane
                const int best = (int)__reduce_min_sync(0xffffffffu, (unsigned)mine);
                turn ^= 1;                                                   // (the other copy was last read two barriers ago)
                if (best != 0x7fffffff) { j = hi - best + seg_off[g]; stopped = true; break; }
                hi -= kPfRows * kPfThreads;
              }
            }
            for (int g = 0; g < nseg; ++g) {   // the regained slots (j, b_abs] take the tensor back: read-modify-write, eight per thread in flight
                const int lo_p = (j + 1 - seg_off[g] > seg_lo[g] ? j + 1 - seg_off[g] : seg_lo[g]), hi_p = seg_hi[g];
                const int k0 = lo_p + (int)threadIdx.x;
#pragma unroll 1
                for (int k = k0; k <= hi_p; k += 8 * kPfThreads) {
                    long long v[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) v[u] = k + u * kPfThreads <= hi_p ? Pw[k + u * kPfThreads] : 0;
#pragma unroll
                    for (int u = 0; u < 8; ++u) if (k + u * kPfThreads <= hi_p) Pw[k + u * kPfThreads] = v[u] + s;
                }
            }
            if (threadIdx.x == 0) s_rj[q] = j;
            if (j < b_abs) { moved += 1; regained += b_abs - j; }
            __syncthreads();
        }
        if ((int)threadIdx.x < nb) {
            const int r = order[q0 + threadIdx.x];
            const int j = s_rj[threadIdx.x];
            new_last[r] = j;
            new_issue[r] = j < s_rb[threadIdx.x] ? (j + 1 <= K ? start[j + 1] : start[j + 1 - K] + T) : mig[r].prefetch_issue_ns;
        }
    }
    __syncthreads();
    if (p_in_smem) for (int64_t k = threadIdx.x; k < K; k += kPfThreads) P[k] = Pw[k];
    __syncthreads();
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
        summary[0] = moved; summary[1] = regained; summary[2] = sl < 0 ? 0 : mx; summary[3] = sl; summary[4] = 0;
    }
}

// ---------------------------------------------------------------------------------------------
// The same pass for a pressure curve too long for shared memory.  The curve stays in global memory, but the block
// keeps two numbers per tile of kPfTile slots in shared memory: an upper bound of the tile's largest pressure and an
// amount still to be added to every slot of the tile.  A search walks the tiles of the range (shared memory only) and
// looks at slots only in a tile whose bound says that it may hold a slot that cannot take the tensor -- one trip to
// global memory, which also makes the tile's bound exact again; a regained range adds the tensor's size to the
// tiles it covers whole (shared memory) and to the slots of the at most two tiles it covers in part (reductions that
// nobody waits for).  The amounts still to be added go into the curve at the end.
// ---------------------------------------------------------------------------------------------
constexpr int kPfTile = 1024;                    // slots per tile
constexpr int kPfNT = 256;                       // threads of the block (few warps: the many block-wide barriers stay cheap)
constexpr int kPfMaxTiles = 8192;
constexpr int kPfBatch = 256;                    // records whose fields are fetched together

// largest of one int per thread over the block (-1 = none); `s_buf` [32], used by one call at a time between barriers
__device__ __forceinline__ int pf_block_max(int v, int *s_buf, int lane, int warp)
{
    v = (int)__reduce_max_sync(0xffffffffu, v);
    __syncthreads();                                       // (s_buf free)
    if (lane == 0) s_buf[warp] = v;
    __syncthreads();
    return (int)__reduce_max_sync(0xffffffffu, lane < kPfNT / 32 ? s_buf[lane] : -1);
}

__global__ void __launch_bounds__(kPfNT) k_schedule_prefetch_tiled(int64_t K, int64_t n, const g10_migration *__restrict__ mig,
                                                                     const int64_t *__restrict__ start, const int64_t *__restrict__ bytes,
                                                                     int64_t cap, int64_t *P, int32_t *order, int32_t *new_last,
                                                                     int64_t *new_issue, int64_t *summary, int sort_in_smem,
                                                                     const unsigned *only_if, int presorted)
{
    // (launched behind the many-block form, which leaves the records alone and sets *only_if when they need this one;
    // `order` is then already there)
    if (only_if != nullptr && *only_if == 0u) return;
    extern __shared__ long long s_dyn[];
    __shared__ int s_ra[kPfBatch], s_rb[kPfBatch], s_rj[kPfBatch];
    __shared__ long long s_rs[kPfBatch];
    __shared__ int s_red[32];
    __shared__ long long s_redl[32];
    __shared__ long long s_mx[32];
    __shared__ int s_sl[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nT = (int)((K + kPfTile - 1) / kPfTile);
    int64_t n2 = 1;
    while (n2 < n) n2 <<= 1;
    long long *tmax = s_dyn + (sort_in_smem ? (n2 * 12 + 7) / 8 : 0);      // [T] upper bound of the tile's largest pressure (amount to add included)
    long long *toff = tmax + nT;                                             // [T] still to be added to every slot of the tile
    const int64_t T = K > 0 ? start[K] : 1;
    if (!presorted) pf_order_records(n, n2, mig, order, s_dyn, sort_in_smem, kPfNT, T);
    __syncthreads();
    // ---- tile maxima, a warp per tile
    for (int t = warp; t < nT; t += kPfNT / 32) {
        long long m = -0x7fffffffffffffffll - 1;
        for (int k0 = t * kPfTile + lane; k0 < (t + 1) * kPfTile; k0 += 8 * 32) {
            long long v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = k0 + 32 * u < K ? __ldcg(&P[k0 + 32 * u]) : m;
#pragma unroll
            for (int u = 0; u < 8; ++u) if (v[u] > m) m = v[u];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { const long long x = __shfl_xor_sync(0xffffffffu, m, o); if (x > m) m = x; }
        if (lane == 0) { tmax[t] = m; toff[t] = 0; }
    }
    __syncthreads();
    long long moved = 0, regained = 0;
    for (int64_t q0 = 0; q0 < n; q0 += kPfBatch) {
        const int nb = (int)(n - q0 < kPfBatch ? n - q0 : kPfBatch);
        __syncthreads();
        if ((int)threadIdx.x < nb) {
            const int r = order[q0 + threadIdx.x];
            s_ra[threadIdx.x] = mig[r].absent_first; s_rb[threadIdx.x] = mig[r].absent_last;
            s_rs[threadIdx.x] = bytes[mig[r].tensor];
        }
        __syncthreads();
        for (int q = 0; q < nb; ++q) {
            const int ua = s_ra[q], ub = s_rb[q];              // unrolled slots; beyond K only for a steady-state plan
            const long long s = s_rs[q], lim = cap - s;        // a slot takes the tensor iff its pressure is at most lim
            int j = ua - 1;                                     // result: last slot that stays absent (unrolled)
            // the range as at most two runs of physical slots, the later one first: the part in the next iteration (slot x
            // stands for slot x - K), then the part in this one
            const int Ki = (int)K;
            int seg_lo[2], seg_hi[2], seg_off[2], nseg = 0;
            if (ub >= Ki) { seg_lo[nseg] = (ua > Ki ? ua : Ki) - Ki; seg_hi[nseg] = ub - Ki; seg_off[nseg] = Ki; ++nseg; }
            if (ua < Ki) { seg_lo[nseg] = ua; seg_hi[nseg] = ub < Ki ? ub : Ki - 1; seg_off[nseg] = 0; ++nseg; }
            bool stopped = false;
            for (int g = 0; g < nseg && !stopped; ++g) {
            const int a_abs = seg_lo[g], b_abs = seg_hi[g];
            const int lo_t = a_abs / kPfTile;
            int t_cur = b_abs / kPfTile;
            while (t_cur >= lo_t) {
                // highest tile at or below t_cur whose bound says it may hold a slot that cannot take the tensor
                int found = -1;
                for (int base = t_cur; base >= lo_t && found < 0; base -= kPfNT) {
                    const int t = base - (int)threadIdx.x;
                    found = pf_block_max((t >= lo_t && tmax[t] > lim) ? t : -1, s_red, lane, warp);
                }
                if (found < 0) break;
                // its slots: the highest one inside the range that cannot take the tensor, and the tile's exact maximum
                long long m = -0x7fffffffffffffffll - 1;
                int jt = -1;
                {
                    long long val[kPfTile / kPfNT];
                    const long long add = toff[found];
#pragma unroll
                    for (int u = 0; u < kPfTile / kPfNT; ++u) {
                        const int64_t k = (int64_t)found * kPfTile + u * kPfNT + threadIdx.x;
                        val[u] = k < K ? __ldcg(&P[k]) + add : m;   // (L2: earlier reductions are there, not in L1)
                    }
#pragma unroll
                    for (int u = 0; u < kPfTile / kPfNT; ++u) {
                        const int64_t k = (int64_t)found * kPfTile + u * kPfNT + threadIdx.x;
                        if (val[u] > m) m = val[u];
                        if (k >= a_abs && k <= b_abs && val[u] > lim) jt = (int)k;     // (k grows with u: the highest one stays)
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) { const long long x = __shfl_xor_sync(0xffffffffu, m, o); if (x > m) m = x; }
                const int jw = (int)__reduce_max_sync(0xffffffffu, jt);
                __syncthreads();                                   // (s_red, s_redl free)
                if (lane == 0) { s_red[warp] = jw; s_redl[warp] = m; }
                __syncthreads();
                const int jj = (int)__reduce_max_sync(0xffffffffu, lane < kPfNT / 32 ? s_red[lane] : -1);
                if (warp == 0) {
                    long long mm = lane < kPfNT / 32 ? s_redl[lane] : -0x7fffffffffffffffll - 1;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) { const long long x = __shfl_xor_sync(0xffffffffu, mm, o); if (x > mm) mm = x; }
                    if (lane == 0) tmax[found] = mm;
                }
                if (jj >= 0) { j = jj + seg_off[g]; stopped = true; break; }
                t_cur = found - 1;
                __syncthreads();                                   // (the refreshed bound is read by the next search)
            }
            __syncthreads();
            }
            for (int g = 0; g < nseg; ++g) {
            // the regained slots (j, ub] take the tensor back: this run's share of them
            const int b_abs = seg_hi[g];
            const int k0 = j + 1 - seg_off[g] > seg_lo[g] ? j + 1 - seg_off[g] : seg_lo[g];
            if (k0 <= b_abs) {
                const int t0 = k0 / kPfTile, t1 = b_abs / kPfTile;
                const int first_full = (k0 % kPfTile) ? t0 + 1 : t0, last_full = (b_abs % kPfTile == kPfTile - 1) ? t1 : t1 - 1;
                for (int t = first_full + (int)threadIdx.x; t <= last_full; t += kPfNT) { toff[t] += s; tmax[t] += s; }
                if (first_full > t0) {                             // the tile the range starts in, covered in part
#pragma unroll
                    for (int u = 0; u < kPfTile / kPfNT; ++u) {
                        const int64_t k = (int64_t)t0 * kPfTile + u * kPfNT + threadIdx.x;
                        if (k >= k0 && k <= b_abs) atomicAdd((ull *)&P[k], (ull)s);
                    }
                    if (threadIdx.x == 0) tmax[t0] += s;
                }
                if (last_full < t1 && (t1 > t0 || first_full == t0)) {   // the tile it ends in, covered in part (and not done above)
#pragma unroll
                    for (int u = 0; u < kPfTile / kPfNT; ++u) {
                        const int64_t k = (int64_t)t1 * kPfTile + u * kPfNT + threadIdx.x;
                        if (k >= k0 && k <= b_abs) atomicAdd((ull *)&P[k], (ull)s);
                    }
                    if (threadIdx.x == 0) tmax[t1] += s;
                }
            }
            __syncthreads();                                       // (a tile may belong to both runs)
            }
            if (j < ub) { moved += 1; regained += ub - j; }
            if (threadIdx.x == 0) s_rj[q] = j;
            __syncthreads();
        }
        if ((int)threadIdx.x < nb) {
            const int r = order[q0 + threadIdx.x];
            const int j = s_rj[threadIdx.x];
            new_last[r] = j;
            new_issue[r] = j < s_rb[threadIdx.x] ? (j + 1 <= K ? start[j + 1] : start[j + 1 - K] + T) : mig[r].prefetch_issue_ns;
        }
    }
    __syncthreads();
    // ---- what is still to be added goes into the curve; new peak and its lowest slot
    long long mx = 0;
    int sl = -1;
    for (int64_t k0 = threadIdx.x; k0 < K; k0 += 8 * kPfNT) {           // eight slots per thread in flight
        long long pv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) pv[u] = k0 + u * kPfNT < K ? __ldcg(&P[k0 + u * kPfNT]) : 0;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int64_t k = k0 + u * kPfNT;
            if (k < K) {
                const long long add = toff[k / kPfTile];
                if (add) { pv[u] += add; P[k] = pv[u]; }
                if (sl < 0 || pv[u] > mx) { mx = pv[u]; sl = (int)k; }
            }
        }
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
        for (int w = 1; w < kPfNT / 32; ++w)
            if (s_sl[w] >= 0 && (sl < 0 || s_mx[w] > mx || (s_mx[w] == mx && s_sl[w] < sl))) { mx = s_mx[w]; sl = s_sl[w]; }
        summary[0] = moved; summary[1] = regained; summary[2] = sl < 0 ? 0 : mx; summary[3] = sl; summary[4] = 0;
    }
}

// ---------------------------------------------------------------------------------------------
// The pass with many blocks.  The visits only look sequential: a visit reads and changes the pressure of the slots
// between the record's absent_first and absent_last, so records whose ranges lie apart do not see each other.  The
// timeline is cut into slices of L slots, one per block, each kept in its block's shared memory for the whole pass.
// Every block walks ALL records in visiting order and takes part in those whose range meets its slice:
//   - a search starts in the slice that holds absent_last (no waiting: that block owns the start);
//   - if every slot of the range inside the slice can take the tensor and the range goes on to the left, the
//     block adds the tensor to those slots and hands the record to the block on its left;
//   - where a slot cannot take the tensor, or the range ends, the record is finished there.
// One word per record says where its search stands: 0 = at its first slice, 2 + c = handed to block c, 1 = finished.
// A block that comes to a record whose range meets its slice further left waits until the word says "finished" (the
// search ended before it reached the slice) or names the block itself.  The record with the lowest position that is
// not yet finished is always held by a block that has nothing left to wait for, so the pass cannot lock up; every
// wait is bounded all the same.  Slices see exactly the sequence of changes the one-block pass would make.
// Records of a steady-state plan that wrap around the end of the timeline are not handled here: the preparing kernel
// then raises `fallback`, this kernel returns at once and the one-block form, launched behind it, does the pass.
// ---------------------------------------------------------------------------------------------
constexpr int kPpBatch = 512;                    // records fetched together
constexpr int kPpResults = 256;                  // finished records a block keeps before it writes them out
constexpr unsigned kPpGaveUp = 0xffffffffu;       // (in place of a record's word: the wait for it ran out)

// Visiting order by counting: the position of a record is the number of records that come before it -- earlier
// moment of the prefetch inside the iteration, or the same moment and a lower index.  Every (record, record) pair is
// compared once, by a grid of blocks that each hold one run of 2048 keys in shared memory: for the few ten thousand
// records of a plan this is a few microseconds of the whole GPU, where a sorting network in one block takes hundreds.
constexpr int kRankNT = 256, kRankChunk = 2048;
__global__ void __launch_bounds__(kRankNT) k_pf_rank(int64_t n, const g10_migration *__restrict__ mig, const int64_t *__restrict__ start,
                                                    int64_t K, unsigned *rank)
{
    __shared__ long long s_key[kRankChunk];
    const int64_t T = K > 0 ? start[K] : 1;
    const int64_t j0 = (int64_t)blockIdx.y * kRankChunk;
    const int m = (int)(n - j0 < kRankChunk ? n - j0 : kRankChunk);
    for (int x = threadIdx.x; x < m; x += kRankNT) s_key[x] = mig[j0 + x].prefetch_issue_ns % T;
    const int64_t i = (int64_t)blockIdx.x * kRankNT + threadIdx.x;
    const long long key = i < n ? mig[i].prefetch_issue_ns % T : 0;
    __syncthreads();
    if (i >= n) return;
    // records of the run below i win ties, those above lose them
    const int below = (int)(i - j0 < 0 ? 0 : (i - j0 > m ? m : i - j0));
    unsigned c = 0;
    int x = 0;
    for (; x < below; ++x) c += s_key[x] <= key ? 1u : 0u;
    for (x = below; x < m; ++x) c += s_key[x] < key ? 1u : 0u;      // (x == i - j0 is the record itself: not counted)
    if (c) atomicAdd(&rank[i], c);
}

// The records' fields, in visiting order, for every block of the pass.
__global__ void __launch_bounds__(kRankNT) k_pf_prepare(int64_t K, int64_t n, const g10_migration *__restrict__ mig,
                                                        const int64_t *__restrict__ bytes, int32_t *order, PrefetchScratch w,
                                                        int64_t *summary)
{
    const int64_t i = (int64_t)blockIdx.x * kRankNT + threadIdx.x;
    if (blockIdx.x == 0 && threadIdx.x < 5) summary[threadIdx.x] = 0;
    if (i >= n) return;
    const unsigned q = w.rank[i];
    const int a = mig[i].absent_first, b = mig[i].absent_last;
    order[q] = (int32_t)i;
    w.first[q] = a;
    w.last[q] = b;
    w.size[q] = bytes[mig[i].tensor];
    if (a < 0 || b < 0 || b >= K) *w.fallback = 1u;          // (wraps around, or nothing this form knows: one block takes the pass)
}

// A slice is kept as raw values plus one amount still to be added to all of them (`off`), with its exact largest raw
// value beside it (`rmax`), both in a register of every thread: a record that arrives from the right and whose whole
// slice can take the tensor -- the common case on the long run of a far-moving prefetch -- costs one comparison and one
// addition, no barrier, and the hand-over to the next block goes out at once.
// Where the records of a batch stand is polled for the whole batch at a time (a thread per record) and kept in shared
// memory; "finished" never changes again, so the walk skips such records without touching global memory and polls again
// only when it comes to a record that was still under way at the last poll.
template <int NT>
__global__ void __launch_bounds__(NT) k_pf_pipe(int64_t K, int64_t n, int L, const g10_migration *__restrict__ mig,
                                                const int64_t *__restrict__ start, int64_t cap, int64_t *P,
                                                const int32_t *__restrict__ order, int32_t *new_last, int64_t *new_issue,
                                                int64_t *summary, PrefetchScratch w, int hook)
{
    constexpr int kPer = kPpBatch / NT, kWarps = NT / 32;
#ifdef G10_TEST_HOOKS
    // test build: block `hook - 1` keeps every record it should hand over or finish to itself, and waits last a millisecond
    const bool mute = hook != 0 && (int)blockIdx.x == hook - 1;
    const ull wait_ns = hook != 0 ? 1000000ull : kBarrierTimeoutNs;
#else
    (void)hook;
    constexpr bool mute = false;
    constexpr ull wait_ns = kBarrierTimeoutNs;
#endif
    extern __shared__ long long Ps[];            // this block's slice of the pressure curve (raw values)
    __shared__ int s_lq[kPpBatch], s_la[kPpBatch], s_lb[kPpBatch];      // the batch's records that concern this block, in order
    __shared__ long long s_ls[kPpBatch];
    __shared__ unsigned s_st[kPpBatch];                                  // where each stood when last polled
    __shared__ int s_cnt[kPer][kWarps];
    __shared__ int s_resq[kPpResults], s_resj[kPpResults];
    __shared__ int s_wj[kWarps];
    __shared__ long long s_wmax[kWarps];
    __shared__ long long s_mx[kWarps];
    __shared__ int s_sl[kWarps];
    __shared__ int s_last;
    if (*w.fallback != 0u) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = (int)blockIdx.x, G = (int)gridDim.x;
    const int s0 = b * L, s1 = (int)((int64_t)(b + 1) * L < K ? (int64_t)(b + 1) * L : K);   // slice [s0, s1)
    const unsigned here = 2u + (unsigned)b;
    long long off = 0, rmax = -0x7fffffffffffffffll - 1;
    {
        long long m = rmax;
        for (int k = s0 + (int)threadIdx.x; k < s1; k += NT) { const long long v = P[k]; Ps[k - s0] = v; m = v > m ? v : m; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { const long long x = __shfl_xor_sync(0xffffffffu, m, o); m = x > m ? x : m; }
        if (lane == 0) s_wmax[warp] = m;
        __syncthreads();
        for (int x = 0; x < kWarps; ++x) rmax = s_wmax[x] > rmax ? s_wmax[x] : rmax;
        __syncthreads();
    }
    long long moved = 0, regained = 0;           // (thread 0's count)
    int nres = 0;
    bool dead = false;                           // a wait ran out: nothing more is visited
    auto flush_results = [&]() {                 // the finished records kept so far go to the outputs
        __syncthreads();
        for (int e = threadIdx.x; e < nres; e += NT) {
            const int q = s_resq[e], j = s_resj[e];
            const int r = order[q];
            new_last[r] = j;
            new_issue[r] = j < w.last[q] ? start[j + 1] : mig[r].prefetch_issue_ns;
        }
        __syncthreads();
        nres = 0;
    };
    for (int64_t q0 = 0; q0 < n && !dead; q0 += kPpBatch) {
        // ---- the batch's records whose range meets this slice and that are not finished yet, kept in order
        int qa[kPer], qb[kPer];
        long long qs[kPer];
        unsigned qw[kPer];
        bool keep[kPer];
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const int64_t q = q0 + u * NT + threadIdx.x;
            keep[u] = false;
            if (q < n) {
                qa[u] = w.first[q];
                qb[u] = w.last[q];
                // mine from the start (absent_last in the slice), or the range passes absent_last's slice and reaches this one
                const bool own = qb[u] >= s0 && qb[u] < s1;
                keep[u] = own || (qb[u] >= s1 && qa[u] < s1 && qa[u] <= qb[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const int64_t q = q0 + u * NT + threadIdx.x;
            qw[u] = 0u;
            if (keep[u]) {
                qs[u] = w.size[q];
                if (qb[u] >= s1) {
                    qw[u] = ld_relaxed_u32(&w.word[q]);
                    if (qw[u] == 1u) keep[u] = false;            // finished before it came here
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const unsigned m = __ballot_sync(0xffffffffu, keep[u]);
            if (lane == 0) s_cnt[u][warp] = __popc(m);
        }
        __syncthreads();
        int cnt = 0;
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const unsigned m = __ballot_sync(0xffffffffu, keep[u]);
            int pos = cnt;
            for (int x = 0; x < kWarps; ++x) {
                const int c = s_cnt[u][x];
                if (x < warp) pos += c;
                cnt += c;
            }
            if (keep[u]) {
                pos += __popc(m & ((1u << lane) - 1u));
                s_lq[pos] = (int)(q0 + u * NT + threadIdx.x);
                s_la[pos] = qa[u]; s_lb[pos] = qb[u]; s_ls[pos] = qs[u]; s_st[pos] = qw[u];
            }
        }
        __syncthreads();
        // ---- their visits, one after the other
        int e = 0;
        while (e < cnt) {
            unsigned st = s_st[e];
            if (st == 1u) { ++e; continue; }
            const int q = s_lq[e], ua = s_la[e], ub = s_lb[e];
            const bool own = ub < s1;
            if (!own && st != here) {
                // under way when last polled: poll this one and those behind it again, all at once
                __syncthreads();                                 // (every thread has read s_st[e])
                for (int x = e + (int)threadIdx.x; x < cnt; x += NT)
                    if (s_lb[x] >= s1 && s_st[x] != 1u) s_st[x] = ld_relaxed_u32(&w.word[s_lq[x]]);
                __syncthreads();
                st = s_st[e];
                if (st != 1u && st != here) {                    // still under way: thread 0 waits for it
                    __syncthreads();
                    if (threadIdx.x == 0) {
                        const ull t0 = global_timer_ns();
                        unsigned polls = 0, v;
                        while (true) {
                            v = ld_relaxed_u32(&w.word[q]);
                            if (v == 1u || v == here) break;
                            // (every so often: out of time, or another block has given up -- then this wait is in vain too)
                            if ((++polls & 255u) == 0u && (global_timer_ns() - t0 > wait_ns || *(volatile ull *)w.status != 0)) {
                                raise_status(w.status, G10_DEV_TIMEOUT);
                                v = kPpGaveUp;
                                break;
                            }
                        }
                        s_st[e] = v;
                    }
                    __syncthreads();
                    st = s_st[e];
                    if (st == kPpGaveUp) { dead = true; break; }
                }
                if (st == 1u) { ++e; continue; }
            }
            // ---- the record is this block's to visit
            const long long s = s_ls[e], lim = cap - s;          // a slot takes the tensor iff its pressure is at most lim
            ++e;
            if (!own && ua <= s0 && rmax + off <= lim) {
                // it covers the whole slice and all of it takes the tensor
                off += s;
                if (ua < s0) {
                    if (threadIdx.x == 0 && !mute) st_relaxed_u32(&w.word[q], here - 1u);
                } else {                                         // the range ends with the slice's first slot
                    if (threadIdx.x == 0) {
                        s_resq[nres] = q; s_resj[nres] = ua - 1;
                        if (!mute) st_relaxed_u32(&w.word[q], 1u);
                        moved += 1; regained += ub - (ua - 1);
                    }
                    if (++nres == kPpResults) flush_results();
                }
                continue;
            }
            const int lo = ua > s0 ? ua : s0, hi = ub < s1 ? ub : s1 - 1;
            const long long liml = lim - off;                    // the same test on raw values
            // highest slot of [lo, hi] that cannot take the tensor
            int jt = -1;
            for (int k = hi - (int)threadIdx.x; k >= lo; k -= 4 * NT) {          // four slots per thread in flight
                long long v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) v[u] = k - u * NT >= lo ? Ps[k - u * NT - s0] : liml;
                int hit = -1;
#pragma unroll
                for (int u = 3; u >= 0; --u) hit = v[u] > liml ? k - u * NT : hit;     // (the highest one stays)
                if (hit >= 0) { jt = hit; break; }
            }
            jt = (int)__reduce_max_sync(0xffffffffu, jt);
            if (lane == 0) s_wj[warp] = jt;
            __syncthreads();
            int j = s_wj[0];
#pragma unroll
            for (int x = 1; x < kWarps; ++x) j = s_wj[x] > j ? s_wj[x] : j;
            const bool ends = j >= 0 || ua >= s0;                // blocked here, or the range ends in this slice
            const int jf = j >= 0 ? j : (ua - 1 < ub ? ua - 1 : ub);         // (if it ends) last slot that stays absent
            if (threadIdx.x == 0) {                              // (the word first: a block may be waiting for it)
                if (ends) {
                    if (!mute) st_relaxed_u32(&w.word[q], 1u);
                    s_resq[nres] = q; s_resj[nres] = jf;
                    if (jf < ub) { moved += 1; regained += ub - jf; }
                } else {
                    if (!mute) st_relaxed_u32(&w.word[q], here - 1u);
                }
            }
            // the regained slots (j, hi] take the tensor; the slice's largest raw value afterwards
            const int from = j >= 0 ? j + 1 : lo;
            long long m = -0x7fffffffffffffffll - 1;
            for (int k = s0 + (int)threadIdx.x; k < s1; k += 4 * NT) {
                long long v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) v[u] = k + u * NT < s1 ? Ps[k + u * NT - s0] : m;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int kk = k + u * NT;
                    if (kk >= from && kk <= hi && kk < s1) { v[u] += s; Ps[kk - s0] = v[u]; }
                    m = v[u] > m ? v[u] : m;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) { const long long x = __shfl_xor_sync(0xffffffffu, m, o); m = x > m ? x : m; }
            if (lane == 0) s_wmax[warp] = m;
            __syncthreads();                                     // (the slice as the next visit must see it; s_wj free)
            rmax = s_wmax[0];
#pragma unroll
            for (int x = 1; x < kWarps; ++x) rmax = s_wmax[x] > rmax ? s_wmax[x] : rmax;
            if (ends && ++nres == kPpResults) flush_results();
        }
    }
    flush_results();
    // ---- the slice goes back; its largest pressure and lowest such slot; the last block to finish takes the overall peak
    long long mx = 0;
    int sl = -1;
    for (int k = s0 + (int)threadIdx.x; k < s1; k += NT) {
        const long long pv = Ps[k - s0] + off;
        P[k] = pv;
        if (sl < 0 || pv > mx) { mx = pv; sl = k; }
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
        for (int x = 1; x < kWarps; ++x)
            if (s_sl[x] >= 0 && (sl < 0 || s_mx[x] > mx || (s_mx[x] == mx && s_sl[x] < sl))) { mx = s_mx[x]; sl = s_sl[x]; }
        w.block_max[b] = mx;
        w.block_slot[b] = sl;
        if (moved) atomicAdd((ull *)&summary[0], (ull)moved);
        if (regained) atomicAdd((ull *)&summary[1], (ull)regained);
        if (dead) raise_status(w.status, G10_DEV_TIMEOUT);
        __threadfence();
        s_last = atomicAdd(w.ticket, 1u) == (unsigned)(G - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    mx = 0;
    sl = -1;
    for (int x = threadIdx.x; x < G; x += NT) {
        const long long omx = __ldcg(&w.block_max[x]);
        const int osl = __ldcg(&w.block_slot[x]);
        if (osl >= 0 && (sl < 0 || omx > mx || (omx == mx && osl < sl))) { mx = omx; sl = osl; }
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
        for (int x = 1; x < kWarps; ++x)
            if (s_sl[x] >= 0 && (sl < 0 || s_mx[x] > mx || (s_mx[x] == mx && s_sl[x] < sl))) { mx = s_mx[x]; sl = s_sl[x]; }
        summary[2] = sl < 0 ? 0 : mx;
        summary[3] = sl;
        summary[4] = (int64_t)*(volatile ull *)w.status;
    }
}

// Blocks, block width and slice length of the many-block form for a timeline of K slots, or false if no choice keeps
// every slice in shared memory with all blocks resident at once (the blocks wait for one another: a cooperative launch).
// Many short slices are tried first (four blocks per SM measured fastest on the stress trace: a visit that has to look at
// the slots costs time in proportion to the slice, a hand-over to the next block only a round trip through the L2).
static const void *pf_pipe_kernel(int per_sm)
{
    return per_sm == 1 ? (const void *)k_pf_pipe<512> : per_sm == 2 ? (const void *)k_pf_pipe<256> : (const void *)k_pf_pipe<128>;
}
static bool pf_pipe_geometry(int64_t K, int *blocks, int *slice, int *per_sm_out)
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return false;
    for (int per_sm = 4; per_sm >= 1; per_sm >>= 1) {
        int64_t G = (int64_t)sms * per_sm;
        if (G > kPfMaxBlocks) continue;
        int64_t L = ((K + G - 1) / G + 31) / 32 * 32;
        if (L < 256) L = 256;
        G = (K + L - 1) / L;
        const size_t dyn = (size_t)L * 8;
        if (dyn > 200 * 1024) continue;
        const void *f = pf_pipe_kernel(per_sm);
        if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess) return false;
        int occ = 0;
        const int nt = per_sm == 1 ? 512 : per_sm == 2 ? 256 : 128;
        cudaError_t e = per_sm == 1   ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_pf_pipe<512>, nt, dyn)
                        : per_sm == 2 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_pf_pipe<256>, nt, dyn)
                                      : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_pf_pipe<128>, nt, dyn);
        if (e != cudaSuccess) return false;
        if ((int64_t)occ * sms >= G) { *blocks = (int)G; *slice = (int)L; *per_sm_out = per_sm; return true; }
    }
    return false;
}

cudaError_t launch_schedule_prefetch(int64_t K, int64_t n, const g10_migration *mig, const int64_t *start, const int64_t *bytes,
                                     uint64_t gpu_capacity_bytes, int64_t *P, int32_t *order, int32_t *new_last, int64_t *new_issue,
                                     int64_t *summary, const PrefetchScratch &scratch, cudaStream_t s)
{
    int64_t cap = gpu_capacity_bytes >= ((uint64_t)1 << 63) ? INT64_MAX : (int64_t)gpu_capacity_bytes;
    // the pressure curve in shared memory if it fits beside the kernel's own arrays
    size_t dyn = 0;
    int in_smem = 0;
    if (K > 0 && (size_t)K * 8 <= 120 * 1024) { dyn = (size_t)K * 8; in_smem = 1; }
    int64_t n2 = 1;
    while (n2 < n) n2 <<= 1;
    int sort_smem = 0;
    if (n > 0 && (size_t)n2 * 12 <= 64 * 1024) { dyn += (size_t)n2 * 12; sort_smem = 1; }
    const int64_t tiles = (K + kPfTile - 1) / kPfTile;
    if (in_smem || n == 0) {
        if (dyn > 0) {
            const cudaError_t e = cudaFuncSetAttribute(k_schedule_prefetch<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
            if (e != cudaSuccess) return e;
        }
        k_schedule_prefetch<256><<<1, 256, dyn, s>>>(K, n, mig, start, bytes, cap, P, order, new_last, new_issue, summary, in_smem, sort_smem); count_launch();
        return cudaGetLastError();
    }
    int G = 0, L = 0, per_sm = 0;
    const unsigned *only_if = nullptr;
    int presorted = 0;
    // (the visiting order by counting compares all pairs of records: fine for the tens of thousands of a plan, too slow
    // far beyond that)
    constexpr int64_t kPfMaxRanked = 262144;
    if (scratch.word != nullptr && n <= kPfMaxRanked && tiles <= kPfMaxTiles && pf_pipe_geometry(K, &G, &L, &per_sm)) {
        // many blocks, one slice of the timeline each; behind them the one-block form, which runs only if the records ask for it
        k_pf_rank<<<dim3((unsigned)((n + kRankNT - 1) / kRankNT), (unsigned)((n + kRankChunk - 1) / kRankChunk)), kRankNT, 0, s>>>(n, mig, start, K, scratch.rank); count_launch();
        k_pf_prepare<<<(unsigned)((n + kRankNT - 1) / kRankNT), kRankNT, 0, s>>>(K, n, mig, bytes, order, scratch, summary); count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        int Li = L;
        PrefetchScratch w = scratch;
        int hook = 0;
#ifdef G10_TEST_HOOKS
        if (const char *h = getenv("G10_TEST_PREFETCH_MUTE_BLOCK")) hook = atoi(h) + 1;
#endif
        void *args[] = {&K, &n, &Li, &mig, &start, &cap, &P, &order, &new_last, &new_issue, &summary, &w, &hook};
        e = cudaLaunchCooperativeKernel(pf_pipe_kernel(per_sm), dim3(G), dim3(per_sm == 1 ? 512 : per_sm == 2 ? 256 : 128), args, (size_t)L * 8, s);
        if (e != cudaSuccess) return e;
        only_if = scratch.fallback;
        presorted = 1;
    }
    if (tiles <= kPfMaxTiles) {
        sort_smem = (!presorted && (size_t)n2 * 12 + (size_t)tiles * 16 <= 200 * 1024) ? 1 : 0;   // (this kernel has most of the SM's shared memory to itself)
        dyn = (sort_smem ? ((size_t)n2 * 12 + 7) / 8 * 8 : 0) + (size_t)tiles * 16;
        const cudaError_t e = cudaFuncSetAttribute(k_schedule_prefetch_tiled, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
        if (e != cudaSuccess) return e;
        k_schedule_prefetch_tiled<<<1, kPfNT, dyn, s>>>(K, n, mig, start, bytes, cap, P, order, new_last, new_issue, summary, sort_smem, only_if, presorted); count_launch();
    } else {
        if (dyn > 0) {
            const cudaError_t e = cudaFuncSetAttribute(k_schedule_prefetch<1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
            if (e != cudaSuccess) return e;
        }
        k_schedule_prefetch<1024><<<1, 1024, dyn, s>>>(K, n, mig, start, bytes, cap, P, order, new_last, new_issue, summary, in_smem, sort_smem); count_launch();
    }
    return cudaGetLastError();
}

}  // namespace g10

// Smart tensor prefetching (Section 4.4): after the eviction plan is made, the evicted periods are visited in
// the order of their latest safe prefetch time and every prefetch is moved back to the earliest slot from which
// the GPU can hold the tensor with the space that is left; the pressure curve is updated as it goes.
//
// The pass is a strict sequence over the plan records (each move changes the pressure the next search sees), so
// one block does it: the records are ordered by a bitonic network over their indices, then, record by record, the
// block searches backward in chunks of eight times its own width (a chunk stops the search as soon as one of its
// slots cannot take the tensor) and adds the tensor's size to the slots it regained.  Parallelism is inside each search.
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
                for (int64_t t = threadIdx.x; t < n2 / 2; t += nthreads) {
                    const int64_t blk = t / j, off = t % j;
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
                for (int64_t t = threadIdx.x; t < n2 / 2; t += nthreads) {
                    const int64_t blk = t / j, off = t % j;
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
        summary[0] = moved; summary[1] = regained; summary[2] = sl < 0 ? 0 : mx; summary[3] = sl;
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
                                                                     int64_t *new_issue, int64_t *summary, int sort_in_smem)
{
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
    pf_order_records(n, n2, mig, order, s_dyn, sort_in_smem, kPfNT, T);
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
        summary[0] = moved; summary[1] = regained; summary[2] = sl < 0 ? 0 : mx; summary[3] = sl;
    }
}

cudaError_t launch_schedule_prefetch(int64_t K, int64_t n, const g10_migration *mig, const int64_t *start, const int64_t *bytes,
                                     uint64_t gpu_capacity_bytes, int64_t *P, int32_t *order, int32_t *new_last, int64_t *new_issue,
                                     int64_t *summary, cudaStream_t s)
{
    const int64_t cap = gpu_capacity_bytes >= ((uint64_t)1 << 63) ? INT64_MAX : (int64_t)gpu_capacity_bytes;
    // the pressure curve in shared memory if it fits beside the kernel's own arrays
    size_t dyn = 0;
    int in_smem = 0;
    if (K > 0 && (size_t)K * 8 <= 120 * 1024) { dyn = (size_t)K * 8; in_smem = 1; }
    int64_t n2 = 1;
    while (n2 < n) n2 <<= 1;
    int sort_smem = 0;
    if (n > 0 && (size_t)n2 * 12 <= 64 * 1024) { dyn += (size_t)n2 * 12; sort_smem = 1; }
    const int64_t tiles = (K + kPfTile - 1) / kPfTile;
    if (in_smem) {
        if (dyn > 0) {
            const cudaError_t e = cudaFuncSetAttribute(k_schedule_prefetch<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
            if (e != cudaSuccess) return e;
        }
        k_schedule_prefetch<256><<<1, 256, dyn, s>>>(K, n, mig, start, bytes, cap, P, order, new_last, new_issue, summary, in_smem, sort_smem); count_launch();
    } else if (tiles <= kPfMaxTiles) {
        sort_smem = (n > 0 && (size_t)n2 * 12 + (size_t)tiles * 16 <= 200 * 1024) ? 1 : 0;   // (this kernel has most of the SM's shared memory to itself)
        dyn = (sort_smem ? ((size_t)n2 * 12 + 7) / 8 * 8 : 0) + (size_t)tiles * 16;
        const cudaError_t e = cudaFuncSetAttribute(k_schedule_prefetch_tiled, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
        if (e != cudaSuccess) return e;
        k_schedule_prefetch_tiled<<<1, kPfNT, dyn, s>>>(K, n, mig, start, bytes, cap, P, order, new_last, new_issue, summary, sort_smem); count_launch();
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

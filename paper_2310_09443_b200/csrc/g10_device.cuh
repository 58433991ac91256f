// Device-side building blocks shared by the passes: acquire/release accesses, bounded waits,
// warp/block reductions, the single-pass (decoupled look-back) scan state and a bounded grid barrier.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "g10.h"

namespace g10 {

typedef unsigned __int128 u128;
typedef unsigned long long ull;

constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;
constexpr int kScanTile = kScanThreads * kScanItems;   // 2048 items per tile
constexpr unsigned kSpinLimit = 1u << 24;               // polls before a wait gives up
constexpr ull kBarrierTimeoutNs = 4000000000ull;        // 4 s

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(unsigned *p, unsigned v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// (relaxed forms: for a word that is itself all that is handed over -- no other memory is published with it)
__device__ __forceinline__ unsigned ld_relaxed_u32(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u32(unsigned *p, unsigned v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ ull global_timer_ns()
{
    ull t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void raise_status(ull *status, ull bits) { atomicOr(status, bits); }

__device__ __forceinline__ long long warp_sum_i64(long long v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;   // valid in lane 0
}
__device__ __forceinline__ long long warp_inclusive_scan_i64(long long v, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        long long n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
    }
    return v;
}
__device__ __forceinline__ u128 warp_sum_u128(u128 v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ull lo = __shfl_down_sync(0xffffffffu, (ull)v, o);
        ull hi = __shfl_down_sync(0xffffffffu, (ull)(v >> 64), o);
        v += ((u128)hi << 64) | lo;
    }
    return v;   // valid in lane 0
}

// ---------------------------------------------------------------------------------------------
// Single-pass scan with decoupled look-back.  One TileState per scan; flag[t]: 0 = nothing yet,
// 1 = the tile's own aggregate is published, 2 = its inclusive prefix is published.  Tiles are
// handed out by an atomic ticket so that every predecessor of a running tile has started.
// NV is the number of int64 running sums carried together (1, or 2 for the fused vitality pass).
// ---------------------------------------------------------------------------------------------
template <int NV>
struct TileState {
    unsigned *ticket;     // [1]
    unsigned *flag;       // [tiles]
    long long *agg;       // [tiles * NV]
    long long *incl;      // [tiles * NV]
};

template <int NV>
struct Sums {
    long long v[NV];
};

// Called by all 32 lanes of one warp.  Publishes `mine` for `tile`, walks back over the predecessors
// and returns the exclusive prefix of the tile (same value in every lane), then publishes the
// inclusive prefix.  A predecessor that never shows up makes the wait give up after kSpinLimit polls:
// the status word gets G10_DEV_TIMEOUT and the prefix is garbage (the caller's outputs stay in bounds).
template <int NV>
__device__ Sums<NV> lookback_exclusive(const TileState<NV> &st, int tile, Sums<NV> mine, int lane, ull *status)
{
    if (lane == 0) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            st.agg[(size_t)tile * NV + j] = mine.v[j];
            if (tile == 0) st.incl[j] = mine.v[j];
        }
        st_release_u32(&st.flag[tile], tile == 0 ? 2u : 1u);
    }
    Sums<NV> excl;
#pragma unroll
    for (int j = 0; j < NV; ++j) excl.v[j] = 0;
    if (tile == 0) return excl;
    int base = tile - 1;
    for (;;) {
        int t = base - lane;
        unsigned f = 3u;   // "before the first tile": contributes nothing and ends the walk
        if (t >= 0) {
            unsigned polls = 0;
            f = ld_acquire_u32(&st.flag[t]);
            while (f == 0u) {
                if (++polls > kSpinLimit) { raise_status(status, G10_DEV_TIMEOUT); f = 3u; break; }
                __nanosleep(20);
                f = ld_acquire_u32(&st.flag[t]);
            }
        }
        unsigned m = __ballot_sync(0xffffffffu, f >= 2u);
        int stop = m ? (__ffs(m) - 1) : 32;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            long long v = 0;
            if (lane < stop) v = __ldcg(&st.agg[(size_t)t * NV + j]);
            else if (lane == stop && f == 2u) v = __ldcg(&st.incl[(size_t)t * NV + j]);
            v = warp_sum_i64(v);
            excl.v[j] += __shfl_sync(0xffffffffu, v, 0);
        }
        if (m) break;
        base -= 32;
    }
    if (lane == 0) {
#pragma unroll
        for (int j = 0; j < NV; ++j) st.incl[(size_t)tile * NV + j] = excl.v[j] + mine.v[j];
        st_release_u32(&st.flag[tile], 2u);
    }
    return excl;
}

// Block-wide exclusive scan of one value per thread (kScanThreads threads) plus the tile's global
// exclusive prefix from the look-back.  Returns this thread's exclusive prefix INCLUDING the tile
// prefix; *tile_total_out gets the running total after this tile (valid in all threads).
template <int NV>
__device__ Sums<NV> block_exclusive_with_lookback(const TileState<NV> &st, int tile, Sums<NV> thread_sum,
                                                  ull *status, Sums<NV> *incl_total_out)
{
    __shared__ long long s_warp[NV][kScanThreads / 32];
    __shared__ long long s_tile_excl[NV];
    __shared__ long long s_tile_sum[NV];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    Sums<NV> incl;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        incl.v[j] = warp_inclusive_scan_i64(thread_sum.v[j], lane);
        if (lane == 31) s_warp[j][warp] = incl.v[j];
    }
    __syncthreads();
    if (warp == 0) {
        Sums<NV> mine;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            long long w = lane < kScanThreads / 32 ? s_warp[j][lane] : 0;
            long long wi = warp_inclusive_scan_i64(w, lane);
            if (lane < kScanThreads / 32) s_warp[j][lane] = wi - w;   // exclusive prefix of each warp
            mine.v[j] = __shfl_sync(0xffffffffu, wi, 31);
        }
        Sums<NV> ex = lookback_exclusive<NV>(st, tile, mine, lane, status);
        if (lane == 0) {
#pragma unroll
            for (int j = 0; j < NV; ++j) { s_tile_excl[j] = ex.v[j]; s_tile_sum[j] = mine.v[j]; }
        }
    }
    __syncthreads();
    Sums<NV> out;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        out.v[j] = s_tile_excl[j] + s_warp[j][warp] + incl.v[j] - thread_sum.v[j];
        incl_total_out->v[j] = s_tile_excl[j] + s_tile_sum[j];
    }
    return out;
}

// Hands out tile numbers in launch-independent order.
__device__ __forceinline__ int next_tile(unsigned *ticket)
{
    __shared__ int s_tile;
    __syncthreads();
    if (threadIdx.x == 0) s_tile = (int)atomicAdd(ticket, 1u);
    __syncthreads();
    return s_tile;
}


// ---------------------------------------------------------------------------------------------
// Candidate geometry of one inactive period (Algorithm 1 / Section 4.4) for one destination.
// ---------------------------------------------------------------------------------------------
// Time to move `bytes` at `bw` bytes per second, in ns, rounded up; saturates at 2^62.
__device__ __forceinline__ int64_t transfer_time_ns(int64_t bytes, uint64_t bw)
{
    const u128 num = (u128)(uint64_t)bytes * (u128)1000000000ull;
    u128 q = num / (u128)bw;
    if (q * (u128)bw != num) q += 1;
    const u128 sat = (u128)1 << 62;
    return (int64_t)(q > sat ? sat : q);
}

// Period between uses u and v of a tensor of s bytes; `start` is the slot clock (global or shared memory).
// The eviction occupies [t_r, t_r + t) from the period's start, the prefetch [t_end - t, t_end) up to its end;
// the tensor is absent in the slots that lie wholly between the two.  (-1, -2) when they leave no such slot.
__device__ __forceinline__ void period_geometry(const int64_t *start, int u, int v, int64_t s, uint64_t bw, int64_t *t_out,
                                                int *a_abs_out, int *b_abs_out)
{
    const int64_t t_r = start[u + 1], t_end = start[v], L = t_end - t_r;
    const int64_t t = transfer_time_ns(s, bw);
    int a_abs = -1, b_abs = -2;
    if (t <= L && 2 * t <= L) {
        // first k in [u+1, v] with start[k] >= t_r + t   (start[v] = t_end > t_r + t - 1 always qualifies)
        int lo = u + 1, hi = v;
        const int64_t ev_end = t_r + t;
        while (lo < hi) { const int mid = lo + (hi - lo) / 2; if (start[mid] >= ev_end) hi = mid; else lo = mid + 1; }
        const int ap = lo;
        // last j in [u+1, v] with start[j] <= t_end - t   (start[u+1] = t_r qualifies)
        lo = u + 1; hi = v;
        const int64_t pf_beg = t_end - t;
        while (lo < hi) { const int mid = lo + (hi - lo + 1) / 2; if (start[mid] <= pf_beg) lo = mid; else hi = mid - 1; }
        const int bp = lo - 1;
        if (ap <= bp) { a_abs = ap; b_abs = bp; }
    }
    *t_out = t; *a_abs_out = a_abs; *b_abs_out = b_abs;
}

// ---------------------------------------------------------------------------------------------
// Grid barrier for the persistent planner kernel (launched cooperatively, so all blocks are
// resident).  Sense comes from a generation counter.  A wait that lasts longer than
// kBarrierTimeoutNs sets `error`; from then on every barrier returns false at once and the
// kernel winds down.
// ---------------------------------------------------------------------------------------------
struct GridBarrier {
    unsigned count;
    unsigned gen;
    unsigned error;
    unsigned pad;
};

__device__ __forceinline__ bool grid_barrier(GridBarrier *b, unsigned nblocks, unsigned &my_gen)
{
    __shared__ unsigned s_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        // (no look at the error word before arriving: a block that arrives after another one gave up finds the word
        // set at its next check while polling, which costs one round trip less on every barrier that succeeds)
        unsigned ok = 1u;
        ull limit_ns = kBarrierTimeoutNs;
        bool arrive = true;
#ifdef G10_TEST_HOOKS
        // Test build only: in a call made with G10_FLAG_TEST_SKIP_ARRIVAL block (pad - 1) never arrives at a barrier (its
        // own barrier calls fail at once) and every wait of the call gives up after a millisecond: the other blocks find
        // that nobody completes the barrier, set the error word, and the kernel winds down with G10_DEV_TIMEOUT.
        const unsigned hook = *(volatile unsigned *)&b->pad;
        if (hook) {
            limit_ns = 1000000ull;
            if (blockIdx.x == hook - 1u) { arrive = false; ok = 0u; }
        }
#endif
        // arrival is an acquire-release add (it publishes this block's writes, ordered before it by the block barrier
        // above, and the last arrival has acquired everyone's); the generation is stored with release and polled with
        // acquire: no separate fences
        unsigned arrived = 0u;
        if (arrive) asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(arrived) : "l"(&b->count) : "memory");
        if (!arrive) {
            // (test build: this block does not arrive; ok is already 0)
        } else if (arrived == nblocks - 1u) {
            b->count = 0u;
            st_release_u32(&b->gen, my_gen + 1u);
        } else {
            ull t0 = global_timer_ns();
            unsigned polls = 0;
            while (ld_acquire_u32(&b->gen) == my_gen) {
                if ((++polls & 1023u) == 0u) {
                    if (ld_acquire_u32(&b->error)) { ok = 0u; break; }
                    if (global_timer_ns() - t0 > limit_ns) { atomicExch(&b->error, 1u); ok = 0u; break; }
                }
            }
        }
        s_ok = ok;
    }
    my_gen += 1u;
    __syncthreads();
    return s_ok != 0u;
}

}  // namespace g10

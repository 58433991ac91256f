// Pieces shared by the two planner kernels (Algorithm 1): arguments, exact candidate comparison,
// channel-window test, scoring of one period, commit of a winner and the final summary.
#pragma once
#include "g10_device.cuh"
#include "g10_internal.h"

namespace g10 {

constexpr int kPlanThreads = 512;
constexpr int kPlanWarps = kPlanThreads / 32;
constexpr int kSlotTile = 1024;            // slots are owned by blocks in tiles of this size (round robin)

struct PlanArgs {
    int64_t K;
    const int64_t *Pn_dev;                 // number of periods (device)
    int64_t geo_stride;
    const int64_t *start, *dur, *bytes;
    const int32_t *per_t, *per_u, *per_v;
    const int64_t *geo_t;
    const int32_t *geo_a, *geo_b;
    int64_t *P;                            // pressure, updated in place (= final_pressure)
    int64_t *busy;                         // [4][K]: SSD out, SSD in, host out, host in
    int64_t *hocc;                         // [K]
    unsigned char *dead;                   // period erased (committed, or no destination can ever take it)
    int64_t cap;
    int fits_always;
    uint64_t host_capacity;
    int64_t max_iterations;
    g10_migration *out;
    int64_t out_cap;
    int64_t *summary;
    Proposal *proposals;
    int64_t *peak_part;
    int *peak_key;
    GridBarrier *bar;
    ull *status;
};

struct Cand {
    u128 ben;
    ull cost;
    int idx;     // -1 = none
    int dest;
};

// a beats b: higher benefit/cost (exact, 128-bit cross products), ties to the lower period index
__device__ __forceinline__ bool cand_beats(const Cand &a, const Cand &b)
{
    if (a.idx < 0) return false;
    if (b.idx < 0) return true;
    if (a.ben == b.ben && a.cost == b.cost) return a.idx < b.idx;      // (repeated layers: identical scores are common)
    const u128 l = a.ben * (u128)b.cost, r = b.ben * (u128)a.cost;
    if (l != r) return l > r;
    return a.idx < b.idx;
}

__device__ __forceinline__ Cand cand_shfl_down(const Cand &c, int o)
{
    Cand r;
    const ull lo = __shfl_down_sync(0xffffffffu, (ull)c.ben, o);
    const ull hi = __shfl_down_sync(0xffffffffu, (ull)(c.ben >> 64), o);
    r.ben = ((u128)hi << 64) | lo;
    r.cost = __shfl_down_sync(0xffffffffu, c.cost, o);
    r.idx = __shfl_down_sync(0xffffffffu, c.idx, o);
    r.dest = __shfl_down_sync(0xffffffffu, c.dest, o);
    return r;
}

__device__ __forceinline__ Cand cand_shfl_xor(const Cand &c, int o)
{
    Cand r;
    const ull lo = __shfl_xor_sync(0xffffffffu, (ull)c.ben, o);
    const ull hi = __shfl_xor_sync(0xffffffffu, (ull)(c.ben >> 64), o);
    r.ben = ((u128)hi << 64) | lo;
    r.cost = __shfl_xor_sync(0xffffffffu, c.cost, o);
    r.idx = __shfl_xor_sync(0xffffffffu, c.idx, o);
    r.dest = __shfl_xor_sync(0xffffffffu, c.dest, o);
    return r;
}

// Is the channel free for the window [w0, w1) over slots k0..k1?  Each slot offers dur[k] ns of channel
// time per device and direction; the window may be booked iff booked + overlap <= dur in every slot.
// Called by a whole warp; returns the same answer in every lane.
// kCyclic (steady-state planning): slot indices and A.start are unrolled over two iterations, while pressure, bookings,
// host occupancy and durations belong to the physical slot (index - K beyond the first iteration).
template <bool kCyclic>
__device__ __forceinline__ int phys_slot(int64_t K, int k) { return kCyclic && k >= K ? k - (int)K : k; }

template <bool kCyclic = false>
__device__ __forceinline__ bool window_free(const PlanArgs &A, const int64_t *busy, int64_t w0, int64_t w1, int k0, int k1, int lane)
{
    bool ok = true;
    for (int k = k0 + lane; k <= k1; k += 32) {
        const int64_t s0 = A.start[k], s1 = A.start[k + 1];
        const int64_t lo = w0 > s0 ? w0 : s0, hi = w1 < s1 ? w1 : s1;
        const int64_t ov = hi > lo ? hi - lo : 0;
        if (busy[phys_slot<kCyclic>(A.K, k)] + ov > s1 - s0) ok = false;
    }
    return __all_sync(0xffffffffu, ok);
}

// A window [w0, w1) over slots wk0..wk1 is booked on a channel.  Can another window [q0, q1) over slots qk0..qk1,
// admissible before, still be booked on it?  Only slots of both windows matter.  A slot strictly inside the booking is
// full (it takes the slot's whole duration) and every slot of q's range needs time; so q survives only if the ranges
// meet in the booking's first / last slot alone and the sums still fit there.
// kBooked: `busy` already includes the booking (else its share of the slot is added here).  kL2: read busy at L2.
template <bool kBooked, bool kL2>
__device__ __forceinline__ bool window_conflict(const int64_t *start, const int64_t *busy, int wk0, int wk1, int64_t w0, int64_t w1,
                                                int64_t q0, int64_t q1, int qk0, int qk1, int Kc = 0 /* physical slots, if the indices are unrolled */)
{
    const int i0 = qk0 > wk0 ? qk0 : wk0, i1 = qk1 < wk1 ? qk1 : wk1;
    if (i0 > i1) return false;
    if ((i0 > wk0 + 1 ? i0 : wk0 + 1) <= (i1 < wk1 - 1 ? i1 : wk1 - 1)) return true;
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int k = e == 0 ? i0 : i1;
        if (e == 1 && i1 == i0) break;
        const int64_t s0 = start[k], s1 = start[k + 1];
        const int64_t lo = q0 > s0 ? q0 : s0, hi = q1 < s1 ? q1 : s1;
        int64_t need = hi > lo ? hi - lo : 0;
        if (!kBooked) {
            const int64_t wl = w0 > s0 ? w0 : s0, wh = w1 < s1 ? w1 : s1;
            need += wh > wl ? wh - wl : 0;
        }
        const int kp = Kc && k >= Kc ? k - Kc : k;
        const int64_t booked = kL2 ? __ldcg(&busy[kp]) : busy[kp];
        if (booked + need > s1 - s0) return true;
    }
    return false;
}

// Pressure tiles: 32 consecutive slots with their smallest and largest pressure.  A tile wholly at least s above the
// capacity counts s for its whole time in a benefit, one wholly within capacity nothing; only the others are read.
constexpr int kTileO = 32;

// smallest / largest pressure of tile t, by one warp (pressures are never negative: compared as unsigned halves)
__device__ __forceinline__ void tile_refresh_warp(const int64_t *sP, int K, int t, int64_t *tmin, int64_t *tmax, int lane)
{
    const int k = t * kTileO + lane;
    const bool in = k < K;
    const ull v = in ? (ull)sP[k] : 0ull;
    const unsigned hi = (unsigned)(v >> 32), lo = (unsigned)v;
    const unsigned xh = __reduce_max_sync(0xffffffffu, in ? hi : 0u);
    const unsigned xl = __reduce_max_sync(0xffffffffu, in && hi == xh ? lo : 0u);
    const unsigned nh = __reduce_min_sync(0xffffffffu, in ? hi : 0xffffffffu);
    const unsigned nl = __reduce_min_sync(0xffffffffu, in && hi == nh ? lo : 0xffffffffu);
    if (lane == 0) { tmax[t] = (int64_t)(((ull)xh << 32) | xl); tmin[t] = (int64_t)(((ull)nh << 32) | nl); }
}

// Benefit of physical slots [lo, hi] for a tensor of s bytes, by one warp: every lane's share (sum them afterwards).
__device__ __forceinline__ u128 benefit_tiles_warp(const int64_t *sP, const int64_t *sStart, const int64_t *tmin, const int64_t *tmax,
                                                   int64_t cap, int64_t s, int lo, int hi, int lane)
{
    u128 acc = 0;
    const int ta = lo / kTileO, tb = hi / kTileO;
#pragma unroll 1
    for (int t0 = ta; t0 <= tb; t0 += 32) {
        const int t = t0 + lane;
        bool mixed = false;
        if (t <= tb) {
            const int k_lo = t * kTileO > lo ? t * kTileO : lo, k_hi = t * kTileO + kTileO - 1 < hi ? t * kTileO + kTileO - 1 : hi;
            const int64_t mn = tmin[t], mx = tmax[t];
            if (mx > cap) {
                if (mn >= cap && mn - cap >= s) acc += (u128)(ull)s * (u128)(ull)(sStart[k_hi + 1] - sStart[k_lo]);
                else mixed = true;
            }
        }
        unsigned m = __ballot_sync(0xffffffffu, mixed);
#pragma unroll 1
        while (m) {
            const int tt = t0 + __ffs(m) - 1;
            m &= m - 1;
            const int k = tt * kTileO + lane;
            if (k >= lo && k <= hi) {
                int64_t ex = sP[k] - cap;
                if (ex > 0) {
                    if (ex > s) ex = s;
                    acc += (u128)(ull)ex * (u128)(ull)(sStart[k + 1] - sStart[k]);
                }
            }
        }
    }
    return acc;
}

// Scores period p against the current state: destination (SSD first, then host) and benefit.
// Whole warp; result valid in lane 0.  Returns false if no destination is admissible (permanent).
template <bool kCyclic = false>
__device__ __forceinline__ bool score_period(const PlanArgs &A, int64_t p, int lane, Cand *out)
{
    const int i = A.per_t[p];
    const int u = A.per_u[p], v = A.per_v[p];
    const int a = u + 1, b = v - 1;
    const int64_t s = A.bytes[i];
    const int64_t t_r = A.start[a], t_end = A.start[v];
    int dest = -1, ap = 0, bp = -1;
    int64_t t = 0;
    for (int X = 0; X < 2 && dest < 0; ++X) {
        ap = A.geo_a[X * A.geo_stride + p];
        if (ap < 0) continue;
        bp = A.geo_b[X * A.geo_stride + p];
        t = A.geo_t[X * A.geo_stride + p];
        if (!window_free<kCyclic>(A, A.busy + (size_t)(2 * X) * A.K, t_r, t_r + t, a, ap - 1, lane)) continue;
        if (!window_free<kCyclic>(A, A.busy + (size_t)(2 * X + 1) * A.K, t_end - t, t_end, bp + 1, b, lane)) continue;
        if (X == G10_DEST_HOST && A.host_capacity != 0) {
            bool ok = true;
            for (int k = a + lane; k <= b; k += 32)
                if ((uint64_t)A.hocc[phys_slot<kCyclic>(A.K, k)] + (uint64_t)s > A.host_capacity) ok = false;
            if (!__all_sync(0xffffffffu, ok)) continue;
        }
        dest = X;
    }
    if (dest < 0) return false;
    u128 acc = 0;
    for (int k = ap + lane; k <= bp; k += 32) {
        const int kp = phys_slot<kCyclic>(A.K, k);
        int64_t ex = A.P[kp] - A.cap;
        if (ex > 0) {
            if (ex > s) ex = s;
            acc += (u128)(ull)ex * (u128)(ull)A.dur[kp];
        }
    }
    acc = warp_sum_u128(acc);
    out->ben = acc; out->cost = 2ull * (ull)t; out->idx = (int)p; out->dest = dest;
    return true;
}


// Block-wide reduction of the best candidate (cand_beats order); result valid in every thread.
__device__ __forceinline__ Cand block_best(Cand x, Cand *s_tmp /* [kPlanWarps + 1] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll 1
    for (int o = 16; o > 0; o >>= 1) {
        const Cand y = cand_shfl_down(x, o);
        if (cand_beats(y, x)) x = y;
    }
    __syncthreads();
    if (lane == 0) s_tmp[warp] = x;
    __syncthreads();
    if (warp == 0) {
        Cand z;
        z.ben = 0; z.cost = 1; z.idx = -1; z.dest = -1;
        if (lane < kPlanWarps) z = s_tmp[lane];
#pragma unroll 1
        for (int o = kPlanWarps / 2; o > 0; o >>= 1) {
            const Cand y = cand_shfl_down(z, o);
            if (cand_beats(y, z)) z = y;
        }
        if (lane == 0) s_tmp[kPlanWarps] = z;
    }
    __syncthreads();
    return s_tmp[kPlanWarps];
}

// Same result as block_best, much shorter dependent chain.  A double-precision ratio orders candidates
// correctly whenever two ratios differ by more than a few ulps, so the block first takes the maximum of the
// rounded ratios (cheap shuffles), keeps as finalists the candidates within 1e-10 of it (the true best is
// always among them: each rounded ratio is within 4 * 2^-53 of the exact one) and only the finalists --
// usually one -- go through the exact 128-bit comparison.  More than 32 finalists fall back to block_best.
struct BestScratch {
    double key[kPlanWarps];
    Cand fin[33];
    int nfin;
};

__device__ __forceinline__ double cand_key(const Cand &c)
{
    if (c.idx < 0) return -1.0;
    const double b = __ull2double_rn((ull)(c.ben >> 64)) * 18446744073709551616.0 + __ull2double_rn((ull)c.ben);
    return b / __ull2double_rn(c.cost);
}

__device__ __forceinline__ Cand block_best_fast(const Cand &x, BestScratch *sc, Cand *s_tmp /* [kPlanWarps + 1] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const double k = cand_key(x);
    double m = k;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { const double y = __shfl_xor_sync(0xffffffffu, m, o); if (y > m) m = y; }
    __syncthreads();                       // previous use of the scratch is over
    if (lane == 0) sc->key[warp] = m;
    if (threadIdx.x == 0) sc->nfin = 0;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kPlanWarps; ++w) { const double y = sc->key[w]; if (y > m) m = y; }
    if (k >= 0.0 && k >= m * (1.0 - 1e-10)) {
        const int pos = atomicAdd(&sc->nfin, 1);
        if (pos < 32) sc->fin[pos] = x;
    }
    __syncthreads();
    const int n = sc->nfin;
    if (n > 32) return block_best(x, s_tmp);
    if (threadIdx.x == 0) {
        Cand w;
        w.ben = 0; w.cost = 1; w.idx = -1; w.dest = -1;
        for (int i = 0; i < n; ++i) if (cand_beats(sc->fin[i], w)) w = sc->fin[i];
        sc->fin[32] = w;
    }
    __syncthreads();
    return sc->fin[32];
}

__device__ __forceinline__ long long block_max_i64(long long m, long long *s_tmp /* [kPlanWarps + 1] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { const long long x = __shfl_down_sync(0xffffffffu, m, o); if (x > m) m = x; }
    __syncthreads();
    if (lane == 0) s_tmp[warp] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kPlanWarps; ++w) if (s_tmp[w] > m) m = s_tmp[w];
        s_tmp[kPlanWarps] = m;
    }
    __syncthreads();
    return s_tmp[kPlanWarps];
}

// Max of the pressure slots owned by this block (tiles c, c + G, ...).
__device__ __forceinline__ long long own_slots_max(const PlanArgs &A, int c, int G, long long *s_tmp)
{
    const int n_slot_tiles = (int)((A.K + kSlotTile - 1) / kSlotTile);
    long long m = 0;
    for (int tl = c; tl < n_slot_tiles; tl += G) {
        const int64_t k0 = (int64_t)tl * kSlotTile;
        for (int64_t k = k0 + threadIdx.x; k < k0 + kSlotTile && k < A.K; k += kPlanThreads) {
            const long long pv = A.P[k];
            if (pv > m) m = pv;
        }
    }
    return block_max_i64(m, s_tmp);
}

// Commits period p with destination X: pressure range-subtract and host occupancy on the slots this block
// owns, channel bookings, the plan record and the erase flag by block 0.  Returns true if this block's
// pressure slots changed.
template <bool kCyclic = false>
__device__ __forceinline__ bool commit_winner(const PlanArgs &A, int64_t p, int X, int64_t it, int64_t n_mig, int c, int G,
                                              int64_t *bytes_out, bool with_bookings = true)
{
    const int64_t K = A.K;
    const int i = A.per_t[p], u = A.per_u[p], v = A.per_v[p];
    const int a = u + 1, b = v - 1;
    const int64_t s = A.bytes[i];
    const int ap = A.geo_a[X * A.geo_stride + p], bp = A.geo_b[X * A.geo_stride + p];
    const int64_t t = A.geo_t[X * A.geo_stride + p];
    const int64_t t_r = A.start[a], t_end = A.start[v];
    bool touched = false;
    // adds `delta` to arr over the unrolled slots [lo, hi], on the tiles this block owns (a range that reaches into the next
    // iteration -- steady-state planning only -- is two runs of physical slots)
    auto range_add = [&](int64_t *arr, int lo, int hi, int64_t delta, bool mark) {
        for (int part = 0; part < (kCyclic ? 2 : 1); ++part) {
            int plo = lo, phi = hi;
            if (kCyclic) {
                if (part == 0) { if (lo >= K) continue; phi = hi < K ? hi : (int)K - 1; }
                else { if (hi < K) continue; plo = (lo > K ? lo : (int)K) - (int)K; phi = hi - (int)K; }
            }
            for (int tl = plo / kSlotTile; tl <= phi / kSlotTile; ++tl) {
                if (tl % G != c) continue;
                if (mark) touched = true;
                const int64_t k0 = (int64_t)tl * kSlotTile;
                for (int64_t k = k0 + threadIdx.x; k < k0 + kSlotTile && k < K; k += kPlanThreads)
                    if (k >= plo && k <= phi) arr[k] += delta;
            }
        }
    };
    range_add(A.P, ap, bp, -s, true);
    if (X == G10_DEST_HOST && A.host_capacity != 0) range_add(A.hocc, a, b, s, false);
    if (c == 0) {
        if (with_bookings) {
            int64_t *bo = A.busy + (size_t)(2 * X) * K, *bi = A.busy + (size_t)(2 * X + 1) * K;
            for (int k = a + threadIdx.x; k <= ap - 1; k += kPlanThreads) {
                const int64_t s0 = A.start[k], s1 = A.start[k + 1];
                const int64_t lo = t_r > s0 ? t_r : s0, hi = (t_r + t) < s1 ? (t_r + t) : s1;
                if (hi > lo) bo[phys_slot<kCyclic>(K, k)] += hi - lo;
            }
            for (int k = bp + 1 + threadIdx.x; k <= b; k += kPlanThreads) {
                const int64_t s0 = A.start[k], s1 = A.start[k + 1];
                const int64_t lo = (t_end - t) > s0 ? (t_end - t) : s0, hi = t_end < s1 ? t_end : s1;
                if (hi > lo) bi[phys_slot<kCyclic>(K, k)] += hi - lo;
            }
        }
        if (threadIdx.x == 0) {
            A.dead[p] = 1;
            if (n_mig < A.out_cap) {
                g10_migration m;
                m.period = (int32_t)p; m.tensor = i; m.dest = X; m.absent_first = ap; m.absent_last = bp;
                m.iteration = (int32_t)it; m.evict_issue_ns = t_r; m.prefetch_issue_ns = t_end - t; m.transfer_ns = t;
                A.out[n_mig] = m;
            } else raise_status(A.status, G10_DEV_PLAN_OVERFLOW);
        }
    }
    *bytes_out = s;
    return touched;
}

// The channel bookings of a committed period (one block adds them, all its threads).
__device__ __forceinline__ void book_winner(const PlanArgs &A, int64_t p, int X)
{
    const int64_t K = A.K;
    const int u = A.per_u[p], v = A.per_v[p];
    const int a = u + 1, b = v - 1;
    const int ap = A.geo_a[X * A.geo_stride + p], bp = A.geo_b[X * A.geo_stride + p];
    const int64_t t = A.geo_t[X * A.geo_stride + p];
    const int64_t t_r = A.start[a], t_end = A.start[v];
    int64_t *bo = A.busy + (size_t)(2 * X) * K, *bi = A.busy + (size_t)(2 * X + 1) * K;
    for (int k = a + threadIdx.x; k <= ap - 1; k += kPlanThreads) {
        const int64_t s0 = A.start[k], s1 = A.start[k + 1];
        const int64_t lo = t_r > s0 ? t_r : s0, hi = (t_r + t) < s1 ? (t_r + t) : s1;
        if (hi > lo) bo[k] += hi - lo;
    }
    for (int k = bp + 1 + threadIdx.x; k <= b; k += kPlanThreads) {
        const int64_t s0 = A.start[k], s1 = A.start[k + 1];
        const int64_t lo = (t_end - t) > s0 ? (t_end - t) : s0, hi = t_end < s1 ? t_end : s1;
        if (hi > lo) bi[k] += hi - lo;
    }
}

// Final peak slot (lowest slot holding the peak) and the summary words.  Every block calls it.
__device__ __forceinline__ void plan_epilogue(const PlanArgs &A, int c, int G, unsigned &gen, int status, long long peak,
                                              int64_t n_mig, int64_t rounds, int64_t bytes_ssd, int64_t bytes_host)
{
    const int64_t K = A.K;
    if (status == -2) {
        if (c == 0 && threadIdx.x == 0) {
            raise_status(A.status, G10_DEV_TIMEOUT);
            A.summary[0] = n_mig; A.summary[1] = rounds; A.summary[2] = -1; A.summary[3] = 0; A.summary[4] = -1;
            A.summary[5] = bytes_ssd; A.summary[6] = bytes_host;
        }
        return;
    }
    const int n_slot_tiles = (int)((K + kSlotTile - 1) / kSlotTile);
    int key = 0;
    for (int tl = c; tl < n_slot_tiles; tl += G) {
        const int64_t k0 = (int64_t)tl * kSlotTile;
        for (int64_t k = k0 + threadIdx.x; k < k0 + kSlotTile && k < K; k += kPlanThreads)
            if (A.P[k] == peak) { const int kk = (int)(K - k); if (kk > key) key = kk; }
    }
    if (key > 0) atomicMax(A.peak_key, key);
    if (!grid_barrier(A.bar, G, gen)) { if (c == 0 && threadIdx.x == 0) raise_status(A.status, G10_DEV_TIMEOUT); return; }
    if (c == 0 && threadIdx.x == 0) {
        const int kk = *((volatile int *)A.peak_key);
        A.summary[0] = n_mig; A.summary[1] = rounds; A.summary[2] = status;
        A.summary[3] = K > 0 ? peak : 0;
        A.summary[4] = kk > 0 ? K - kk : -1;
        A.summary[5] = bytes_ssd; A.summary[6] = bytes_host;
    }
}

void fill_plan_args(const DeviceTrace &t, const Workspace &w, const PlanParams &p, PlanArgs &A);

}  // namespace g10

// Algorithm 1 with the same plan as the printed loop and far fewer rescorings (the default planner).
//
// Pressure only falls and booked channel time / host occupancy only rise while the loop runs.  So, for a
// fixed destination, a period's benefit can only fall: the benefit computed earlier is an upper bound of
// the current one.  Every live period carries its exact destination, its last computed benefit and one of
// three states:
//   FRESH  nothing it depends on changed since it was scored: the cached score is exact;
//   STALE  a later commit lowered the pressure inside its absent range: the cached score is an upper bound;
//   DIRTY  a later commit booked channel time (or host memory) inside one of its transfer windows: its
//          destination has to be chosen again before anything can be said.
// After a commit every block classifies the periods it owns against the winner's slot ranges (a few integer
// comparisons each; whether a booked window still leaves another window of the same channel free is decided in
// constant time).  DIRTY periods are rescored at once; a STALE period is rescored only while its bound may still
// beat the best exact score known to the whole grid, and then by the whole grid together (absent ranges of the
// best candidates span a large part of a long timeline), so that when the iteration decides, the committed score
// is the exact maximum over all live periods, ties included (see k_plan_lazy).
#include "g10_planner.cuh"

namespace g10 {

enum { kFresh = 1, kStale = 2, kDirty = 3 };
constexpr int kMixCap = 1024;            // tiles of one round that a block reads slot by slot, listed
constexpr int kLocalDirty = 128;         // DIRTY periods a block re-examines itself right after its pass

struct LazyArgs {
    unsigned char *c_state;     // 0 = erased; else (dest + 1) | (state << 2)
    ull *c_ben_lo, *c_ben_hi;   // last computed benefit
    ull *c_cost;                // 2 t of the current destination
    double *c_key;              // rounded benefit / cost of the cached score (steers the search; decisions are exact)
    int2 *c_rng;                // absent range [a', b'] of the current destination (a copy of the geometry, so that the
                                // pass over the periods has it in one load, with no look-up by destination)
    int *worklist;              // [2][stride] DIRTY periods of the current round
    unsigned *wl_count;         // [2] lengths of the two work lists; [2..3]: a block could not take its DIRTY periods itself
    LazyProp *props;            // [2][kLazyMaxBlocks] each block's best FRESH candidate and best STALE bounds
    ull *partials;              // [3][kRoundM][2] 128-bit sums of the benefits rescored together (three buffers in turn)
    int64_t *tmin, *tmax;       // [tiles of kSlotTile slots] smallest / largest pressure of each tile
    int64_t stride;
};

__device__ __forceinline__ u128 benefit_partial(const PlanArgs &A, int ap, int bp, int64_t s, int tid, int nthreads)
{
    u128 acc = 0;
    for (int k = ap + tid; k <= bp; k += nthreads) {
        int64_t ex = A.P[k] - A.cap;
        if (ex > 0) {
            if (ex > s) ex = s;
            acc += (u128)(ull)ex * (u128)(ull)A.dur[k];
        }
    }
    return acc;
}

// The same sum for one tile read by one warp: eight slots per lane in flight (the tile comes from L2).
__device__ __forceinline__ u128 benefit_tile_warp(const PlanArgs &A, int k_lo, int k_hi, int64_t s, int lane)
{
    u128 acc = 0;
#pragma unroll 1
    for (int k0 = k_lo + lane; k0 <= k_hi; k0 += 8 * 32) {
        int64_t ex[8], du[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int k = k0 + 32 * j;
            ex[j] = k <= k_hi ? A.P[k] : 0;
            du[j] = k <= k_hi ? A.dur[k] : 0;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            int64_t e = ex[j] - A.cap;
            if (k0 + 32 * j <= k_hi && e > 0) {
                if (e > s) e = s;
                acc += (u128)(ull)e * (u128)(ull)du[j];
            }
        }
    }
    return acc;
}

__device__ __forceinline__ void store_score(const PlanArgs &A, const LazyArgs &L, int64_t p, int dest, int state, u128 ben, ull cost)
{
    L.c_rng[p] = make_int2(A.geo_a[dest * A.geo_stride + p], A.geo_b[dest * A.geo_stride + p]);
    L.c_ben_lo[p] = (ull)ben;
    L.c_ben_hi[p] = (ull)(ben >> 64);
    L.c_cost[p] = cost;
    Cand cd;
    cd.ben = ben; cd.cost = cost; cd.idx = 0; cd.dest = dest;
    L.c_key[p] = ben == 0 ? 0.0 : cand_key(cd);
    L.c_state[p] = (unsigned char)((dest + 1) | (state << 2));
}

// One warp brings period p up to date (destination if DIRTY, benefit always).
__device__ __forceinline__ void eval_warp(const PlanArgs &A, const LazyArgs &L, int64_t p, int lane)
{
    const unsigned char st = L.c_state[p];
    if (st == 0) return;
    if ((st >> 2) == kDirty) {
        Cand cd;
        if (!score_period(A, p, lane, &cd)) { if (lane == 0) L.c_state[p] = 0; return; }
        if (lane == 0) store_score(A, L, p, cd.dest, kFresh, cd.ben, cd.cost);
        return;
    }
    const int d = (st & 3) - 1;
    const int ap = A.geo_a[d * A.geo_stride + p], bp = A.geo_b[d * A.geo_stride + p];
    const int64_t s = A.bytes[A.per_t[p]];
    u128 acc = warp_sum_u128(benefit_partial(A, ap, bp, s, lane, 32));
    if (lane == 0) store_score(A, L, p, d, kFresh, acc, 2ull * (ull)A.geo_t[d * A.geo_stride + p]);
}

// One warp re-chooses the destination of DIRTY period p (SSD first, then host).  The period is erased if no
// destination is left; otherwise it becomes STALE with an unbounded score, so that it is rescored with the others.
// pend (optional): a commit whose channel bookings are not in A.busy yet; its share of every slot is added on the fly
// (the same amounts book_winner adds later), so that the answer is the one the booked arrays will give.
struct Winner;
__device__ __forceinline__ bool window_free_pending(const PlanArgs &A, const int64_t *busy, int64_t w0, int64_t w1, int k0, int k1, int lane,
                                                    int vk0, int vk1, int64_t v0, int64_t v1)
{
    bool ok = true;
    for (int k = k0 + lane; k <= k1; k += 32) {
        const int64_t s0 = A.start[k], s1 = A.start[k + 1];
        const int64_t lo = w0 > s0 ? w0 : s0, hi = w1 < s1 ? w1 : s1;
        const int64_t ov = hi > lo ? hi - lo : 0;
        int64_t extra = 0;
        if (k >= vk0 && k <= vk1) {
            const int64_t vl = v0 > s0 ? v0 : s0, vh = v1 < s1 ? v1 : s1;
            extra = vh > vl ? vh - vl : 0;
        }
        if (busy[k] + extra + ov > s1 - s0) ok = false;
    }
    return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void dest_warp(const PlanArgs &A, const LazyArgs &L, int64_t p, int lane, int pend_dest = -1, int pa = 0, int pap = 0,
                                          int pbp = 0, int pb = 0, int64_t pt = 0, int64_t pt_r = 0, int64_t pt_end = 0)
{
    if (L.c_state[p] == 0) return;
    const int u = A.per_u[p], v = A.per_v[p];
    const int a = u + 1, b = v - 1;
    const int64_t s = A.bytes[A.per_t[p]];
    const int64_t t_r = A.start[a], t_end = A.start[v];
    int dest = -1;
    int64_t t = 0;
    for (int X = 0; X < 2 && dest < 0; ++X) {
        const int ap = A.geo_a[X * A.geo_stride + p];
        if (ap < 0) continue;
        const int bp = A.geo_b[X * A.geo_stride + p];
        t = A.geo_t[X * A.geo_stride + p];
        if (X == pend_dest) {
            if (!window_free_pending(A, A.busy + (size_t)(2 * X) * A.K, t_r, t_r + t, a, ap - 1, lane, pa, pap - 1, pt_r, pt_r + pt)) continue;
            if (!window_free_pending(A, A.busy + (size_t)(2 * X + 1) * A.K, t_end - t, t_end, bp + 1, b, lane, pbp + 1, pb, pt_end - pt, pt_end)) continue;
        } else {
            if (!window_free(A, A.busy + (size_t)(2 * X) * A.K, t_r, t_r + t, a, ap - 1, lane)) continue;
            if (!window_free(A, A.busy + (size_t)(2 * X + 1) * A.K, t_end - t, t_end, bp + 1, b, lane)) continue;
        }
        if (X == G10_DEST_HOST && A.host_capacity != 0) {
            bool ok = true;
            for (int k = a + lane; k <= b; k += 32)
                if ((uint64_t)A.hocc[k] + (uint64_t)s > A.host_capacity) ok = false;
            if (!__all_sync(0xffffffffu, ok)) continue;
        }
        dest = X;
    }
    if (lane == 0) {
        if (dest < 0) L.c_state[p] = 0;
        else {
            L.c_ben_lo[p] = 0; L.c_ben_hi[p] = 0; L.c_cost[p] = 2ull * (ull)t;
            L.c_rng[p] = make_int2(A.geo_a[dest * A.geo_stride + p], A.geo_b[dest * A.geo_stride + p]);
            L.c_key[p] = __longlong_as_double(0x7ff0000000000000ll);      // +infinity: rescored before anything is decided
            L.c_state[p] = (unsigned char)((dest + 1) | (kStale << 2));
        }
    }
}


// Smallest and largest pressure of slot tile tl, recomputed by the whole block (the tile's owner).
__device__ __forceinline__ void tile_minmax(const PlanArgs &A, const LazyArgs &L, int tl, long long *s_red /* [2 * kPlanWarps] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t k0 = (int64_t)tl * kSlotTile;
    long long mn = 0x7fffffffffffffffll, mx = -0x7fffffffffffffffll - 1;
    for (int64_t k = k0 + threadIdx.x; k < k0 + kSlotTile && k < A.K; k += kPlanThreads) {
        const long long pv = A.P[k];
        if (pv < mn) mn = pv;
        if (pv > mx) mx = pv;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const long long a = __shfl_xor_sync(0xffffffffu, mn, o), b = __shfl_xor_sync(0xffffffffu, mx, o);
        if (a < mn) mn = a;
        if (b > mx) mx = b;
    }
    __syncthreads();
    if (lane == 0) { s_red[2 * warp] = mn; s_red[2 * warp + 1] = mx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kPlanWarps; ++w) { if (s_red[2 * w] < mn) mn = s_red[2 * w]; if (s_red[2 * w + 1] > mx) mx = s_red[2 * w + 1]; }
        L.tmin[tl] = mn; L.tmax[tl] = mx;
    }
}

// Largest pressure over the tiles this block owns (tiles c, c + G, ...), from the tile maxima.
__device__ __forceinline__ long long own_tiles_max(const PlanArgs &A, const LazyArgs &L, int c, int G, long long *s_tmp)
{
    const int n_slot_tiles = (int)((A.K + kSlotTile - 1) / kSlotTile);
    long long m = 0;
    for (int tl = c + (int)threadIdx.x * G; tl < n_slot_tiles; tl += kPlanThreads * G) {
        const long long x = L.tmax[tl];
        if (x > m) m = x;
    }
    return block_max_i64(m, s_tmp);
}

// Commits period p with destination X on what this block owns: the pressure slots of its tiles (with their new
// minima / maxima) and host occupancy; block 0 also writes the plan record and the erase flag.  The channel
// bookings are added later (book_winner).  Returns true if a tile of this block changed.
__device__ __forceinline__ bool commit_lazy(const PlanArgs &A, const LazyArgs &L, int64_t p, int X, int64_t it, int64_t n_mig, int c, int G,
                                            long long *s_red, int a, int ap, int bp, int b, int64_t t)
{
    // (the winner's slot ranges and transfer time come from the caller, which looked them up when it decided; only the
    // tensor's size is fetched here)
    const int64_t K = A.K;
    const int i = A.per_t[p];
    const int64_t s = A.bytes[i];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    bool touched = false;
    {
        const int ta = ap / kSlotTile, tb = bp / kSlotTile;
        int tl = ta + ((c - ta % G) % G + G) % G;            // first tile >= ta that this block owns
        for (; tl <= tb; tl += G) {
            touched = true;
            // one pass over the tile: subtract inside the range, and the tile's new minimum and maximum from the same values
            const int64_t k0 = (int64_t)tl * kSlotTile;
            long long mn = 0x7fffffffffffffffll, mx = -0x7fffffffffffffffll - 1;
            for (int64_t k = k0 + threadIdx.x; k < k0 + kSlotTile && k < K; k += kPlanThreads) {
                long long pv = A.P[k];
                if (k >= ap && k <= bp) { pv -= s; A.P[k] = pv; }
                if (pv < mn) mn = pv;
                if (pv > mx) mx = pv;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const long long x = __shfl_xor_sync(0xffffffffu, mn, o), y = __shfl_xor_sync(0xffffffffu, mx, o);
                if (x < mn) mn = x;
                if (y > mx) mx = y;
            }
            __syncthreads();                                   // (s_red free)
            if (lane == 0) { s_red[2 * warp] = mn; s_red[2 * warp + 1] = mx; }
            __syncthreads();
            if (warp == 0) {
                long long x = lane < kPlanWarps ? s_red[2 * lane] : 0x7fffffffffffffffll;
                long long y = lane < kPlanWarps ? s_red[2 * lane + 1] : -0x7fffffffffffffffll - 1;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const long long x2 = __shfl_xor_sync(0xffffffffu, x, o), y2 = __shfl_xor_sync(0xffffffffu, y, o);
                    if (x2 < x) x = x2;
                    if (y2 > y) y = y2;
                }
                if (lane == 0) { L.tmin[tl] = x; L.tmax[tl] = y; }
            }
        }
    }
    if (X == G10_DEST_HOST && A.host_capacity != 0) {
        const int ta = a / kSlotTile, tb = b / kSlotTile;
        int tl = ta + ((c - ta % G) % G + G) % G;
        for (; tl <= tb; tl += G) {
            const int64_t k0 = (int64_t)tl * kSlotTile;
            for (int64_t k = k0 + threadIdx.x; k < k0 + kSlotTile && k < K; k += kPlanThreads)
                if (k >= a && k <= b) A.hocc[k] += s;
        }
    }
    if (c == 0 && threadIdx.x == 0) {
        A.dead[p] = 1;
        if (n_mig < A.out_cap) {
            g10_migration m;
            m.period = (int32_t)p; m.tensor = i; m.dest = X; m.absent_first = ap; m.absent_last = bp;
            m.iteration = (int32_t)it; m.evict_issue_ns = A.start[a]; m.prefetch_issue_ns = A.start[b + 1] - t; m.transfer_ns = t;
            A.out[n_mig] = m;
        } else raise_status(A.status, G10_DEV_PLAN_OVERFLOW);
    }
    return touched;
}

// This block's share of the benefit of absent range [ap, bp] for a tensor of s bytes: tiles ta + c, ta + c + G, ...
// of the range, one warp.  A tile whose smallest pressure is at least capacity + s counts s for its whole time,
// one whose largest pressure is within capacity counts nothing; only the others are read slot by slot.
__device__ __forceinline__ u128 benefit_tiles(const PlanArgs &A, const LazyArgs &L, int ap, int bp, int64_t s, int c, int G, int lane)
{
    u128 acc = 0;
    const int ta = ap / kSlotTile, tb = bp / kSlotTile;
    for (int tl = ta + c; tl <= tb; tl += G) {
        const int64_t t0 = (int64_t)tl * kSlotTile, t1 = t0 + kSlotTile - 1;
        const int k_lo = (int)(t0 > ap ? t0 : ap), k_hi = (int)(t1 < bp ? t1 : bp);
        const long long mn = L.tmin[tl], mx = L.tmax[tl];
        if (mx <= A.cap) continue;
        if (mn >= A.cap && mn - A.cap >= s) {
            if (lane == 0) acc += (u128)(ull)s * (u128)(ull)(A.start[k_hi + 1] - A.start[k_lo]);
            continue;
        }
        acc += benefit_partial(A, k_lo, k_hi, s, lane, 32);
    }
    return acc;
}

// What a block tells the grid after a pass over its periods: its best FRESH candidate (exact) and its kTopT best
// STALE bounds (rounded ratio and period, descending; idx < 0 = none).  Any STALE period it did not list has a
// bound no larger than the last one listed.
__device__ __forceinline__ void store_prop(LazyProp *pr, const Cand &c, const double *tk, const int *ti)
{
    LazyProp q;
    q.ben_lo = (ull)c.ben; q.ben_hi = (ull)(c.ben >> 64); q.cost = c.cost; q.idx = c.idx; q.dest = c.dest;
#pragma unroll
    for (int j = 0; j < kTopT; ++j) { q.skey[j] = tk[j]; q.sidx[j] = ti[j]; }
    *pr = q;
}

// Block-wide maximum of (key, idx), larger idx on equal keys: uniform result.
__device__ __forceinline__ void block_max_key(double &k, int &idx, double *s_k /* [kPlanWarps] */, int *s_i /* [kPlanWarps] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double yk = __shfl_xor_sync(0xffffffffu, k, o);
        const int yi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (yk > k || (yk == k && yi > idx)) { k = yk; idx = yi; }
    }
    __syncthreads();
    if (lane == 0) { s_k[warp] = k; s_i[warp] = idx; }
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kPlanWarps; ++w) {
        const double yk = s_k[w];
        const int yi = s_i[w];
        if (yk > k || (yk == k && yi > idx)) { k = yk; idx = yi; }
    }
}

// Can STALE period p, whose cached score (rounded ratio `key`) bounds its current one, still beat candidate t
// (rounded ratio t_key)?  Clear cases by the rounded ratios, anything within 1e-10 by the exact comparison of the
// cached benefit and cost (a tie goes to the lower period index, as in the final decision).
__device__ __forceinline__ bool bound_may_beat(const LazyArgs &L, int p, double key, double t_key, const Cand *t)
{
    if (!(key > 0.0)) return false;
    if (!t || t->idx < 0) return true;
    if (key > t_key * (1.0 + 1e-10)) return true;
    if (key < t_key * (1.0 - 1e-10)) return false;
    Cand x;
    x.ben = ((u128)__ldcg(&L.c_ben_hi[p]) << 64) | __ldcg(&L.c_ben_lo[p]); x.cost = __ldcg(&L.c_cost[p]); x.idx = p; x.dest = 0;
    return cand_beats(x, *t);
}

struct Winner {
    int idx, dest, a, ap, bp, b;      // evict slots [a, ap-1], absent [ap, bp], prefetch [bp+1, b]
    int64_t t, t_r, t_end;            // transfer time, start of the eviction, end of the prefetch
};

// One pass of a block over the periods it owns (period p belongs to block (p / kPlanThreads) mod G).  With
// `classify` the pending winner's slot ranges are applied first (FRESH -> STALE where its absent range meets
// theirs, -> DIRTY where its booking leaves one of their transfer windows no room; the bookings are not in
// A.busy yet) and DIRTY periods are appended to the work list.  Returns the block's best FRESH candidate (exact)
// and leaves its kTopT best STALE bounds in s_tk / s_ti (uniform).
__device__ __forceinline__ Cand scan_owned(const PlanArgs &A, const LazyArgs &L, int64_t Pn, bool classify, const Winner &w,
                                           int par, BestScratch *sc, Cand *s_cand, double *s_k, int *s_i, double *s_tk, int *s_ti,
                                           const Cand *floor = nullptr, int *s_dl = nullptr, int *s_ndl = nullptr)
{
    // with a floor (the best exact score known to the grid) only the STALE bounds that can beat it are listed
    const double floor_key = floor && floor->idx >= 0 ? cand_key(*floor) : -1.0;
    const int G = gridDim.x, c = blockIdx.x, lane = threadIdx.x & 31;
    double kf = -1.0;
    int pf = -1;
    double tk[kTopT];
    int ti[kTopT];
#pragma unroll
    for (int j = 0; j < kTopT; ++j) { tk[j] = -1.0; ti[j] = -1; }
    const int64_t *bo = A.busy + (size_t)(2 * (w.dest < 0 ? 0 : w.dest)) * A.K, *bi = bo + A.K;
    // The pass is a chain of L2 latencies: the loads of four periods of this thread are in flight together.
    constexpr int kAhead = 4;
    const int64_t step = (int64_t)G * kPlanThreads;
    for (int64_t p00 = (int64_t)c * kPlanThreads; p00 < Pn; p00 += kAhead * step) {
      unsigned char st_q[kAhead];
      double key_q[kAhead];
      int u_q[kAhead], v_q[kAhead];
      int2 rng_q[kAhead];
#pragma unroll
      for (int q = 0; q < kAhead; ++q) {
          const int64_t pq = p00 + q * step + threadIdx.x;
          st_q[q] = 0; key_q[q] = 0.0; u_q[q] = 0; v_q[q] = 0; rng_q[q] = make_int2(0, -1);
          if (pq < Pn) {
              st_q[q] = L.c_state[pq]; key_q[q] = L.c_key[pq];
              if (classify) { u_q[q] = A.per_u[pq]; v_q[q] = A.per_v[pq]; rng_q[q] = L.c_rng[pq]; }     // (the range: rubbish while the period is DIRTY, not used then)
          }
      }
#pragma unroll
      for (int q = 0; q < kAhead; ++q) {
        const int64_t p0 = p00 + q * step;
        if (p0 >= Pn) break;                                  // (uniform in the block)
        const int64_t p = p0 + threadIdx.x;
        bool dirty = false;
        unsigned char st = st_q[q];
        const double key_ld = key_q[q];
        const int u = u_q[q], v = v_q[q];
        if (p < Pn) {
            if (st != 0) {
                int state = st >> 2;
                const int d = (st & 3) - 1;
                if (classify) {
                    if (p == w.idx) { L.c_state[p] = 0; st = 0; }
                    else if (state != kDirty) {
                        if (u + 1 <= w.b && w.a <= v - 1) {          // the two periods share slots
                            const int ap = rng_q[q].x, bp = rng_q[q].y;
                            bool hit = false;
                            if (d == w.dest) {
                                const bool meet_out = u + 1 <= w.ap - 1 && w.a <= ap - 1, meet_in = bp + 1 <= w.b && w.bp + 1 <= v - 1;
                                if (meet_out || meet_in) {
                                    const int64_t tq = A.geo_t[d * A.geo_stride + p];
                                    const int64_t q_r = A.start[u + 1], q_end = A.start[v];
                                    hit = (meet_out && window_conflict<false, true>(A.start, bo, w.a, w.ap - 1, w.t_r, w.t_r + w.t, q_r, q_r + tq, u + 1, ap - 1)) ||
                                          (meet_in && window_conflict<false, true>(A.start, bi, w.bp + 1, w.b, w.t_end - w.t, w.t_end, q_end - tq, q_end, bp + 1, v - 1));
                                }
                                if (!hit && d == G10_DEST_HOST && A.host_capacity != 0) hit = true;
                            }
                            if (hit) state = kDirty;
                            else if (state == kFresh && ap <= w.bp && w.ap <= bp) state = kStale;
                            if (state != (st >> 2)) { st = (unsigned char)((st & 3) | (state << 2)); L.c_state[p] = st; }
                        }
                    }
                }
                if (st != 0) {
                    if (state == kDirty) dirty = true;
                    else {
                        const double key = key_ld;
                        if (key > 0.0) {
                            if (state == kFresh) {
                                bool take = key > kf;
                                if (pf >= 0 && key >= kf * (1.0 - 1e-10) && kf >= key * (1.0 - 1e-10)) {
                                    Cand x, y;                       // too close to call by rounding: exact
                                    x.ben = ((u128)L.c_ben_hi[p] << 64) | L.c_ben_lo[p]; x.cost = L.c_cost[p]; x.idx = (int)p; x.dest = 0;
                                    y.ben = ((u128)L.c_ben_hi[pf] << 64) | L.c_ben_lo[pf]; y.cost = L.c_cost[pf]; y.idx = pf; y.dest = 0;
                                    take = cand_beats(x, y);
                                }
                                if (take) { kf = key; pf = (int)p; }
                            } else if (key > tk[kTopT - 1] && bound_may_beat(L, (int)p, key, floor_key, floor)) {
                                // insertion into this thread's sorted best STALE bounds
                                int j = kTopT - 1;
#pragma unroll
                                for (int q = kTopT - 1; q > 0; --q)
                                    if (j == q && key > tk[q - 1]) { tk[q] = tk[q - 1]; ti[q] = ti[q - 1]; j = q - 1; }
                                tk[j] = key; ti[j] = (int)p;
                            }
                        }
                    }
                }
            }
        }
        if (classify) {
            // DIRTY periods go on the work list (one atomic per warp)
            const unsigned md = __ballot_sync(0xffffffffu, dirty);
            if (md) {
                unsigned base = 0;
                if (lane == 0) base = atomicAdd(&L.wl_count[par], (unsigned)__popc(md));
                base = __shfl_sync(0xffffffffu, base, 0);
                if (dirty) L.worklist[(size_t)par * L.stride + base + __popc(md & ((1u << lane) - 1u))] = (int)p;
                if (s_dl != nullptr) {                         // ... and on the block's own list
                    int lb = 0;
                    if (lane == 0) lb = atomicAdd(s_ndl, __popc(md));
                    lb = __shfl_sync(0xffffffffu, lb, 0);
                    const int q2 = lb + __popc(md & ((1u << lane) - 1u));
                    if (dirty && q2 < kLocalDirty) s_dl[q2] = (int)p;
                }
            }
        }
      }
    }
    Cand x;
    x.ben = 0; x.cost = 1; x.idx = -1; x.dest = -1;
    if (pf >= 0) {
        x.ben = ((u128)L.c_ben_hi[pf] << 64) | L.c_ben_lo[pf]; x.cost = L.c_cost[pf]; x.idx = pf;
        x.dest = (L.c_state[pf] & 3) - 1;
    }
    const Cand bestF = block_best_fast(x, sc, s_cand);
    // the block's kTopT best bounds: every warp takes the kTopT best of its lanes' lists with shuffles alone (kTopT rounds
    // of a warp-wide maximum over the lanes' current heads; larger index on equal keys), then warp 0 takes the kTopT best
    // of the warps' results the same way
    __shared__ double s_wk[kPlanWarps * kTopT];
    __shared__ int s_wi[kPlanWarps * kTopT];
    const int warp = threadIdx.x >> 5;
    auto warp_take = [&](double &hk, int &hi) {              // warp-wide maximum of (hk, hi); uniform result
        double k = hk;
        int idx = hi;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const double yk = __shfl_xor_sync(0xffffffffu, k, o);
            const int yi = __shfl_xor_sync(0xffffffffu, idx, o);
            if (yk > k || (yk == k && yi > idx)) { k = yk; idx = yi; }
        }
        hk = k; hi = idx;
    };
#pragma unroll 1
    for (int r = 0; r < kTopT; ++r) {
        double k = tk[0];
        int idx = ti[0];
        warp_take(k, idx);
        if (idx >= 0 && idx == ti[0]) {                 // this lane's head was taken: next one moves up
#pragma unroll
            for (int q = 0; q < kTopT - 1; ++q) { tk[q] = tk[q + 1]; ti[q] = ti[q + 1]; }
            tk[kTopT - 1] = -1.0; ti[kTopT - 1] = -1;
        }
        if (lane == 0) { s_wk[warp * kTopT + r] = idx >= 0 ? k : -1.0; s_wi[warp * kTopT + r] = idx; }
    }
    __syncthreads();
    if (warp == 0) {
        // kPlanWarps * kTopT entries, kPerLane per lane, kept in descending order by the lane
        constexpr int kPerLane = (kPlanWarps * kTopT + 31) / 32;
        double ek[kPerLane];
        int ei[kPerLane];
#pragma unroll
        for (int h = 0; h < kPerLane; ++h) {
            const int e = lane + 32 * h;
            double k = e < kPlanWarps * kTopT ? s_wk[e] : -1.0;
            int idx = e < kPlanWarps * kTopT ? s_wi[e] : -1;
            if (idx < 0) k = -1.0;
            // insertion into ek[0..h)
#pragma unroll
            for (int q = 0; q < kPerLane; ++q) {
                if (q < h && (k > ek[q] || (k == ek[q] && idx > ei[q]))) { const double a = ek[q]; ek[q] = k; k = a; const int b2 = ei[q]; ei[q] = idx; idx = b2; }
            }
            ek[h] = k; ei[h] = idx;
        }
#pragma unroll 1
        for (int r = 0; r < kTopT; ++r) {
            double k = ek[0];
            int idx = ei[0];
            warp_take(k, idx);
            if (idx >= 0 && idx == ei[0]) {
#pragma unroll
                for (int q = 0; q < kPerLane - 1; ++q) { ek[q] = ek[q + 1]; ei[q] = ei[q + 1]; }
                ek[kPerLane - 1] = -1.0; ei[kPerLane - 1] = -1;
            }
            if (lane == 0) { s_tk[r] = idx >= 0 ? k : -1.0; s_ti[r] = idx; }
        }
    }
    __syncthreads();
    return bestF;
}

// Could a STALE bound with rounded ratio `key` beat (or tie with) candidate t?  Conservative by 1e-10.
__device__ __forceinline__ bool may_beat(double key, const Cand &t)
{
    if (!(key > 0.0)) return false;
    if (t.idx < 0) return true;
    return key >= cand_key(t) * (1.0 - 1e-10);
}

// Per iteration:
//  A  every block applies the previous commit to the pressure slots it owns, classifies the periods it owns
//     and publishes its best FRESH candidate and its kTopT best STALE bounds; grid barrier;
//  B  every block reads all publications: the best FRESH score of the grid, the peak, the stop tests; block 0
//     adds the previous commit's bookings; DIRTY periods, if any, are rescored (shared out over the grid) and
//     everything is published again;
//  R  rounds: the (at most kRoundM) best published bounds that may still beat the best exact score are rescored
//     by the whole grid together -- every block sums its slice of each absent range, a barrier, every block adds
//     up the slices -- and the best exact score is updated; a block whose published bounds are used up while the
//     last of them may still beat the best score looks again and publishes more;
//  D  no bound left that may beat it: the best exact score is the exact maximum over all live periods; commit.
// All decisions are taken from data every block has, so the control flow is the same in every block.
__global__ void __launch_bounds__(kPlanThreads, 1) k_plan_lazy(PlanArgs A, LazyArgs L)
{
    __shared__ Cand s_cand[kPlanWarps + 1];
    __shared__ BestScratch s_best;
    __shared__ long long s_max[2 * kPlanWarps + 1];
    __shared__ double s_k[kPlanWarps];
    __shared__ int s_i[kPlanWarps];
    __shared__ double s_tk[kTopT];
    __shared__ int s_ti[kTopT];
    __shared__ double s_pkey[kLazyMaxBlocks * kTopT];      // published bounds of all blocks
    __shared__ int s_pidx[kLazyMaxBlocks * kTopT];
    __shared__ unsigned char s_pdone[kLazyMaxBlocks * kTopT];
    // what a round keeps per rescored period, in dynamic shared memory (kLazyDynBytes)
    extern __shared__ __align__(16) unsigned char s_dyn_lazy[];
    Cand *s_new = (Cand *)s_dyn_lazy;                                   // [kRoundM]
    ull *s_acc = (ull *)(s_new + kRoundM);                              // [2 * kRoundM]
    long long *s_it_s = (long long *)(s_acc + 2 * kRoundM);             // [kRoundM]
    ull *s_it_cost = (ull *)(s_it_s + kRoundM);                         // [kRoundM]
    int *s_sel = (int *)(s_it_cost + kRoundM);                          // [kRoundM]
    int *s_it_d = s_sel + kRoundM, *s_it_ap = s_it_d + kRoundM, *s_it_bp = s_it_ap + kRoundM;
    __shared__ int s_wcnt[kPlanWarps];
    __shared__ int s_mix[kMixCap];
    __shared__ int s_nmix;
    __shared__ int s_flag;
    __shared__ unsigned char s_refresh[kLazyMaxBlocks];
    __shared__ int s_dl[kLocalDirty];
    __shared__ int s_ndl;
    const int G = gridDim.x, c = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t Pn = *A.Pn_dev < A.geo_stride ? *A.Pn_dev : A.geo_stride;
    const int64_t limit = (A.max_iterations <= 0 || A.max_iterations > Pn) ? Pn : A.max_iterations;
    unsigned gen = 0;
    int64_t n_mig = 0, rounds = 0, bytes_ssd = 0, bytes_host = 0;
    int status = -1;
    long long peak = 0;
    int par = 0;                               // which worklist buffer this iteration fills
    int pbuf = 0;                              // which publication buffer is written next
    int pp = 0;                                // which slice buffer is written next

    if (c == 0) for (int j = threadIdx.x; j < 3 * kRoundM * 2; j += kPlanThreads) L.partials[j] = 0;
    // every period starts DIRTY: its first evaluation chooses the destination
    for (int64_t p = (int64_t)c * kPlanThreads + threadIdx.x; p < Pn; p += (int64_t)G * kPlanThreads) {
        L.c_state[p] = (unsigned char)(kDirty << 2);
        L.c_key[p] = 0.0;
    }
    {
        const int n_slot_tiles = (int)((A.K + kSlotTile - 1) / kSlotTile);
        for (int tl = c; tl < n_slot_tiles; tl += G) tile_minmax(A, L, tl, s_max);
        __syncthreads();
        const long long m = own_tiles_max(A, L, c, G, s_max);
        if (threadIdx.x == 0) A.peak_part[c] = m;
    }
    if (!grid_barrier(A.bar, G, gen)) status = -2;

    bool pending = false;                      // a commit decided in the previous iteration, not yet applied
    Winner win;
    win.idx = -1; win.dest = -1; win.a = 0; win.ap = 0; win.bp = -1; win.b = -1; win.t = 0; win.t_r = 0; win.t_end = 0;
    Cand gBest;

    // reads the published bounds from buffer `buf` into shared memory, unused; with only_flagged just those of
    // the blocks that published again (s_refresh)
    auto load_bounds = [&](int buf, bool only_flagged) {
        for (int e = threadIdx.x; e < G * kTopT; e += kPlanThreads) {
            const int j = e / kTopT, q = e % kTopT;
            if (only_flagged && !s_refresh[j]) continue;
            const LazyProp *pr = &L.props[(size_t)buf * kLazyMaxBlocks + j];
            s_pkey[e] = __ldcg(&pr->skey[q]);
            s_pidx[e] = __ldcg(&pr->sidx[q]);
            s_pdone[e] = 0;
        }
        __syncthreads();
    };
    auto load_best = [&](int buf) -> Cand {
        Cand x;
        x.ben = 0; x.cost = 1; x.idx = -1; x.dest = -1;
        for (int j = threadIdx.x; j < G; j += kPlanThreads) {
            const LazyProp *pr = &L.props[(size_t)buf * kLazyMaxBlocks + j];
            Cand y;
            const ull lo = __ldcg(&pr->ben_lo), hi = __ldcg(&pr->ben_hi);
            y.ben = ((u128)hi << 64) | lo; y.cost = __ldcg(&pr->cost); y.idx = __ldcg(&pr->idx); y.dest = __ldcg(&pr->dest);
            if (cand_beats(y, x)) x = y;
        }
        return block_best_fast(x, &s_best, s_cand);
    };

    for (int64_t it = 0; status == -1; ++it) {
        bool barrier_since_booking = true;
        // ---------------- A: apply the pending commit to the slots this block owns (bookings: after the barrier)
        if (pending) {
            const bool touched = commit_lazy(A, L, win.idx, win.dest, it - 1, n_mig - 1, c, G, s_max, win.a, win.ap, win.bp, win.b, win.t);
            if (touched) {
                __syncthreads();
                const long long m = own_tiles_max(A, L, c, G, s_max);
                if (threadIdx.x == 0) A.peak_part[c] = m;
            }
        }
        // classify the owned periods against the commit, collect DIRTY ones, local bests
        // (on the first iteration `win` matches nothing and every period is DIRTY)
        // With unlimited host memory a DIRTY period's new destination depends on the channel bookings alone, and the
        // pending commit's share of them is known here: the block re-examines its DIRTY periods itself, at once, which
        // spares the grid two barriers (with finite host memory the occupancy of other blocks' slots is needed too).
        const bool own_dirty = pending && A.host_capacity == 0;
        if (threadIdx.x == 0) s_ndl = 0;
        __syncthreads();
        {
            const Cand bestF = scan_owned(A, L, Pn, true, win, par, &s_best, s_cand, s_k, s_i, s_tk, s_ti, nullptr,
                                          own_dirty ? s_dl : nullptr, &s_ndl);
            if (threadIdx.x == 0) store_prop(&L.props[(size_t)pbuf * kLazyMaxBlocks + c], bestF, s_tk, s_ti);
        }
        if (own_dirty) {
            const int ndl = s_ndl;                              // (scan_owned ends with a barrier)
            if (ndl > kLocalDirty) { if (threadIdx.x == 0) atomicOr(&L.wl_count[2 + par], 1u); }
            else
                for (int e = warp; e < ndl; e += kPlanWarps)
                    dest_warp(A, L, s_dl[e], lane, win.dest, win.a, win.ap, win.bp, win.b, win.t, win.t_r, win.t_end);
        }
        if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }
        int rbuf = pbuf;
        pbuf ^= 1;

        // ---------------- B: best FRESH score of the grid, peak, stop tests
        long long m = 0;
        for (int j = threadIdx.x; j < G; j += kPlanThreads) {
            const long long pm = __ldcg(&A.peak_part[j]);
            if (pm > m) m = pm;
        }
        peak = block_max_i64(m, s_max);
        gBest = load_best(rbuf);
        const unsigned W = __ldcg(&L.wl_count[par]);
        const bool dirty_done = own_dirty && __ldcg(&L.wl_count[2 + par]) == 0u;     // every block took its own
        if (A.fits_always || peak <= A.cap) { status = n_mig == 0 ? G10_ALREADY_FITS : G10_FIT; break; }
        if (it >= limit) { status = limit < Pn ? G10_ITERATION_LIMIT : G10_EXHAUSTED; break; }
        rounds += 1;
        if (pending && c == 0) { book_winner(A, win.idx, win.dest); barrier_since_booking = false; }
        if (pending) barrier_since_booking = false;
        pending = false;
        const int *wl = L.worklist + (size_t)par * L.stride;
        if (c == 0 && threadIdx.x == 0) { L.wl_count[par ^ 1] = 0; L.wl_count[2 + (par ^ 1)] = 0; }
        par ^= 1;
        const bool few_dirty = W > 0 && W <= (unsigned)kDirtyPool && G * kTopT + kDirtyPool <= kLazyMaxBlocks * kTopT;
        if (few_dirty && dirty_done) {
            // (their owners have re-chosen the destinations already; they join the published bounds below)
        } else if (few_dirty) {
            // DIRTY periods need the bookings in place: barrier; one warp re-chooses each one's destination; barrier.
            // They join the published bounds below with an unbounded score and are rescored with the others.
            if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }
            barrier_since_booking = true;
            for (unsigned e = (unsigned)c * kPlanWarps + warp; e < W; e += (unsigned)G * kPlanWarps) dest_warp(A, L, wl[e], lane);
            if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }
        } else if (W > 0) {
            // very many DIRTY periods (the first iteration): rescore them at once, shared out, and look again
            if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }
            barrier_since_booking = true;
            for (unsigned e = (unsigned)c * kPlanWarps + warp; e < W; e += (unsigned)G * kPlanWarps) eval_warp(A, L, wl[e], lane);
            if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }
            {
                const Cand bestF = scan_owned(A, L, Pn, false, win, par, &s_best, s_cand, s_k, s_i, s_tk, s_ti);
                if (threadIdx.x == 0) store_prop(&L.props[(size_t)pbuf * kLazyMaxBlocks + c], bestF, s_tk, s_ti);
            }
            if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }
            rbuf = pbuf;
            pbuf ^= 1;
            gBest = load_best(rbuf);
        }
        load_bounds(rbuf, false);
        int n_pool = G * kTopT;
        if (few_dirty) {
            for (unsigned e = threadIdx.x; e < W; e += kPlanThreads) {
                const int p = wl[e];
                const bool live = __ldcg(&L.c_state[p]) != 0;
                s_pkey[n_pool + e] = __longlong_as_double(0x7ff0000000000000ll);
                s_pidx[n_pool + e] = live ? p : -1;
                s_pdone[n_pool + e] = 0;
            }
            n_pool += (int)W;
            __syncthreads();
        }

        // ---------------- R: rounds of joint rescoring
        bool failed = false;
        int round_no = 0;
#pragma unroll 1
        for (;;) {
            const double gkey = gBest.idx >= 0 ? cand_key(gBest) : -1.0;
            int msel = 0;
            {
                // which published bounds are rescored now (same choice in every block, in publication order):
                // every unused one that may beat the best exact score -- in the first round of an iteration only those
                // within 10 % of the best bound (the winner is usually among them, and a strong exact score spares the
                // rest).  Bounds that cannot beat the best exact score are set aside for good.
                double floor0 = -1.0;
                if (round_no == 0) {
                    double k = -1.0;
                    int e_best = -1;
                    for (int e = threadIdx.x; e < n_pool; e += kPlanThreads)
                        if (!s_pdone[e] && s_pidx[e] >= 0 && s_pkey[e] > k && s_pkey[e] < 1e300) { k = s_pkey[e]; e_best = e; }
                    block_max_key(k, e_best, s_k, s_i);
                    floor0 = 0.9 * k;
                }
                int base = 0;
#pragma unroll 1
                for (int e0 = 0; e0 < n_pool; e0 += kPlanThreads) {
                    const int e = e0 + threadIdx.x;
                    bool take = false;
                    if (e < n_pool && !s_pdone[e] && s_pidx[e] >= 0 && s_pkey[e] >= floor0) {
                        take = bound_may_beat(L, s_pidx[e], s_pkey[e], gkey, &gBest);
                        if (!take) s_pdone[e] = 4;
                    }
                    const unsigned mk = __ballot_sync(0xffffffffu, take);
                    if (lane == 0) s_wcnt[warp] = __popc(mk);
                    __syncthreads();
                    int before = base, total = base;
                    for (int w2 = 0; w2 < kPlanWarps; ++w2) { if (w2 < warp) before += s_wcnt[w2]; total += s_wcnt[w2]; }
                    const int pos = before + __popc(mk & ((1u << lane) - 1u));
                    if (take && pos < kRoundM) { s_sel[pos] = e; s_pdone[e] = 1; }     // beyond the cap: next round
                    base = total;
                    __syncthreads();
                }
                msel = base < kRoundM ? base : kRoundM;
                // what the rescoring needs to know of each chosen period, fetched once, all of them together
                for (int r = threadIdx.x; r < msel; r += kPlanThreads) {
                    const int p = s_pidx[s_sel[r]];
                    const int d = (__ldcg(&L.c_state[p]) & 3) - 1;
                    s_it_d[r] = d;
                    s_it_ap[r] = A.geo_a[d * A.geo_stride + p]; s_it_bp[r] = A.geo_b[d * A.geo_stride + p];
                    s_it_s[r] = A.bytes[A.per_t[p]];
                    s_it_cost[r] = 2ull * (ull)A.geo_t[d * A.geo_stride + p];
                }
            }
            __syncthreads();
            if (msel == 0) {
                if (round_no == 0) { round_no = 1; continue; }      // (the first round only looks at the best bounds)
                // nothing published may beat the best score.  A block that has used all its bounds may hold more.
                if (threadIdx.x == 0) s_flag = 0;
                __syncthreads();
                for (int j = threadIdx.x; j < G; j += kPlanThreads) {
                    bool all = true;
                    for (int q = 0; q < kTopT; ++q) if (s_pidx[j * kTopT + q] < 0 || !s_pdone[j * kTopT + q]) all = false;
                    const double lastk = s_pkey[j * kTopT + kTopT - 1];
                    const bool again = all && lastk > 0.0 && (gBest.idx < 0 || lastk >= gkey * (1.0 - 1e-10));
                    s_refresh[j] = again ? 1 : 0;
                    if (again) s_flag = 1;
                }
                __syncthreads();
                if (!s_flag) break;
                if (s_refresh[c]) {
                    const Cand bestF = scan_owned(A, L, Pn, false, win, par, &s_best, s_cand, s_k, s_i, s_tk, s_ti, &gBest);
                    if (threadIdx.x == 0) store_prop(&L.props[(size_t)pbuf * kLazyMaxBlocks + c], bestF, s_tk, s_ti);
                }
                if (!grid_barrier(A.bar, G, gen)) { failed = true; break; }
                barrier_since_booking = true;
                load_bounds(pbuf, true);
                pbuf ^= 1;
                continue;
            }
            round_no += 1;
            // every block sums its share of each chosen period's absent range: tiles ta + c, ta + c + G, ... of the
            // range.  One thread per period classifies its tiles from their pressure minima / maxima (a tile wholly
            // at least s above capacity counts s for its whole time, one wholly within capacity nothing); the few
            // tiles in between are read slot by slot, one warp each.
            for (int r = threadIdx.x; r < msel; r += kPlanThreads) { s_acc[2 * r] = 0; s_acc[2 * r + 1] = 0; }
            if (threadIdx.x == 0) s_nmix = 0;
            __syncthreads();
            {
                int nsub = 1;                                    // threads per period (a power of two)
                while (nsub < 8 && 2 * nsub * msel <= kPlanThreads) nsub *= 2;
                const int r = (int)threadIdx.x / nsub, sub = (int)threadIdx.x % nsub;
                if (r < msel) {
                    const int ap = s_it_ap[r], bp = s_it_bp[r];
                    const int64_t sz = s_it_s[r];
                    u128 acc = 0;
                    const int ta = ap / kSlotTile, tb = bp / kSlotTile;
                    // (which block takes the range's first tile rotates with the period: ranges shorter than G tiles would
                    // otherwise all land on the low-numbered blocks)
                    const int ce = (c + r * 37) % G;
                    for (int tl = ta + ce + sub * G; tl <= tb; tl += nsub * G) {
                        const int64_t t0 = (int64_t)tl * kSlotTile, t1 = t0 + kSlotTile - 1;
                        const int k_lo = (int)(t0 > ap ? t0 : ap), k_hi = (int)(t1 < bp ? t1 : bp);
                        const long long mn = L.tmin[tl], mx = L.tmax[tl];
                        if (mx <= A.cap) continue;
                        if (mn >= A.cap && mn - A.cap >= sz) { acc += (u128)(ull)sz * (u128)(ull)(A.start[k_hi + 1] - A.start[k_lo]); continue; }
                        const int pos = atomicAdd(&s_nmix, 1);
                        if (pos < kMixCap) s_mix[pos] = (r << 22) | tl;
                        else acc += benefit_partial(A, k_lo, k_hi, sz, 0, 1);          // list full: this thread reads the tile itself
                    }
                    if (acc != 0) {
                        const ull lo = (ull)acc;
                        const ull old = atomicAdd(&s_acc[2 * r], lo);
                        atomicAdd(&s_acc[2 * r + 1], (ull)(acc >> 64) + (old + lo < old ? 1ull : 0ull));
                    }
                }
            }
            __syncthreads();
            {
                const int nmix = s_nmix < kMixCap ? s_nmix : kMixCap;
#pragma unroll 1
                for (int m = warp; m < nmix; m += kPlanWarps) {
                    const int r = s_mix[m] >> 22, tl = s_mix[m] & ((1 << 22) - 1);
                    const int ap = s_it_ap[r], bp = s_it_bp[r];
                    const int64_t t0 = (int64_t)tl * kSlotTile, t1 = t0 + kSlotTile - 1;
                    const int k_lo = (int)(t0 > ap ? t0 : ap), k_hi = (int)(t1 < bp ? t1 : bp);
                    const u128 acc = warp_sum_u128(benefit_tile_warp(A, k_lo, k_hi, s_it_s[r], lane));
                    if (lane == 0) {
                        const ull lo = (ull)acc;
                        const ull old = atomicAdd(&s_acc[2 * r], lo);
                        atomicAdd(&s_acc[2 * r + 1], (ull)(acc >> 64) + (old + lo < old ? 1ull : 0ull));
                    }
                }
            }
            __syncthreads();
            // this block's shares go into the grid-wide 128-bit sums (low word first; its carry goes with the high word)
            for (int r = threadIdx.x; r < msel; r += kPlanThreads) {
                const ull lo = s_acc[2 * r], hi = s_acc[2 * r + 1];
                if (lo | hi) {
                    ull *dst = L.partials + ((size_t)pp * kRoundM + r) * 2;
                    const ull old = atomicAdd(&dst[0], lo);
                    const ull up = hi + (old + lo < old ? 1ull : 0ull);
                    if (up) atomicAdd(&dst[1], up);
                }
            }
            if (!grid_barrier(A.bar, G, gen)) { failed = true; break; }
            barrier_since_booking = true;
            // the buffer used two rounds from now was last read one round ago: block 0 clears it
            if (c == 0)
                for (int j = threadIdx.x; j < kRoundM * 2; j += kPlanThreads) L.partials[(size_t)((pp + 2) % 3) * kRoundM * 2 + j] = 0;
            // every block reads the sums; the owner of a period stores its new score
            for (int r = threadIdx.x; r < msel; r += kPlanThreads) {
                const int p = s_pidx[s_sel[r]];
                const int d = s_it_d[r];
                const ull *src = L.partials + ((size_t)pp * kRoundM + r) * 2;
                const u128 tot = ((u128)__ldcg(&src[1]) << 64) | __ldcg(&src[0]);
                Cand x;
                x.ben = tot; x.cost = s_it_cost[r]; x.idx = tot == 0 ? -1 : p; x.dest = d;
                s_new[r] = x;
                if ((int)((p / kPlanThreads) % G) == c) store_score(A, L, p, d, kFresh, tot, x.cost);
            }
            __syncthreads();
            {
                Cand x;
                x.ben = 0; x.cost = 1; x.idx = -1; x.dest = -1;
                if ((int)threadIdx.x < msel) x = s_new[threadIdx.x];
                const Cand b = block_best_fast(x, &s_best, s_cand);
                if (cand_beats(b, gBest)) gBest = b;
            }
            pp = (pp + 1) % 3;
            __syncthreads();
        }
        if (failed) { status = -2; break; }
        if (!barrier_since_booking) { if (!grid_barrier(A.bar, G, gen)) { status = -2; break; } }

        // ---------------- D: decide
        if (gBest.idx < 0) { status = G10_EXHAUSTED; break; }
        {
            const int64_t p = gBest.idx;
            const int X = gBest.dest;
            win.idx = gBest.idx; win.dest = X;
            win.a = A.per_u[p] + 1; win.b = A.per_v[p] - 1;
            win.ap = A.geo_a[X * A.geo_stride + p]; win.bp = A.geo_b[X * A.geo_stride + p];
            win.t = A.geo_t[X * A.geo_stride + p];
            win.t_r = A.start[win.a]; win.t_end = A.start[win.b + 1];
            const int64_t sz = A.bytes[A.per_t[p]];
            if (X == G10_DEST_SSD) bytes_ssd += sz; else bytes_host += sz;
        }
        n_mig += 1;
        pending = true;
    }
    plan_epilogue(A, c, G, gen, status, peak, n_mig, rounds, bytes_ssd, bytes_host);
}

constexpr size_t kLazyDynBytes = (size_t)kRoundM * (sizeof(Cand) + 2 * sizeof(ull) + sizeof(long long) + sizeof(ull) + 4 * sizeof(int));

int plan_lazy_blocks()
{
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaFuncSetAttribute(k_plan_lazy, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kLazyDynBytes) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_plan_lazy, kPlanThreads, kLazyDynBytes) != cudaSuccess) return 0;
    if (per_sm < 1) return 0;
    return sms > kLazyMaxBlocks ? kLazyMaxBlocks : sms;
}

cudaError_t launch_plan_lazy(const PlanArgs &A_in, const Workspace &w, int G, cudaStream_t s)
{
    PlanArgs A = A_in;
    LazyArgs L;
    L.c_state = w.c_state; L.c_ben_lo = w.c_ben_lo; L.c_ben_hi = w.c_ben_hi; L.c_cost = w.c_cost; L.c_key = w.c_key;
    L.c_rng = w.c_rng; L.worklist = w.worklist; L.wl_count = w.wl_count; L.props = w.lazy_props; L.partials = w.lazy_partials; L.stride = A.geo_stride;
    L.tmin = w.lazy_tmin; L.tmax = w.lazy_tmax;
    void *args[] = {&A, &L};
    const cudaError_t e = cudaFuncSetAttribute(k_plan_lazy, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kLazyDynBytes);
    if (e != cudaSuccess) return e;
    return cudaLaunchCooperativeKernel((const void *)k_plan_lazy, dim3(G), dim3(kPlanThreads), args, kLazyDynBytes, s);
}

}  // namespace g10

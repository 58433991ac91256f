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
// comparisons each).  DIRTY periods are rescored at once; a STALE period is rescored only while its bound may
// still beat the best exact score known, so that when the iteration decides, the committed score is the exact
// maximum over all live periods, ties included (see k_plan_lazy).
#include <cstdio>

#include "g10_planner.cuh"

namespace g10 {

constexpr int kLazyMaxBlocks = 256;
enum { kFresh = 1, kStale = 2, kDirty = 3 };

struct LazyArgs {
    unsigned char *c_state;     // 0 = erased; else (dest + 1) | (state << 2)
    ull *c_ben_lo, *c_ben_hi;   // last computed benefit
    ull *c_cost;                // 2 t of the current destination
    double *c_key;              // rounded benefit / cost of the cached score (steers the search; decisions are exact)
    int *worklist;              // [2][stride] DIRTY periods of the current round
    unsigned *wl_count;         // [2]
    Proposal *prop_stale;       // [G] each block's exact best of step C (second proposal buffer)
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

__device__ __forceinline__ void store_score(const LazyArgs &L, int64_t p, int dest, int state, u128 ben, ull cost)
{
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
        if (lane == 0) store_score(L, p, cd.dest, kFresh, cd.ben, cd.cost);
        return;
    }
    const int d = (st & 3) - 1;
    const int ap = A.geo_a[d * A.geo_stride + p], bp = A.geo_b[d * A.geo_stride + p];
    const int64_t s = A.bytes[A.per_t[p]];
    u128 acc = warp_sum_u128(benefit_partial(A, ap, bp, s, lane, 32));
    if (lane == 0) store_score(L, p, d, kFresh, acc, 2ull * (ull)A.geo_t[d * A.geo_stride + p]);
}

// The whole block brings period p up to date (long absent ranges).
__device__ __forceinline__ void eval_block(const PlanArgs &A, const LazyArgs &L, int64_t p, int *s_dest, ull *s_part /* [2*kPlanWarps] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned char st = L.c_state[p];
    if (st == 0) return;                       // uniform across the block
    int d = (st & 3) - 1;
    if ((st >> 2) == kDirty) {
        __syncthreads();
        if (warp == 0) {
            // destination rule: SSD first, then host; the windows are short, one warp checks them
            const int u = A.per_u[p], v = A.per_v[p];
            const int a = u + 1, b = v - 1;
            const int64_t s = A.bytes[A.per_t[p]];
            const int64_t t_r = A.start[a], t_end = A.start[v];
            int dest = -1;
            for (int X = 0; X < 2 && dest < 0; ++X) {
                const int ap = A.geo_a[X * A.geo_stride + p];
                if (ap < 0) continue;
                const int bp = A.geo_b[X * A.geo_stride + p];
                const int64_t t = A.geo_t[X * A.geo_stride + p];
                if (!window_free(A, A.busy + (size_t)(2 * X) * A.K, t_r, t_r + t, a, ap - 1, lane)) continue;
                if (!window_free(A, A.busy + (size_t)(2 * X + 1) * A.K, t_end - t, t_end, bp + 1, b, lane)) continue;
                if (X == G10_DEST_HOST && A.host_capacity != 0) {
                    bool ok = true;
                    for (int k = a + lane; k <= b; k += 32)
                        if ((uint64_t)A.hocc[k] + (uint64_t)s > A.host_capacity) ok = false;
                    if (!__all_sync(0xffffffffu, ok)) continue;
                }
                dest = X;
            }
            if (lane == 0) *s_dest = dest;
        }
        __syncthreads();
        d = *s_dest;
        if (d < 0) { if (threadIdx.x == 0) L.c_state[p] = 0; return; }
    }
    const int ap = A.geo_a[d * A.geo_stride + p], bp = A.geo_b[d * A.geo_stride + p];
    const int64_t s = A.bytes[A.per_t[p]];
    u128 acc = warp_sum_u128(benefit_partial(A, ap, bp, s, threadIdx.x, kPlanThreads));
    __syncthreads();
    if (lane == 0) { s_part[2 * warp] = (ull)acc; s_part[2 * warp + 1] = (ull)(acc >> 64); }
    __syncthreads();
    if (threadIdx.x == 0) {
        u128 tot = 0;
        for (int w = 0; w < kPlanWarps; ++w) tot += ((u128)s_part[2 * w + 1] << 64) | s_part[2 * w];
        store_score(L, p, d, kFresh, tot, 2ull * (ull)A.geo_t[d * A.geo_stride + p]);
    }
}

__device__ __forceinline__ Cand load_proposal(const Proposal *pr)
{
    Cand x;
    const ull lo = __ldcg(&pr->ben_lo), hi = __ldcg(&pr->ben_hi);
    x.ben = ((u128)hi << 64) | lo;
    x.cost = __ldcg(&pr->cost);
    x.idx = __ldcg(&pr->idx);
    x.dest = __ldcg(&pr->dest);
    return x;
}
__device__ __forceinline__ void store_proposal(Proposal *pr, const Cand &c)
{
    Proposal q;
    q.ben_lo = (ull)c.ben; q.ben_hi = (ull)(c.ben >> 64); q.cost = c.cost; q.idx = c.idx; q.dest = c.dest;
    *pr = q;
}

// Best STALE bound of the block by rounded ratio (any of several equal ones): uniform result.
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

// One pass of a block over the periods it owns.  With `classify` the pending winner's slot ranges are applied
// first (FRESH -> STALE where its absent range meets theirs, -> DIRTY where a booked window meets theirs) and
// DIRTY periods are appended to the work list.  Returns the block's best FRESH candidate (exact) and its best
// STALE bound (rounded ratio and period, approximate on purpose: it only says what to rescore next).
struct ScanResult {
    Cand bestF;
    double keyS;
    int idxS;
};

struct Winner {
    int idx, dest, a, ap, bp, b;      // evict slots [a, ap-1], absent [ap, bp], prefetch [bp+1, b]
};

__device__ __forceinline__ ScanResult scan_owned(const PlanArgs &A, const LazyArgs &L, int64_t Pn, bool classify, const Winner &w,
                                                 int par, BestScratch *sc, Cand *s_cand, double *s_k, int *s_i)
{
    const int G = gridDim.x, c = blockIdx.x, lane = threadIdx.x & 31;
    double kf = -1.0, ks = -1.0;
    int pf = -1, ps = -1;
    for (int64_t p0 = (int64_t)c * kPlanThreads; p0 < Pn; p0 += (int64_t)G * kPlanThreads) {
        const int64_t p = p0 + threadIdx.x;
        bool dirty = false;
        if (p < Pn) {
            unsigned char st = L.c_state[p];
            if (st != 0) {
                int state = st >> 2;
                const int d = (st & 3) - 1;
                if (classify) {
                    if (p == w.idx) { L.c_state[p] = 0; st = 0; }
                    else if (state != kDirty) {
                        const int u = A.per_u[p], v = A.per_v[p];
                        if (u + 1 <= w.b && w.a <= v - 1) {          // the two periods share slots
                            const int ap = A.geo_a[d * A.geo_stride + p], bp = A.geo_b[d * A.geo_stride + p];
                            bool hit = false;
                            if (d == w.dest) {
                                hit = (u + 1 <= w.ap - 1 && w.a <= ap - 1) || (bp + 1 <= w.b && w.bp + 1 <= v - 1);
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
                        const double key = L.c_key[p];
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
                            } else if (key > ks) { ks = key; ps = (int)p; }
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
            }
        }
    }
    ScanResult r;
    Cand x;
    x.ben = 0; x.cost = 1; x.idx = -1; x.dest = -1;
    if (pf >= 0) {
        x.ben = ((u128)L.c_ben_hi[pf] << 64) | L.c_ben_lo[pf]; x.cost = L.c_cost[pf]; x.idx = pf;
        x.dest = (L.c_state[pf] & 3) - 1;
    }
    r.bestF = block_best_fast(x, sc, s_cand);
    block_max_key(ks, ps, s_k, s_i);
    r.keyS = ks; r.idxS = ps;
    return r;
}

// Could a STALE bound with rounded ratio `key` beat (or tie with) candidate t?  Conservative by 1e-10.
__device__ __forceinline__ bool may_beat(double key, const Cand &t)
{
    if (!(key > 0.0)) return false;
    if (t.idx < 0) return true;
    return key >= cand_key(t) * (1.0 - 1e-10);
}

// Per iteration: (A) every block applies the previous commit to the slots it owns, classifies the periods it
// owns and finds its best FRESH candidate and best STALE bound; (B) after the first grid barrier every block
// knows the best FRESH score of the grid: DIRTY periods are rescored (shared out over the grid) and each block
// rescores its own best STALE period if the bound may beat that score; (C) each block then makes its own best
// exact -- it rescores its STALE periods, best bound first, while the bound may beat the better of the grid's
// FRESH score and its own best; (D) after the last barrier the maximum of the blocks' exact bests is the exact
// maximum over all live periods (every period left STALE has a bound below its block's best) and is committed.
__global__ void __launch_bounds__(kPlanThreads, 1) k_plan_lazy(PlanArgs A, LazyArgs L)
{
    __shared__ Cand s_cand[kPlanWarps + 1];
    __shared__ BestScratch s_best;
    __shared__ long long s_max[kPlanWarps + 1];
    __shared__ double s_k[kPlanWarps];
    __shared__ int s_i[kPlanWarps];
    __shared__ int s_dest;
    __shared__ ull s_part[2 * kPlanWarps];
    const int G = gridDim.x, c = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t Pn = *A.Pn_dev < A.geo_stride ? *A.Pn_dev : A.geo_stride;
    const int64_t limit = (A.max_iterations <= 0 || A.max_iterations > Pn) ? Pn : A.max_iterations;
    unsigned gen = 0;
    int64_t n_mig = 0, rounds = 0, bytes_ssd = 0, bytes_host = 0;
    int status = -1;
    long long peak = 0;
    int par = 0;                               // which worklist buffer this iteration fills
#ifdef G10_PHASE_CLOCKS
    long long dbg_dirty = 0, dbg_top = 0, dbg_local = 0;
#endif

    // every period starts DIRTY: its first evaluation chooses the destination
    for (int64_t p = (int64_t)c * kPlanThreads + threadIdx.x; p < Pn; p += (int64_t)G * kPlanThreads) {
        L.c_state[p] = (unsigned char)(kDirty << 2);
        L.c_key[p] = 0.0;
    }
    {
        const long long m = own_slots_max(A, c, G, s_max);
        if (threadIdx.x == 0) A.peak_part[c] = m;
    }
    if (!grid_barrier(A.bar, G, gen)) status = -2;

    bool pending = false;                      // a commit decided in the previous iteration, not yet applied
    Winner win;
    win.idx = -1; win.dest = -1; win.a = 0; win.ap = 0; win.bp = -1; win.b = -1;

    for (int64_t it = 0; status == -1; ++it) {
        // ---------------- apply the pending commit to what this block owns
        if (pending) {
            int64_t sz = 0;
            const bool touched = commit_winner(A, win.idx, win.dest, it - 1, n_mig - 1, c, G, &sz);
            if (touched) {
                const long long m = own_slots_max(A, c, G, s_max);
                if (threadIdx.x == 0) A.peak_part[c] = m;
            }
        }
        // ---------------- A: classify the owned periods against the commit, collect DIRTY ones, local bests
        // (on the first iteration `win` matches nothing and every period is DIRTY)
        ScanResult sr = scan_owned(A, L, Pn, true, win, par, &s_best, s_cand, s_k, s_i);
        if (threadIdx.x == 0) store_proposal(&A.proposals[c], sr.bestF);
        pending = false;
        if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }

        // ---------------- B: global best FRESH score so far, peak, stop tests; rescore DIRTY periods (shared
        // out over the grid) and this block's best STALE period if its bound may beat that score
        Cand gF;
        gF.ben = 0; gF.cost = 1; gF.idx = -1; gF.dest = -1;
        long long m = 0;
        for (int j = threadIdx.x; j < G; j += kPlanThreads) {
            const long long pm = __ldcg(&A.peak_part[j]);
            if (pm > m) m = pm;
            const Cand x = load_proposal(&A.proposals[j]);
            if (cand_beats(x, gF)) gF = x;
        }
        peak = block_max_i64(m, s_max);
        gF = block_best_fast(gF, &s_best, s_cand);
        const unsigned W = __ldcg(&L.wl_count[par]);
        if (A.fits_always || peak <= A.cap) { status = n_mig == 0 ? G10_ALREADY_FITS : G10_FIT; break; }
        if (it >= limit) { status = limit < Pn ? G10_ITERATION_LIMIT : G10_EXHAUSTED; break; }
        rounds += 1;
        const int *wl = L.worklist + (size_t)par * L.stride;
        if (W <= 2u * (unsigned)G) {
            for (unsigned e = c; e < W; e += G) eval_block(A, L, wl[e], &s_dest, s_part);
        } else {
            for (unsigned e = (unsigned)c * kPlanWarps + warp; e < W; e += (unsigned)G * kPlanWarps) eval_warp(A, L, wl[e], lane);
        }
        if (sr.idxS >= 0 && may_beat(sr.keyS, gF)) {
            eval_block(A, L, sr.idxS, &s_dest, s_part);
#ifdef G10_PHASE_CLOCKS
            dbg_top += 1;
#endif
        }
#ifdef G10_PHASE_CLOCKS
        dbg_dirty += W;
#endif
        if (c == 0 && threadIdx.x == 0) L.wl_count[par ^ 1] = 0;
        par ^= 1;
        if (W > 0) {                               // DIRTY periods were rescored by other blocks than their owners
            if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }
        } else __syncthreads();

        // ---------------- C: make this block's best exact
        Cand localF;
        for (;;) {
            sr = scan_owned(A, L, Pn, false, win, par, &s_best, s_cand, s_k, s_i);
            localF = sr.bestF;
            const Cand &thr = cand_beats(localF, gF) ? localF : gF;
            if (sr.idxS >= 0 && may_beat(sr.keyS, thr)) {
                eval_block(A, L, sr.idxS, &s_dest, s_part);
                __syncthreads();
#ifdef G10_PHASE_CLOCKS
                dbg_local += 1;
#endif
                continue;
            }
            break;
        }
        if (threadIdx.x == 0) store_proposal(&L.prop_stale[c], localF);      // second buffer: step A reuses the first
        if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }

        // ---------------- D: the exact global argmax; decide
        Cand best;
        best.ben = 0; best.cost = 1; best.idx = -1; best.dest = -1;
        for (int j = threadIdx.x; j < G; j += kPlanThreads) {
            const Cand x = load_proposal(&L.prop_stale[j]);
            if (cand_beats(x, best)) best = x;
        }
        best = block_best_fast(best, &s_best, s_cand);
        if (best.idx < 0) { status = G10_EXHAUSTED; break; }
        {
            const int64_t p = best.idx;
            const int X = best.dest;
            win.idx = best.idx; win.dest = X;
            win.a = A.per_u[p] + 1; win.b = A.per_v[p] - 1;
            win.ap = A.geo_a[X * A.geo_stride + p]; win.bp = A.geo_b[X * A.geo_stride + p];
            const int64_t sz = A.bytes[A.per_t[p]];
            if (X == G10_DEST_SSD) bytes_ssd += sz; else bytes_host += sz;
        }
        n_mig += 1;
        pending = true;
    }
#ifdef G10_PHASE_CLOCKS
    if (threadIdx.x == 0 && (c == 0 || c == 77))
        printf("k_plan_lazy block %d: iterations %lld, DIRTY rescored (grid) %lld, own top STALE rescored %lld, further STALE rescored %lld\n",
               c, (long long)rounds, dbg_dirty, dbg_top, dbg_local);
#endif
    plan_epilogue(A, c, G, gen, status, peak, n_mig, rounds, bytes_ssd, bytes_host);
}

int plan_lazy_blocks()
{
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_plan_lazy, kPlanThreads, 0) != cudaSuccess) return 0;
    if (per_sm < 1) return 0;
    return sms > kLazyMaxBlocks ? kLazyMaxBlocks : sms;
}

cudaError_t launch_plan_lazy(const PlanArgs &A_in, const Workspace &w, int G, cudaStream_t s)
{
    PlanArgs A = A_in;
    LazyArgs L;
    L.c_state = w.c_state; L.c_ben_lo = w.c_ben_lo; L.c_ben_hi = w.c_ben_hi; L.c_cost = w.c_cost; L.c_key = w.c_key;
    L.worklist = w.worklist; L.wl_count = w.wl_count; L.prop_stale = w.prop_stale; L.stride = A.geo_stride;
    void *args[] = {&A, &L};
    return cudaLaunchCooperativeKernel((const void *)k_plan_lazy, dim3(G), dim3(kPlanThreads), args, 0, s);
}

}  // namespace g10

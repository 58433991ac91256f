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
// After a commit every block classifies its share of the periods against the winner's slot ranges (a few
// integer comparisons each).  An iteration then alternates argmax rounds (best FRESH score; best STALE bound
// per block) and evaluation rounds (all DIRTY periods, and the few best STALE periods whose bound still beats
// the best FRESH score) until no DIRTY period is left and no STALE bound beats the best FRESH score: that
// score is then the exact maximum over all live periods, ties included, and is committed.
#include "g10_planner.cuh"

namespace g10 {

constexpr int kLazyMaxBlocks = 256;
constexpr int kStaleBatch = 8;           // STALE periods rescored per evaluation round, at most
enum { kFresh = 1, kStale = 2, kDirty = 3 };

struct LazyArgs {
    unsigned char *c_state;     // 0 = erased; else (dest + 1) | (state << 2)
    ull *c_ben_lo, *c_ben_hi;   // last computed benefit
    ull *c_cost;                // 2 t of the current destination
    int *worklist;              // [2][stride] DIRTY periods of the current round
    unsigned *wl_count;         // [2]
    Proposal *prop_stale;       // [G] best STALE bound of each block
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

__global__ void __launch_bounds__(kPlanThreads, 1) k_plan_lazy(PlanArgs A, LazyArgs L)
{
    __shared__ Cand s_cand[kPlanWarps + 1];
    __shared__ long long s_max[kPlanWarps + 1];
    __shared__ Cand s_stale[kLazyMaxBlocks];
    __shared__ int s_sel[kStaleBatch];
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
    int par = 0;                               // which worklist buffer this round fills

    // every period starts DIRTY: its first evaluation chooses the destination
    for (int64_t p = (int64_t)c * kPlanThreads + threadIdx.x; p < Pn; p += (int64_t)G * kPlanThreads)
        L.c_state[p] = (unsigned char)(kDirty << 2);
    {
        const long long m = own_slots_max(A, c, G, s_max);
        if (threadIdx.x == 0) A.peak_part[c] = m;
    }
    if (!grid_barrier(A.bar, G, gen)) status = -2;

    bool pending = false;                      // a commit decided in the previous iteration, not yet applied
    Cand win;
    win.ben = 0; win.cost = 1; win.idx = -1; win.dest = -1;
    int wa = 0, wap = 0, wbp = -1, wb = -1;    // winner's slot ranges: evict [wa, wap-1], absent [wap, wbp], prefetch [wbp+1, wb]

    for (int64_t it = 0; status == -1; ++it) {
        bool first_round = true;
        bool decided = false;
        while (!decided) {
            // ---------------- apply the pending commit to what this block owns
            if (pending) {
                int64_t sz = 0;
                const bool touched = commit_winner(A, win.idx, win.dest, it - 1, n_mig - 1, c, G, &sz);
                if (touched) {
                    const long long m = own_slots_max(A, c, G, s_max);
                    if (threadIdx.x == 0) A.peak_part[c] = m;
                }
            }
            // ---------------- argmax round over this block's share of the periods
            Cand bestF, bestS;
            bestF.ben = 0; bestF.cost = 1; bestF.idx = -1; bestF.dest = -1;
            bestS = bestF;
            for (int64_t p0 = (int64_t)c * kPlanThreads; p0 < Pn; p0 += (int64_t)G * kPlanThreads) {
                const int64_t p = p0 + threadIdx.x;
                bool dirty = false;
                if (p < Pn) {
                    unsigned char st = L.c_state[p];
                    if (st != 0) {
                        int state = st >> 2;
                        const int d = (st & 3) - 1;
                        if (pending) {
                            if (p == win.idx) { L.c_state[p] = 0; st = 0; }
                            else if (state != kDirty) {
                                const int u = A.per_u[p], v = A.per_v[p];
                                if (u + 1 <= wb && wa <= v - 1) {          // the two periods share slots
                                    const int ap = A.geo_a[d * A.geo_stride + p], bp = A.geo_b[d * A.geo_stride + p];
                                    bool hit = false;
                                    if (d == win.dest) {
                                        hit = (u + 1 <= wap - 1 && wa <= ap - 1) || (bp + 1 <= wb && wbp + 1 <= v - 1);
                                        if (!hit && d == G10_DEST_HOST && A.host_capacity != 0) hit = true;
                                    }
                                    if (hit) state = kDirty;
                                    else if (state == kFresh && ap <= wbp && wap <= bp) state = kStale;
                                    if (state != (st >> 2)) { st = (unsigned char)((st & 3) | (state << 2)); L.c_state[p] = st; }
                                }
                            }
                        }
                        if (st != 0) {
                            if (state == kDirty) dirty = true;
                            else {
                                Cand x;
                                x.ben = ((u128)L.c_ben_hi[p] << 64) | L.c_ben_lo[p];
                                if (x.ben > 0) {
                                    x.cost = L.c_cost[p]; x.idx = (int)p; x.dest = d;
                                    if (state == kFresh) { if (cand_beats(x, bestF)) bestF = x; }
                                    else if (cand_beats(x, bestS)) bestS = x;
                                }
                            }
                        }
                    }
                }
                // DIRTY periods go on the work list (one atomic per warp)
                const unsigned md = __ballot_sync(0xffffffffu, dirty);
                if (md) {
                    unsigned base = 0;
                    if (lane == 0) base = atomicAdd(&L.wl_count[par], (unsigned)__popc(md));
                    base = __shfl_sync(0xffffffffu, base, 0);
                    if (dirty) L.worklist[(size_t)par * L.stride + base + __popc(md & ((1u << lane) - 1u))] = (int)p;
                }
            }
            bestF = block_best(bestF, s_cand);
            bestS = block_best(bestS, s_cand);
            if (threadIdx.x == 0) { store_proposal(&A.proposals[c], bestF); store_proposal(&L.prop_stale[c], bestS); }
            pending = false;
            if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }

            // ---------------- every block: best FRESH score, peak, work list length, STALE bounds that still compete
            Cand gF;
            gF.ben = 0; gF.cost = 1; gF.idx = -1; gF.dest = -1;
            long long m = 0;
            for (int j = threadIdx.x; j < G; j += kPlanThreads) {
                const long long pm = __ldcg(&A.peak_part[j]);
                if (pm > m) m = pm;
                const Cand x = load_proposal(&A.proposals[j]);
                if (cand_beats(x, gF)) gF = x;
                s_stale[j] = load_proposal(&L.prop_stale[j]);
            }
            peak = block_max_i64(m, s_max);
            gF = block_best(gF, s_cand);
            const unsigned W = __ldcg(&L.wl_count[par]);
            if (first_round) {
                if (A.fits_always || peak <= A.cap) { status = n_mig == 0 ? G10_ALREADY_FITS : G10_FIT; break; }
                if (it >= limit) { status = limit < Pn ? G10_ITERATION_LIMIT : G10_EXHAUSTED; break; }
                rounds += 1;
                first_round = false;
            }
            // rank the STALE proposals that beat the best FRESH score; the kStaleBatch best are rescored
            bool qual = false;
            int rank = 0;
            if (threadIdx.x < G) {
                const Cand me = s_stale[threadIdx.x];
                qual = me.idx >= 0 && cand_beats(me, gF);
                if (qual)
                    for (int j = 0; j < G; ++j)
                        if (j != (int)threadIdx.x && cand_beats(s_stale[j], me)) ++rank;
                if (qual && rank < kStaleBatch) s_sel[rank] = me.idx;
            }
            int nS = __syncthreads_count(qual);
            if (nS > kStaleBatch) nS = kStaleBatch;
            if (W == 0 && nS == 0) {
                // nothing can beat the best FRESH score: decide
                if (gF.idx < 0) { status = G10_EXHAUSTED; break; }
                win = gF;
                {
                    const int64_t p = win.idx;
                    const int X = win.dest;
                    wa = A.per_u[p] + 1; wb = A.per_v[p] - 1;
                    wap = A.geo_a[X * A.geo_stride + p]; wbp = A.geo_b[X * A.geo_stride + p];
                    const int64_t sz = A.bytes[A.per_t[p]];
                    if (X == G10_DEST_SSD) bytes_ssd += sz; else bytes_host += sz;
                }
                n_mig += 1;
                pending = true;
                decided = true;
                break;
            }
            // ---------------- evaluation round
            const unsigned T = W + (unsigned)nS;
            const int *wl = L.worklist + (size_t)par * L.stride;
            if (T <= 2u * (unsigned)G) {
                for (unsigned e = c; e < T; e += G) {
                    const int64_t p = e < W ? wl[e] : s_sel[e - W];
                    eval_block(A, L, p, &s_dest, s_part);
                }
            } else {
                for (unsigned e = (unsigned)c * kPlanWarps + warp; e < T; e += (unsigned)G * kPlanWarps) {
                    const int64_t p = e < W ? wl[e] : s_sel[e - W];
                    eval_warp(A, L, p, lane);
                }
            }
            if (c == 0 && threadIdx.x == 0) L.wl_count[par ^ 1] = 0;
            par ^= 1;
            if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }
        }
    }
    // a commit decided in the very last iteration is always applied above before the loop can end:
    // the loop only ends at a first-round test or at an empty argmax, both of which follow the apply step.
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
    L.c_state = w.c_state; L.c_ben_lo = w.c_ben_lo; L.c_ben_hi = w.c_ben_hi; L.c_cost = w.c_cost;
    L.worklist = w.worklist; L.wl_count = w.wl_count; L.prop_stale = w.prop_stale; L.stride = A.geo_stride;
    void *args[] = {&A, &L};
    return cudaLaunchCooperativeKernel((const void *)k_plan_lazy, dim3(G), dim3(kPlanThreads), args, 0, s);
}

}  // namespace g10

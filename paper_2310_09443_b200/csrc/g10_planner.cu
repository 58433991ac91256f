// Algorithm 1 (smart tensor eviction) as one persistent cooperative kernel: every iteration scores
// the live inactive periods in parallel, reduces the best benefit/cost ratio across the grid, commits
// it (pressure range-subtract, channel bookings, host occupancy) and tests the peak, with two grid
// barriers per iteration and no host round trip.
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

// Is the channel free for the window [w0, w1) over slots k0..k1?  Each slot offers dur[k] ns of channel
// time per device and direction; the window may be booked iff booked + overlap <= dur in every slot.
// Called by a whole warp; returns the same answer in every lane.
__device__ __forceinline__ bool window_free(const PlanArgs &A, const int64_t *busy, int64_t w0, int64_t w1, int k0, int k1, int lane)
{
    bool ok = true;
    for (int k = k0 + lane; k <= k1; k += 32) {
        const int64_t s0 = A.start[k], s1 = A.start[k + 1];
        const int64_t lo = w0 > s0 ? w0 : s0, hi = w1 < s1 ? w1 : s1;
        const int64_t ov = hi > lo ? hi - lo : 0;
        if (busy[k] + ov > s1 - s0) ok = false;
    }
    return __all_sync(0xffffffffu, ok);
}

// Scores period p against the current state: destination (SSD first, then host) and benefit.
// Whole warp; result valid in lane 0.  Returns false if no destination is admissible (permanent).
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
    if (dest < 0) return false;
    u128 acc = 0;
    for (int k = ap + lane; k <= bp; k += 32) {
        int64_t ex = A.P[k] - A.cap;
        if (ex > 0) {
            if (ex > s) ex = s;
            acc += (u128)(ull)ex * (u128)(ull)A.dur[k];
        }
    }
    acc = warp_sum_u128(acc);
    out->ben = acc; out->cost = 2ull * (ull)t; out->idx = (int)p; out->dest = dest;
    return true;
}

__global__ void __launch_bounds__(kPlanThreads, 1) k_plan_loop(PlanArgs A)
{
    __shared__ Cand s_cand[kPlanWarps];
    __shared__ long long s_max[kPlanWarps];
    __shared__ Cand s_win;
    __shared__ long long s_peak;
    const int G = gridDim.x, c = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t K = A.K;
    const int64_t Pn = *A.Pn_dev < A.geo_stride ? *A.Pn_dev : A.geo_stride;
    const int64_t limit = (A.max_iterations <= 0 || A.max_iterations > Pn) ? Pn : A.max_iterations;
    const int n_slot_tiles = (int)((K + kSlotTile - 1) / kSlotTile);
    unsigned gen = 0;
    int64_t n_mig = 0, rounds = 0, bytes_ssd = 0, bytes_host = 0;
    int status = -1;
    bool own_dirty = true;

    for (int64_t it = 0;; ++it) {
        // ---- (re)compute the max of the slots this block owns, if a commit touched them
        if (own_dirty) {
            long long m = 0;
            for (int tl = c; tl < n_slot_tiles; tl += G) {
                const int64_t k0 = (int64_t)tl * kSlotTile;
                for (int64_t k = k0 + threadIdx.x; k < k0 + kSlotTile && k < K; k += kPlanThreads) {
                    const long long pv = A.P[k];
                    if (pv > m) m = pv;
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) { const long long x = __shfl_down_sync(0xffffffffu, m, o); if (x > m) m = x; }
            if (lane == 0) s_max[warp] = m;
            __syncthreads();
            if (threadIdx.x == 0) {
                for (int w = 1; w < kPlanWarps; ++w) if (s_max[w] > m) m = s_max[w];
                A.peak_part[c] = m;
            }
            own_dirty = false;
        }
        // ---- score: one warp per live period
        Cand best;
        best.ben = 0; best.cost = 1; best.idx = -1; best.dest = -1;
        for (int64_t p = (int64_t)c * kPlanWarps + warp; p < Pn; p += (int64_t)G * kPlanWarps) {
            if (A.dead[p]) continue;
            Cand cd;
            if (!score_period(A, p, lane, &cd)) {
                if (lane == 0) A.dead[p] = 1;       // channels only fill up: never admissible again
                continue;
            }
            if (lane == 0 && cd.ben > 0 && cand_beats(cd, best)) best = cd;
        }
        if (lane == 0) s_cand[warp] = best;
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < kPlanWarps; ++w) if (cand_beats(s_cand[w], best)) best = s_cand[w];
            Proposal pr;
            pr.ben_lo = (ull)best.ben; pr.ben_hi = (ull)(best.ben >> 64); pr.cost = best.cost; pr.idx = best.idx; pr.dest = best.dest;
            A.proposals[c] = pr;
        }
        if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }

        // ---- reduce peak and proposals (every block, redundantly and identically)
        {
            long long m = 0;
            Cand w;
            w.ben = 0; w.cost = 1; w.idx = -1; w.dest = -1;
            for (int j = threadIdx.x; j < G; j += kPlanThreads) {
                const long long pm = __ldcg(&A.peak_part[j]);
                if (pm > m) m = pm;
                Cand x;
                const ull lo = __ldcg(&A.proposals[j].ben_lo), hi = __ldcg(&A.proposals[j].ben_hi);
                x.ben = ((u128)hi << 64) | lo;
                x.cost = __ldcg(&A.proposals[j].cost);
                x.idx = __ldcg(&A.proposals[j].idx);
                x.dest = __ldcg(&A.proposals[j].dest);
                if (cand_beats(x, w)) w = x;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const long long xm = __shfl_down_sync(0xffffffffu, m, o);
                if (xm > m) m = xm;
                const Cand x = cand_shfl_down(w, o);
                if (cand_beats(x, w)) w = x;
            }
            if (lane == 0) { s_max[warp] = m; s_cand[warp] = w; }
            __syncthreads();
            if (threadIdx.x == 0) {
                for (int q = 1; q < kPlanWarps; ++q) {
                    if (s_max[q] > m) m = s_max[q];
                    if (cand_beats(s_cand[q], w)) w = s_cand[q];
                }
                s_peak = m; s_win = w;
            }
            __syncthreads();
        }
        const long long peak = s_peak;
        const Cand win = s_win;
        if (A.fits_always || peak <= A.cap) { status = n_mig == 0 ? G10_ALREADY_FITS : G10_FIT; break; }
        if (it >= limit) { status = limit < Pn ? G10_ITERATION_LIMIT : G10_EXHAUSTED; break; }
        rounds += 1;
        if (win.idx < 0) { status = G10_EXHAUSTED; break; }

        // ---- commit the winner
        {
            const int64_t p = win.idx;
            const int X = win.dest;
            const int i = A.per_t[p], u = A.per_u[p], v = A.per_v[p];
            const int a = u + 1, b = v - 1;
            const int64_t s = A.bytes[i];
            const int ap = A.geo_a[X * A.geo_stride + p], bp = A.geo_b[X * A.geo_stride + p];
            const int64_t t = A.geo_t[X * A.geo_stride + p];
            const int64_t t_r = A.start[a], t_end = A.start[v];
            // pressure: each block updates the slots it owns
            for (int tl = ap / kSlotTile; tl <= bp / kSlotTile; ++tl) {
                if (tl % G != c) continue;
                own_dirty = true;
                const int64_t k0 = (int64_t)tl * kSlotTile;
                for (int64_t k = k0 + threadIdx.x; k < k0 + kSlotTile && k < K; k += kPlanThreads)
                    if (k >= ap && k <= bp) A.P[k] -= s;
            }
            if (X == G10_DEST_HOST && A.host_capacity != 0) {
                for (int tl = a / kSlotTile; tl <= b / kSlotTile; ++tl) {
                    if (tl % G != c) continue;
                    const int64_t k0 = (int64_t)tl * kSlotTile;
                    for (int64_t k = k0 + threadIdx.x; k < k0 + kSlotTile && k < K; k += kPlanThreads)
                        if (k >= a && k <= b) A.hocc[k] += s;
                }
            }
            if (c == 0) {
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
            n_mig += 1;
            if (X == G10_DEST_SSD) bytes_ssd += s; else bytes_host += s;
        }
        if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }
    }

    // ---- epilogue: lowest slot holding the final peak, then the summary
    if (status == -2) {
        if (c == 0 && threadIdx.x == 0) { raise_status(A.status, G10_DEV_TIMEOUT); }
        if (c == 0 && threadIdx.x == 0) {
            A.summary[0] = n_mig; A.summary[1] = rounds; A.summary[2] = -1; A.summary[3] = 0; A.summary[4] = -1;
            A.summary[5] = bytes_ssd; A.summary[6] = bytes_host;
        }
        return;
    }
    const long long peak = s_peak;
    {
        int key = 0;
        for (int tl = c; tl < n_slot_tiles; tl += G) {
            const int64_t k0 = (int64_t)tl * kSlotTile;
            for (int64_t k = k0 + threadIdx.x; k < k0 + kSlotTile && k < K; k += kPlanThreads)
                if (A.P[k] == peak) { const int kk = (int)(K - k); if (kk > key) key = kk; }
        }
        if (key > 0) atomicMax(A.peak_key, key);
    }
    if (!grid_barrier(A.bar, G, gen)) { if (c == 0 && threadIdx.x == 0) raise_status(A.status, G10_DEV_TIMEOUT); return; }
    if (c == 0 && threadIdx.x == 0) {
        const int key = *((volatile int *)A.peak_key);
        A.summary[0] = n_mig; A.summary[1] = rounds; A.summary[2] = status;
        A.summary[3] = K > 0 ? peak : 0;
        A.summary[4] = key > 0 ? K - key : -1;
        A.summary[5] = bytes_ssd; A.summary[6] = bytes_host;
    }
}

// copies the device status word into summary[7] / counts[2] / *status once everything before it ran
__global__ void k_publish_status(const ull *status, int64_t *dst) { *dst = (int64_t)*status; }

cudaError_t launch_publish_status(const Workspace &w, int64_t *dst, cudaStream_t s)
{
    k_publish_status<<<1, 1, 0, s>>>(w.status, dst);
    return cudaGetLastError();
}

int plan_loop_max_blocks()
{
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_plan_loop, kPlanThreads, 0) != cudaSuccess) return 0;
    if (per_sm < 1) return 0;
    int g = sms;      // one block per SM
    return g > kMaxPlanBlocks ? kMaxPlanBlocks : g;
}

cudaError_t launch_plan_loop(const DeviceTrace &t, const Workspace &w, const PlanParams &p, cudaStream_t s)
{
    PlanArgs A;
    A.K = t.K;
    A.Pn_dev = w.counts + 1;
    A.geo_stride = t.E > 0 ? t.E : 1;
    A.start = w.start; A.dur = t.kernel_ns; A.bytes = t.tensor_bytes;
    A.per_t = w.period_tensor; A.per_u = w.period_prev_use; A.per_v = w.period_next_use;
    A.geo_t = w.geo_t; A.geo_a = w.geo_a; A.geo_b = w.geo_b;
    A.P = p.final_pressure; A.busy = w.busy; A.hocc = w.hocc; A.dead = w.dead;
    A.fits_always = p.gpu_capacity_bytes >= ((uint64_t)1 << 63) ? 1 : 0;
    A.cap = A.fits_always ? INT64_MAX : (int64_t)p.gpu_capacity_bytes;
    A.host_capacity = p.host_capacity_bytes;
    A.max_iterations = p.max_iterations;
    A.out = p.migrations; A.out_cap = p.migrations_cap; A.summary = p.summary;
    A.proposals = w.proposals; A.peak_part = w.peak_part; A.peak_key = w.peak_key;
    A.bar = (GridBarrier *)w.barrier; A.status = w.status;
    int G = plan_loop_max_blocks();
    if (G < 1) return cudaErrorLaunchFailure;
    // no point in more blocks than there is work: periods per warp, slot tiles per block
    void *args[] = {&A};
    return cudaLaunchCooperativeKernel((const void *)k_plan_loop, dim3(G), dim3(kPlanThreads), args, 0, s);
}

}  // namespace g10

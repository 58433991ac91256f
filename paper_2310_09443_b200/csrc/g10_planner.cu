// Algorithm 1 (smart tensor eviction) as printed: one persistent cooperative kernel in which every
// iteration rescores all live inactive periods in parallel, reduces the best benefit/cost ratio across the
// grid, commits it and tests the peak -- two grid barriers per iteration, no host round trip.  Selected by
// G10_FLAG_RESCORE_ALL; the default planner (g10_planner_lazy.cu) gives the same plan with far less work.
#include "g10_planner.cuh"

namespace g10 {

// kCyclic: steady-state planning (period and geometry arrays hold slots unrolled over two iterations, A.start is the
// unrolled clock; see phys_slot) for traces too large for the single-block planner, which runs first: when it has
// produced the plan (`done`), this grid returns at once.
template <bool kCyclic>
__global__ void __launch_bounds__(kPlanThreads, 1) k_plan_loop(PlanArgs A, const unsigned *done)
{
    if (kCyclic && *done) return;          // (same answer in every thread of the grid: written by an earlier launch)
    if (kCyclic && blockIdx.x == 0 && threadIdx.x == 0) A.summary[7] = 0;      // (the single-block planner left "does not fit" there)
    __shared__ Cand s_cand[kPlanWarps + 1];
    __shared__ long long s_max[kPlanWarps + 1];
    const int G = gridDim.x, c = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t Pn = *A.Pn_dev < A.geo_stride ? *A.Pn_dev : A.geo_stride;
    const int64_t limit = (A.max_iterations <= 0 || A.max_iterations > Pn) ? Pn : A.max_iterations;
    unsigned gen = 0;
    int64_t n_mig = 0, rounds = 0, bytes_ssd = 0, bytes_host = 0;
    int status = -1;
    bool own_dirty = true;
    long long peak = 0;

    for (int64_t it = 0;; ++it) {
        if (own_dirty) {
            const long long m = own_slots_max(A, c, G, s_max);
            if (threadIdx.x == 0) A.peak_part[c] = m;
            own_dirty = false;
        }
        // ---- score: one warp per live period
        Cand best;
        best.ben = 0; best.cost = 1; best.idx = -1; best.dest = -1;
        for (int64_t p = (int64_t)c * kPlanWarps + warp; p < Pn; p += (int64_t)G * kPlanWarps) {
            if (A.dead[p]) continue;
            Cand cd;
            if (!score_period<kCyclic>(A, p, lane, &cd)) {
                if (lane == 0) A.dead[p] = 1;       // channels only fill up: never admissible again
                continue;
            }
            if (lane == 0 && cd.ben > 0 && cand_beats(cd, best)) best = cd;
        }
        best = block_best(best, s_cand);
        if (threadIdx.x == 0) {
            Proposal pr;
            pr.ben_lo = (ull)best.ben; pr.ben_hi = (ull)(best.ben >> 64); pr.cost = best.cost; pr.idx = best.idx; pr.dest = best.dest;
            A.proposals[c] = pr;
        }
        if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }

        // ---- reduce peak and proposals (every block, redundantly and identically)
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
        peak = block_max_i64(m, s_max);
        const Cand win = block_best(w, s_cand);
        if (A.fits_always || peak <= A.cap) { status = n_mig == 0 ? G10_ALREADY_FITS : G10_FIT; break; }
        if (it >= limit) { status = limit < Pn ? G10_ITERATION_LIMIT : G10_EXHAUSTED; break; }
        rounds += 1;
        if (win.idx < 0) { status = G10_EXHAUSTED; break; }

        int64_t sz = 0;
        if (commit_winner<kCyclic>(A, win.idx, win.dest, it, n_mig, c, G, &sz)) own_dirty = true;
        n_mig += 1;
        if (win.dest == G10_DEST_SSD) bytes_ssd += sz; else bytes_host += sz;
        if (!grid_barrier(A.bar, G, gen)) { status = -2; break; }
    }
    plan_epilogue(A, c, G, gen, status, peak, n_mig, rounds, bytes_ssd, bytes_host);
}

// copies the device status word into summary[7] / counts[2] / *status once everything before it ran
__global__ void k_publish_status(const ull *status, int64_t *dst) { *dst = (int64_t)*status; }

cudaError_t launch_publish_status(const Workspace &w, int64_t *dst, cudaStream_t s)
{
    k_publish_status<<<1, 1, 0, s>>>(w.status, dst); count_launch();
    return cudaGetLastError();
}

void fill_plan_args(const DeviceTrace &t, const Workspace &w, const PlanParams &p, PlanArgs &A)
{
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
}

static int blocks_for(const void *kernel)
{
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kPlanThreads, 0) != cudaSuccess) return 0;
    if (per_sm < 1) return 0;
    return sms > kMaxPlanBlocks ? kMaxPlanBlocks : sms;      // one block per SM
}

cudaError_t launch_plan_lazy(const PlanArgs &A, const Workspace &w, int G, cudaStream_t s);
int plan_lazy_blocks();
cudaError_t launch_plan_small(const PlanArgs &A, const Workspace &w, int G, int cand_cap, size_t smem, cudaStream_t s);
int plan_small_blocks();
bool plan_small_fits(int64_t K, int64_t E, int G, int *cand_cap_out, size_t *smem_out);
bool plan_one_possible(int64_t K, int64_t E, bool host_cap);
cudaError_t launch_plan_one(const PlanArgs &A, const Workspace &w, cudaStream_t s);

bool plan_keeps_state_on_chip(int64_t K, int64_t E, uint32_t flags)
{
    if ((flags & (G10_FLAG_RESCORE_ALL | G10_FLAG_GLOBAL_STATE)) || K > kSmallMaxSlots) return false;
    int Gs = plan_small_blocks();
    if (Gs > kSmallMaxBlocks) Gs = kSmallMaxBlocks;
    int cand_cap = 0;
    size_t smem = 0;
    return Gs >= 1 && plan_small_fits(K, E, Gs, &cand_cap, &smem);
}

cudaError_t launch_plan_batch(const PlanArgs &A, const Workspace &w, int V, const BatchArgs &B, int64_t *stability, cudaStream_t s);

cudaError_t launch_plan_variants(const DeviceTrace &t, const Workspace &w, const PlanParams &p, int V, int64_t *stability, cudaStream_t s)
{
    PlanArgs A;
    fill_plan_args(t, w, p, A);
    BatchArgs B;
    B.variants = w.batch_variants; B.P0 = w.pressure; B.P_out = p.final_pressure;
    return launch_plan_batch(A, w, V, B, stability, s);
}

cudaError_t launch_plan_one_cyclic(const PlanArgs &A, const Workspace &w, cudaStream_t s);

cudaError_t launch_plan_cyclic(const DeviceTrace &t, const Workspace &w, const PlanParams &p, cudaStream_t s)
{
    PlanArgs A;
    fill_plan_args(t, w, p, A);
    A.start = w.start2;
    // one block plans when everything fits its shared memory (decided on the device); the multi-block planner queued
    // behind it does the work otherwise
    cudaError_t e = launch_plan_one_cyclic(A, w, s);
    if (e != cudaSuccess) return e;
    const int G = blocks_for((const void *)k_plan_loop<true>);
    if (G < 1) return cudaErrorLaunchFailure;
    const unsigned *done = w.one_done;
    void *args[] = {&A, &done};
    return cudaLaunchCooperativeKernel((const void *)k_plan_loop<true>, dim3(G), dim3(kPlanThreads), args, 0, s);
}

// ORs the call's status word into *dst (which the planner may already have written)
__global__ void k_publish_status_or(const ull *status, int64_t *dst) { *dst |= (int64_t)*status; }

cudaError_t launch_publish_status_or(const Workspace &w, int64_t *dst, cudaStream_t s)
{
    k_publish_status_or<<<1, 1, 0, s>>>(w.status, dst); count_launch();
    return cudaGetLastError();
}

cudaError_t launch_plan_loop(const DeviceTrace &t, const Workspace &w, const PlanParams &p, cudaStream_t s)
{
    PlanArgs A;
    fill_plan_args(t, w, p, A);
    if (p.flags & G10_FLAG_RESCORE_ALL) {
        const int G = blocks_for((const void *)k_plan_loop<false>);
        if (G < 1) return cudaErrorLaunchFailure;
        const unsigned *done = w.one_done;
        void *args[] = {&A, &done};
        return cudaLaunchCooperativeKernel((const void *)k_plan_loop<false>, dim3(G), dim3(kPlanThreads), args, 0, s);
    }
    if (plan_keeps_state_on_chip(t.K, t.E, p.flags)) {
        int Gs = plan_small_blocks();
        if (Gs > kSmallMaxBlocks) Gs = kSmallMaxBlocks;
        int cand_cap = 0;
        size_t smem = 0;
        if (Gs >= 1 && plan_small_fits(t.K, t.E, Gs, &cand_cap, &smem)) {
            // one block does the whole loop when the device finds that everything fits its shared memory; the
            // multi-block planner queued behind it returns at once in that case and does the work otherwise
            if (!(p.flags & G10_FLAG_MULTI_BLOCK) && plan_one_possible(t.K, t.E, p.host_capacity_bytes != 0)) {
                const cudaError_t e = launch_plan_one(A, w, s);
                if (e != cudaSuccess) return e;
            }
            return launch_plan_small(A, w, Gs, cand_cap, smem, s);
        }
    }
    const int G = plan_lazy_blocks();
    if (G < 1) return cudaErrorLaunchFailure;
    return launch_plan_lazy(A, w, G, s);
}

}  // namespace g10

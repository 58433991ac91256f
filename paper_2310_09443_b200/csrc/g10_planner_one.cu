// Algorithm 1 for traces small enough for ONE block to hold everything in shared memory: pressure, slot clock,
// channel bookings (and host occupancy), and per period its cached score, exact benefit, size, transfer time,
// slot ranges and state.  With the whole state on one SM an iteration needs no exchange between SMs; what is
// left is the lazy evaluation itself, arranged so that few warps have to issue instructions at any time:
//   - the rounded scores (positive doubles, compared as 64-bit integers) sit under a two-level maximum: one
//     entry per group of 32 periods, refreshed only when a score of the group changed, and a scan of the group
//     entries by one warp;
//   - the top entry is the winner if its score is FRESH (exact for the current state); a STALE score is an
//     upper bound (pressure only falls), so a stale top is rescored by the whole block and the search repeats;
//   - scores within 1e-10 of a fresh top are settled exactly (128-bit cross products, lowest index on ties),
//     after any stale one among them has been rescored;
//   - the winner is applied: pressure range, channel bookings, and every live period is reclassified against
//     the winner's slot ranges (STALE if the absent ranges meet, DIRTY if transfer windows on the same device
//     meet); DIRTY periods have their destination re-examined before the next search, one warp per period,
//     and are rescored only if the destination changed.
// The kernel decides by itself, from the number of periods found on the device, whether the trace fits; if it
// does not, it leaves `done` at zero and the multi-block planner launched right behind it does the work.
//
// Batch mode (kBatch): one block per VARIANT of the same trace -- its own kernel durations, bandwidths and
// capacities -- each running the whole loop independently of the others (re-planning under profiling error,
// other SSD bandwidths or host capacities).  A variant's block builds its own slot clock (block-wide scan of its
// durations) and derives the geometry of a period when it needs it, from that clock in shared memory.
#include "g10_planner.cuh"

namespace g10 {

#ifndef G10_ONE_THREADS
#define G10_ONE_THREADS 512
#endif
constexpr int kOneThreads = G10_ONE_THREADS;
constexpr int kOneWarps = kOneThreads / 32;
constexpr int kOneMaxFin = 64;                // (at least kOneWarps: the list doubles as scratch at the end)
constexpr int kOneDirtyCap = 256;            // DIRTY periods of one commit that are listed (more: full sweep)
enum { kFreshO = 1 << 2, kStaleO = 2 << 2, kStateMaskO = 3 << 2, kDirtyO = 0x10 };

struct OneArgs {
    unsigned *done;          // set to 1 when this kernel produced the plan
    int smem_bytes;          // dynamic shared memory the launch provides
};

struct __align__(8) OneRanges { unsigned short a, b, ap, bp; };   // inactive slots [a, b], absent [ap, bp] (current destination)

// A DIRTY period with the geometry of both destinations, fetched from global memory by the thread that found it
struct __align__(16) OneDirty {
    int li;
    int ap[2], bp[2];
    int pad[3];
    int64_t t[2];
};

// Kc: number of physical slots when the slot indices are unrolled (cyclic mode), else 0
__device__ __forceinline__ int phys_slot(int k, int Kc) { return Kc && k >= Kc ? k - Kc : k; }

// Do the unrolled slot ranges [a1, b1] and [a2, b2] share a slot?  On the cycle also when one of them, taken one
// iteration earlier or later, meets the other.
__device__ __forceinline__ bool ranges_meet(int a1, int b1, int a2, int b2, int Kc)
{
    if (a1 <= b2 && a2 <= b1) return true;
    if (!Kc) return false;
    return (a1 <= b2 + Kc && a2 + Kc <= b1) || (a1 <= b2 - Kc && a2 - Kc <= b1);
}

__device__ __forceinline__ bool window_free_one(const int64_t *sStart, const int64_t *busy, int64_t w0, int64_t w1, int k0, int k1, int lane,
                                                int Kc)
{
    bool ok = true;
#pragma unroll 1
    for (int k = k0 + lane; k <= k1; k += 32) {
        const int64_t s0 = sStart[k], s1 = sStart[k + 1];
        const int64_t lo = w0 > s0 ? w0 : s0, hi = w1 < s1 ? w1 : s1;
        const int64_t ov = hi > lo ? hi - lo : 0;
        if (busy[phys_slot(k, Kc)] + ov > s1 - s0) ok = false;
    }
    return __all_sync(0xffffffffu, ok);
}

// window_conflict on the cycle: the other window may meet the booking as it is, or one iteration earlier / later
// (T = length of the iteration).  Only slots of the booking's own range are read.
__device__ __forceinline__ bool window_conflict_cyc(const int64_t *sStart, const int64_t *busy, int wk0, int wk1, int64_t q0, int64_t q1,
                                                    int qk0, int qk1, int Kc, int64_t T)
{
    if (window_conflict<true, false>(sStart, busy, wk0, wk1, 0, 0, q0, q1, qk0, qk1, Kc)) return true;
    if (!Kc) return false;
    return window_conflict<true, false>(sStart, busy, wk0, wk1, 0, 0, q0 + T, q1 + T, qk0 + Kc, qk1 + Kc, Kc) ||
           window_conflict<true, false>(sStart, busy, wk0, wk1, 0, 0, q0 - T, q1 - T, qk0 - Kc, qk1 - Kc, Kc);
}


// The same for an unrolled slot range [a, b] (at most Kc slots long when Kc != 0): its one or two physical pieces.
__device__ __forceinline__ u128 benefit_range_warp(const int64_t *sP, const int64_t *sStart, const int64_t *tmin, const int64_t *tmax,
                                                   int64_t cap, int64_t s, int a, int b, int Kc, int lane)
{
    if (!Kc || b < Kc) return benefit_tiles_warp(sP, sStart, tmin, tmax, cap, s, a, b, lane);
    if (a >= Kc) return benefit_tiles_warp(sP, sStart, tmin, tmax, cap, s, a - Kc, b - Kc, lane);
    return benefit_tiles_warp(sP, sStart, tmin, tmax, cap, s, a, Kc - 1, lane) + benefit_tiles_warp(sP, sStart, tmin, tmax, cap, s, 0, b - Kc, lane);
}

__host__ __device__ inline size_t one_smem_need(int64_t K, int64_t Pn, bool host_cap, bool cyclic = false)
{
    const int64_t groups = (Pn + 31) / 32;
    return (size_t)(2 * K + 1) * 8 + (cyclic ? (size_t)K * 8 : 0) + (size_t)4 * K * 8 + (host_cap ? (size_t)K * 8 : 0) + (size_t)groups * 32 * 8 + (size_t)Pn * 41 +
           (size_t)groups * 13 + (size_t)((K + 31) / 32) * 16 + 128;
}

// Warp-wide maximum of 64-bit keys with the lowest index among equal keys; same result in every lane.
__device__ __forceinline__ void warp_argmax_u64(ull k, int idx, ull *mk, int *mi)
{
    const unsigned hi = (unsigned)(k >> 32);
    const unsigned mh = __reduce_max_sync(0xffffffffu, hi);
    const unsigned lo = hi == mh ? (unsigned)k : 0u;
    const unsigned ml = __reduce_max_sync(0xffffffffu, lo);
    const bool top = hi == mh && (unsigned)k == ml;
    *mk = ((ull)mh << 32) | ml;
    *mi = (int)__reduce_min_sync(0xffffffffu, top ? (unsigned)idx : 0x7fffffffu);
}


template <bool kBatch, bool kCyclic>
__global__ void __launch_bounds__(kOneThreads, 1) k_plan_one(PlanArgs A, OneArgs O, BatchArgs B)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_fin[kOneMaxFin];
    __shared__ OneDirty s_dirty[kOneDirtyCap];
    __shared__ int s_n_over, s_ndirty, s_nlist, s_nfin, s_force, s_win, s_top, s_flagged;
    __shared__ ull s_topkey;
    __shared__ long long s_pk[kOneWarps];
    __shared__ int s_ps[kOneWarps];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = (int)A.K;
    const int64_t Pn64 = *A.Pn_dev < A.geo_stride ? *A.Pn_dev : A.geo_stride;
    const int64_t *P_src = A.P;
    uint64_t bw[2] = {0, 0};
    const int64_t *var_dur = nullptr;
    if (kBatch) {
        const BatchVariant var = B.variants[blockIdx.x];
        A.fits_always = var.cap >= ((uint64_t)1 << 63) ? 1 : 0;
        A.cap = A.fits_always ? INT64_MAX : (int64_t)var.cap;
        A.host_capacity = var.host_capacity;
        A.out += (size_t)blockIdx.x * A.out_cap;
        A.summary += (size_t)blockIdx.x * 8;
        P_src = B.P0;
        A.P = B.P_out + (size_t)blockIdx.x * K;
        bw[G10_DEST_SSD] = var.ssd_bw; bw[G10_DEST_HOST] = var.host_bw;
        var_dur = var.kernel_ns;
    }
    const bool host_cap = A.host_capacity != 0;
    unsigned dev_bits = 0;                              // device status bits of this block's plan
    const int Kc = kCyclic ? (int)A.K : 0;             // physical slots when the indices are unrolled
    if (A.K > (kCyclic ? 32000 : 65000) || Pn64 > 0x7fffffff || one_smem_need(A.K, Pn64, host_cap, kCyclic) > (size_t)O.smem_bytes) {
        if ((kBatch || kCyclic) && threadIdx.x == 0) {
            for (int j = 0; j < 7; ++j) A.summary[j] = j == 2 || j == 4 ? -1 : 0;
            A.summary[7] = G10_DEV_BATCH_UNFIT;
        }
        return;
    }
    const int Pn = (int)Pn64;
    const int G1 = (Pn + 31) / 32;
    const int64_t limit = (A.max_iterations <= 0 || A.max_iterations > Pn64) ? Pn64 : A.max_iterations;

    int64_t *sP = (int64_t *)smem_raw;
    int64_t *sStart = sP + K;
    int64_t *sBusy = sStart + (kCyclic ? 2 * K : K) + 1; // [4][K]  (the clock has 2K + 1 entries in cyclic mode)
    int64_t *sHocc = sBusy + (size_t)4 * K;             // [K] if host_cap
    const int NT = (K + kTileO - 1) / kTileO;
    int64_t *tmin = sHocc + (host_cap ? K : 0);         // [NT] smallest pressure of each tile of 32 slots
    int64_t *tmax = tmin + NT;                          // [NT] largest
    ull *ckey = (ull *)(tmax + NT);                     // [G1 * 32] bits of the rounded score (0 = none)
    ull *gkey = ckey + (size_t)G1 * 32;                 // [G1] maximum of each group
    int64_t *cbytes = (int64_t *)(gkey + G1);
    int64_t *ct = cbytes + Pn;                          // transfer time of the current destination
    ull *cben_lo = (ull *)(ct + Pn);
    ull *cben_hi = cben_lo + Pn;
    OneRanges *crng = (OneRanges *)(cben_hi + Pn);
    int *garg = (int *)(crng + Pn);                     // [G1] period holding the group's maximum
    unsigned char *cstate = (unsigned char *)(garg + G1);   // 0 = erased, else (destination + 1) | state | dirty flag
    unsigned char *gflag = cstate + Pn;                 // [G1] a score of the group changed

    if (tid == 0) { s_n_over = 0; s_ndirty = Pn; s_nlist = kOneDirtyCap + 1; s_nfin = 0; s_force = 0x7fffffff; s_win = -1; s_flagged = 1; }
    __syncthreads();
    {
        int over = 0;
#pragma unroll 1
        for (int k = tid; k < K; k += kOneThreads) {
            const int64_t pv = P_src[k];
            sP[k] = pv;
            if (pv > A.cap) ++over;
        }
        if (!kBatch) {
#pragma unroll 1
            for (int k = tid; k <= (kCyclic ? 2 * K : K); k += kOneThreads) sStart[k] = A.start[k];
        } else {
            // slot clock of this variant: exclusive scan of its durations (each thread a run of consecutive kernels);
            // a duration outside [1, 2^44) counts as 1 and raises the status bit, as in the trace-level pass
            const int chunk = (K + kOneThreads - 1) / kOneThreads;
            const int k0 = tid * chunk < K ? tid * chunk : K, k1 = k0 + chunk < K ? k0 + chunk : K;
            long long sum = 0;
#pragma unroll 1
            for (int k = k0; k < k1; ++k) {
                long long d = var_dur[k];
                if (d < 1 || d >= ((long long)1 << 44)) { d = 1; dev_bits |= G10_DEV_BAD_DURATION; }
                sum += d;
            }
            const long long incl = warp_inclusive_scan_i64(sum, lane);
            if (lane == 31) s_pk[warp] = incl;
            __syncthreads();
            long long run = incl - sum;
#pragma unroll 1
            for (int w = 0; w < warp; ++w) run += s_pk[w];
#pragma unroll 1
            for (int k = k0; k < k1; ++k) {
                long long d = var_dur[k];
                if (d < 1 || d >= ((long long)1 << 44)) d = 1;
                sStart[k] = run;
                run += d;
            }
            if (k1 == K) sStart[K] = run;              // every thread at or past the end holds the total
        }
#pragma unroll 1
        for (int k = tid; k < (host_cap ? 5 : 4) * K; k += kOneThreads) sBusy[k] = 0;
#pragma unroll 1
        for (int li = tid; li < G1 * 32; li += kOneThreads) ckey[li] = 0;
#pragma unroll 1
        for (int g = tid; g < G1; g += kOneThreads) { gkey[g] = 0; garg[g] = g * 32; gflag[g] = 0; }
#pragma unroll 1
        for (int li = tid; li < Pn; li += kOneThreads) {
            OneRanges r;
            r.a = (unsigned short)(A.per_u[li] + 1); r.b = (unsigned short)(A.per_v[li] - 1); r.ap = 0; r.bp = 0;
            crng[li] = r;
            cbytes[li] = A.bytes[A.per_t[li]];
            ct[li] = 0; cben_lo[li] = 0; cben_hi[li] = 0;
            cstate[li] = (unsigned char)kDirtyO;
        }
        over = __reduce_add_sync(0xffffffffu, over);
        if (lane == 0 && over) atomicAdd(&s_n_over, over);
    }
    __syncthreads();
    for (int t = warp; t < NT; t += kOneWarps) tile_refresh_warp(sP, K, t, tmin, tmax, lane);
    __syncthreads();

    int64_t n_mig = 0, rounds = 0, bytes_ssd = 0, bytes_host = 0;
    int status = -1;
#pragma unroll 1
    for (int64_t it = 0;; ++it) {
        if (A.fits_always || s_n_over == 0) { status = n_mig == 0 ? G10_ALREADY_FITS : G10_FIT; break; }
        if (it >= limit) { status = limit < Pn64 ? G10_ITERATION_LIMIT : G10_EXHAUSTED; break; }
        rounds += 1;
        // ---------------- 1. DIRTY periods: destination (SSD first, then host), one warp per period; a new score
        // only if the destination changed
        if (s_ndirty > 0) {
            const int nlist = s_nlist;
            const bool listed = nlist <= kOneDirtyCap;            // else: sweep all periods for the flag
            // listed periods go round the warps one by one; a sweep hands each warp 32 consecutive periods at a time
            const int n_items = listed ? nlist : (Pn + 31) / 32 * 32;
            const int step = listed ? kOneWarps : kOneThreads;
#pragma unroll 1
            for (int base = listed ? warp : warp * 32; base < n_items; base += step) {
                unsigned m = 1u;
                if (!listed) { const int mine = base + lane; m = __ballot_sync(0xffffffffu, mine < Pn && (cstate[mine] & kDirtyO) != 0); }
#pragma unroll 1
                while (m) {
                    const int j = base + __ffs(m) - 1;
                    m &= m - 1;
                    const int li = listed ? s_dirty[j].li : j;
                    const unsigned char st = cstate[li];
                    const OneRanges r = crng[li];
                    const int a = r.a, b = r.b;
                    const int64_t s = cbytes[li];
                    const int64_t t_r = sStart[a], t_end = sStart[b + 1];
                    int d = -1, ap = 0, bp = -1;
                    int64_t t = 0;
#pragma unroll 1
                    for (int X = 0; X < 2 && d < 0; ++X) {
                        if (listed) { ap = s_dirty[j].ap[X]; bp = s_dirty[j].bp[X]; t = s_dirty[j].t[X]; }
                        else if (kBatch) period_geometry(sStart, a - 1, b + 1, s, bw[X], &t, &ap, &bp);
                        else {
                            ap = __ldg(&A.geo_a[X * A.geo_stride + li]);
                            bp = __ldg(&A.geo_b[X * A.geo_stride + li]);
                            t = __ldg(&A.geo_t[X * A.geo_stride + li]);
                        }
                        if (ap < 0) continue;
                        if (!window_free_one(sStart, sBusy + (size_t)(2 * X) * K, t_r, t_r + t, a, ap - 1, lane, Kc)) continue;
                        if (!window_free_one(sStart, sBusy + (size_t)(2 * X + 1) * K, t_end - t, t_end, bp + 1, b, lane, Kc)) continue;
                        if (X == G10_DEST_HOST && host_cap) {
                            bool ok = true;
#pragma unroll 1
                            for (int k = a + lane; k <= b; k += 32)
                                if ((uint64_t)sHocc[phys_slot(k, Kc)] + (uint64_t)s > A.host_capacity) ok = false;
                            if (!__all_sync(0xffffffffu, ok)) continue;
                        }
                        d = X;
                    }
                    if (d < 0) {                                  // channels only fill up: gone for good
                        if (lane == 0) { cstate[li] = 0; ckey[li] = 0; gflag[li >> 5] = 1; s_flagged = 1; }
                        continue;
                    }
                    if (d == (int)(st & 3) - 1) {                 // same destination: score and state stand
                        if (lane == 0) cstate[li] = (unsigned char)(st & ~kDirtyO);
                        continue;
                    }
                    const u128 acc = warp_sum_u128(benefit_range_warp(sP, sStart, tmin, tmax, A.cap, s, ap, bp, Kc, lane));
                    if (lane == 0) {
                        Cand cd;
                        cd.ben = acc; cd.cost = 2ull * (ull)t; cd.idx = 0; cd.dest = d;
                        OneRanges w = r;
                        w.ap = (unsigned short)ap; w.bp = (unsigned short)bp;
                        crng[li] = w; ct[li] = t;
                        cben_lo[li] = (ull)acc; cben_hi[li] = (ull)(acc >> 64);
                        ckey[li] = acc == 0 ? 0ull : (ull)__double_as_longlong(cand_key(cd));
                        cstate[li] = (unsigned char)((d + 1) | kFreshO);
                        gflag[li >> 5] = 1; s_flagged = 1;
                    }
                }
            }
            __syncthreads();
            if (tid == 0) { s_ndirty = 0; s_nlist = 0; }
        }
        // ---------------- 2. search: warp 0 refreshes the group maxima that changed, takes the top and, while the top is
        // STALE, rescores it (from the pressure tiles) and looks again; the other warps wait at the barrier
        int win = -1;
        bool exhausted = false;
        // rescoring of one period by warp 0 (uniform arguments)
        auto rescore_warp0 = [&](int target) {
            const OneRanges r = crng[target];
            const u128 tot = warp_sum_u128(benefit_range_warp(sP, sStart, tmin, tmax, A.cap, cbytes[target], r.ap, r.bp, Kc, lane));
            if (lane == 0) {
                Cand cd;
                cd.ben = tot; cd.cost = 2ull * (ull)ct[target]; cd.idx = 0; cd.dest = 0;
                cben_lo[target] = (ull)tot; cben_hi[target] = (ull)(tot >> 64);
                ckey[target] = tot == 0 ? 0ull : (ull)__double_as_longlong(cand_key(cd));
                cstate[target] = (unsigned char)((cstate[target] & 3) | kFreshO);
                gflag[target >> 5] = 1; s_flagged = 1;
            }
            __syncwarp();
        };
#pragma unroll 1
        for (;;) {
            if (warp == 0) {
#pragma unroll 1
                for (;;) {
                    if (s_flagged) {
                        __syncwarp();
                        if (lane == 0) s_flagged = 0;
#pragma unroll 1
                        for (int g0 = 0; g0 < G1; g0 += 32) {
                            unsigned m = __ballot_sync(0xffffffffu, g0 + lane < G1 && gflag[g0 + lane] != 0);
#pragma unroll 1
                            while (m) {
                                const int g = g0 + __ffs(m) - 1;
                                m &= m - 1;
                                ull mk; int mi;
                                warp_argmax_u64(ckey[g * 32 + lane], g * 32 + lane, &mk, &mi);
                                if (lane == 0) { gkey[g] = mk; garg[g] = mi; gflag[g] = 0; }
                            }
                        }
                    }
                    __syncwarp();
                    ull bk = 0; int bi = 0x7fffffff;
#pragma unroll 4
                    for (int g = lane; g < G1; g += 32) {
                        const ull k = gkey[g];
                        if (k > bk) { bk = k; bi = garg[g]; }         // g ascending: the lowest index stays on ties
                    }
                    ull mk; int mi;
                    warp_argmax_u64(bk, bi, &mk, &mi);
                    if (mk == 0 || (cstate[mi] & kStateMaskO) != kStaleO) {
                        if (lane == 0) { s_topkey = mk; s_top = mi; }
                        break;
                    }
                    rescore_warp0(mi);
                }
            }
            __syncthreads();
            const ull topkey = s_topkey;
            const int top = s_top;
            if (topkey == 0) { exhausted = true; break; }
            // a fresh top: can anything else within 1e-10 of it beat it exactly?  (A stale entry competes with its
            // bound: if even the bound loses, the period cannot win this iteration.)
            const double thr = __longlong_as_double((long long)topkey) * (1.0 - 1e-10);
            const ull thr_bits = (ull)__double_as_longlong(thr);
            bool other = false;
#pragma unroll 4
            for (int g = warp; g < G1; g += kOneWarps) {
                if (gkey[g] < thr_bits) continue;
                const int li = g * 32 + lane;
                if (ckey[li] < thr_bits || li == top) continue;
                Cand x, y;
                x.ben = ((u128)cben_hi[li] << 64) | cben_lo[li]; x.cost = 2ull * (ull)ct[li]; x.idx = li; x.dest = 0;
                y.ben = ((u128)cben_hi[top] << 64) | cben_lo[top]; y.cost = 2ull * (ull)ct[top]; y.idx = top; y.dest = 0;
                if (!cand_beats(x, y)) continue;
                other = true;
                if ((cstate[li] & kStateMaskO) == kStaleO) atomicMin(&s_force, li);
                else { const int pos = atomicAdd(&s_nfin, 1); if (pos < kOneMaxFin) s_fin[pos] = li; }
            }
            if (!__syncthreads_or(other)) { win = top; break; }
            const int forced = s_force;
            if (forced != 0x7fffffff) {
                // a stale period whose bound beats the top exactly: rescore it, then search again
                __syncthreads();                   // everyone has read s_force
                if (warp == 0) {
                    rescore_warp0(forced);
                    if (lane == 0) { s_force = 0x7fffffff; s_nfin = 0; }
                    __syncwarp();
                }
                continue;
            }
            if (tid == 0) {
                Cand w;
                w.ben = ((u128)cben_hi[top] << 64) | cben_lo[top]; w.cost = 2ull * (ull)ct[top]; w.idx = top; w.dest = 0;
                const int n = s_nfin;
                if (n <= kOneMaxFin) {
                    for (int i = 0; i < n; ++i) {
                        const int li = s_fin[i];
                        Cand x;
                        x.ben = ((u128)cben_hi[li] << 64) | cben_lo[li]; x.cost = 2ull * (ull)ct[li]; x.idx = li; x.dest = 0;
                        if (cand_beats(x, w)) w = x;
                    }
                } else {
                    for (int li = 0; li < Pn; ++li) {      // very many close scores: plain sweep
                        if (ckey[li] < thr_bits || (cstate[li] & kStateMaskO) != kFreshO) continue;
                        Cand x;
                        x.ben = ((u128)cben_hi[li] << 64) | cben_lo[li]; x.cost = 2ull * (ull)ct[li]; x.idx = li; x.dest = 0;
                        if (cand_beats(x, w)) w = x;
                    }
                }
                s_win = w.idx; s_nfin = 0;
            }
            __syncthreads();
            win = s_win;
            break;
        }
        if (exhausted) { status = G10_EXHAUSTED; break; }
        // ---------------- 3. apply the winner
        {
            const OneRanges r = crng[win];
            const int X = (cstate[win] & 3) - 1;
            const int wa = r.a, wb = r.b, wap = r.ap, wbp = r.bp;
            const int64_t s = cbytes[win], t = ct[win];
            const int64_t t_r = sStart[wa], t_end = sStart[wb + 1];
            int win_tensor = 0;
            if (tid == 0) win_tensor = A.per_t[win];              // needed only for the record written at the end
            __syncthreads();                       // everyone has read the winner's entry before it is erased
            int fell = 0;
#pragma unroll 1
            for (int k = wap + tid; k <= wbp; k += kOneThreads) {
                const int kp = phys_slot(k, Kc);
                const int64_t before = sP[kp], after = before - s;
                sP[kp] = after;
                if (before > A.cap && after <= A.cap) ++fell;
            }
            if (fell) atomicSub(&s_n_over, fell);
            int64_t *bo = sBusy + (size_t)(2 * X) * K, *bi = sBusy + (size_t)(2 * X + 1) * K;
#pragma unroll 1
            for (int k = wa + tid; k <= wap - 1; k += kOneThreads) {
                const int64_t s0 = sStart[k], s1 = sStart[k + 1];
                const int64_t lo = t_r > s0 ? t_r : s0, hi = (t_r + t) < s1 ? (t_r + t) : s1;
                if (hi > lo) bo[phys_slot(k, Kc)] += hi - lo;
            }
#pragma unroll 1
            for (int k = wbp + 1 + tid; k <= wb; k += kOneThreads) {
                const int64_t s0 = sStart[k], s1 = sStart[k + 1];
                const int64_t lo = (t_end - t) > s0 ? (t_end - t) : s0, hi = t_end < s1 ? t_end : s1;
                if (hi > lo) bi[phys_slot(k, Kc)] += hi - lo;
            }
            if (X == G10_DEST_HOST && host_cap)
#pragma unroll 1
                for (int k = wa + tid; k <= wb; k += kOneThreads) sHocc[phys_slot(k, Kc)] += s;
            __syncthreads();                       // the bookings are in place for the conflict tests below
            // the pressure tiles the commit touched (one or two physical pieces of the absent range), one warp per tile
            {
                const int lo0 = phys_slot(wap, Kc), hi0 = (Kc && wap < Kc && wbp >= Kc) ? Kc - 1 : phys_slot(wbp, Kc);
                for (int t = lo0 / kTileO + warp; t <= hi0 / kTileO; t += kOneWarps) tile_refresh_warp(sP, K, t, tmin, tmax, lane);
                if (Kc && wap < Kc && wbp >= Kc)
                    for (int t = warp; t <= (wbp - Kc) / kTileO; t += kOneWarps) tile_refresh_warp(sP, K, t, tmin, tmax, lane);
            }
            int newly_dirty = 0;
#pragma unroll 2
            for (int li = tid; li < Pn; li += kOneThreads) {
                const unsigned char st = cstate[li];
                if (st == 0) continue;
                if (li == win) { cstate[li] = 0; ckey[li] = 0; gflag[li >> 5] = 1; s_flagged = 1; continue; }
                if (st & kDirtyO) continue;
                const int d = (st & 3) - 1;
                const OneRanges q = crng[li];
                if (!ranges_meet(q.a, q.b, wa, wb, Kc)) continue;
                unsigned char ns = st;
                if ((st & kStateMaskO) == kFreshO && ranges_meet(q.ap, q.bp, wap, wbp, Kc)) ns = (unsigned char)((st & 3) | kStaleO);
                if (d == X) {
                    // same device: is one of its transfer windows no longer free?  (host occupancy: looked at in full)
                    const bool meet_out = ranges_meet(q.a, (int)q.ap - 1, wa, wap - 1, Kc);
                    const bool meet_in = ranges_meet((int)q.bp + 1, q.b, wbp + 1, wb, Kc);
                    bool hit = false;
                    if (meet_out || meet_in) {
                        const int64_t tq = ct[li];
                        const int64_t q_r = sStart[q.a], q_end = sStart[(int)q.b + 1];
                        const int64_t T = kCyclic ? sStart[K] : 0;
                        hit = (meet_out && window_conflict_cyc(sStart, bo, wa, wap - 1, q_r, q_r + tq, q.a, (int)q.ap - 1, Kc, T)) ||
                              (meet_in && window_conflict_cyc(sStart, bi, wbp + 1, wb, q_end - tq, q_end, (int)q.bp + 1, q.b, Kc, T));
                    }
                    if (!hit && d == G10_DEST_HOST && host_cap) hit = true;
                    if (hit) {
                        ns |= kDirtyO; ++newly_dirty;
                        const int pos = atomicAdd(&s_nlist, 1);
                        if (pos < kOneDirtyCap) {                  // fetch both geometries now: the latency hides behind the rest
                            OneDirty e;
                            e.li = li;
#pragma unroll
                            for (int Y = 0; Y < 2; ++Y) {
                                if (kBatch) period_geometry(sStart, (int)q.a - 1, (int)q.b + 1, cbytes[li], bw[Y], &e.t[Y], &e.ap[Y], &e.bp[Y]);
                                else {
                                    e.ap[Y] = __ldg(&A.geo_a[Y * A.geo_stride + li]);
                                    e.bp[Y] = __ldg(&A.geo_b[Y * A.geo_stride + li]);
                                    e.t[Y] = __ldg(&A.geo_t[Y * A.geo_stride + li]);
                                }
                            }
                            e.pad[0] = e.pad[1] = e.pad[2] = 0;
                            s_dirty[pos] = e;
                        }
                    }
                }
                if (ns != st) cstate[li] = ns;
            }
            if (newly_dirty) atomicAdd(&s_ndirty, newly_dirty);
            if (tid == 0) {
                if (n_mig < A.out_cap) {
                    g10_migration m;
                    m.period = (int32_t)win; m.tensor = win_tensor; m.dest = X; m.absent_first = wap; m.absent_last = wbp;
                    m.iteration = (int32_t)it; m.evict_issue_ns = t_r; m.prefetch_issue_ns = t_end - t; m.transfer_ns = t;
                    A.out[n_mig] = m;
                } else dev_bits |= G10_DEV_PLAN_OVERFLOW;
            }
            n_mig += 1;
            if (X == G10_DEST_SSD) bytes_ssd += s; else bytes_host += s;
        }
        __syncthreads();
    }
    // ---------------- epilogue: final pressure, peak and its lowest slot, summary
    __syncthreads();
    long long pk = 0;
    int ps = -1;
#pragma unroll 1
    for (int k = tid; k < K; k += kOneThreads) {
        const long long pv = sP[k];
        A.P[k] = pv;
        if (ps < 0 || pv > pk) { pk = pv; ps = k; }      // k ascending per thread: first maximum kept
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const long long yk = __shfl_xor_sync(0xffffffffu, pk, o);
        const int ys = __shfl_xor_sync(0xffffffffu, ps, o);
        if (ys >= 0 && (ps < 0 || yk > pk || (yk == pk && ys < ps))) { pk = yk; ps = ys; }
    }
    if (lane == 0) { s_pk[warp] = pk; s_ps[warp] = ps; }
    __syncthreads();
    if (tid == 0) {
#pragma unroll 1
        for (int j = 1; j < kOneWarps; ++j)
            if (s_ps[j] >= 0 && (ps < 0 || s_pk[j] > pk || (s_pk[j] == pk && s_ps[j] < ps))) { pk = s_pk[j]; ps = s_ps[j]; }
        A.summary[0] = n_mig; A.summary[1] = rounds; A.summary[2] = status;
        A.summary[3] = ps < 0 ? 0 : pk; A.summary[4] = ps;
        A.summary[5] = bytes_ssd; A.summary[6] = bytes_host;
        if (!kBatch) *O.done = 1u;
    }
    // status bits found by this block: the batch keeps them per variant, a single plan in the call's status word
    dev_bits = __reduce_or_sync(0xffffffffu, dev_bits);
    if (lane == 0) s_fin[warp] = (int)dev_bits;           // (the finalist list is no longer in use)
    __syncthreads();
    if (tid == 0) {
        unsigned bits = 0;
#pragma unroll 1
        for (int j = 0; j < kOneWarps; ++j) bits |= (unsigned)s_fin[j];
        if (kBatch || kCyclic) A.summary[7] = bits;          // (the call-wide status word is folded in afterwards)
        else if (bits) raise_status(A.status, bits);
    }
}

// Shared memory a launch can offer (opt-in maximum minus the kernel's static part); 0 if the device query fails.
template <bool kBatch, bool kCyclic>
static int one_smem_budget()
{
    int dev = 0, optin = 0;
    cudaFuncAttributes fa;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return 0;
    if (cudaFuncGetAttributes(&fa, (const void *)k_plan_one<kBatch, kCyclic>) != cudaSuccess) return 0;
    const int room = optin - (int)fa.sharedSizeBytes;
    return room > 0 ? room : 0;
}

// Worth launching: the fixed part of the state (pressure, clock, bookings) leaves room for at least a few
// hundred periods.  Whether the periods fit too is only known on the device.
bool plan_one_possible(int64_t K, int64_t E, bool host_cap)
{
    if (K > 65000 || E < 1) return false;
    const int budget = one_smem_budget<false, false>();
    return budget > 0 && one_smem_need(K, E < 512 ? E : 512, host_cap) <= (size_t)budget;
}

cudaError_t launch_plan_one(const PlanArgs &A_in, const Workspace &w, cudaStream_t s)
{
    PlanArgs A = A_in;
    OneArgs O;
    BatchArgs B;
    B.variants = nullptr; B.P0 = nullptr; B.P_out = nullptr;
    O.done = w.one_done;
    O.smem_bytes = one_smem_budget<false, false>();
    cudaError_t e = cudaFuncSetAttribute((const void *)k_plan_one<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, O.smem_bytes);
    if (e != cudaSuccess) return e;
    k_plan_one<false, false><<<1, kOneThreads, (size_t)O.smem_bytes, s>>>(A, O, B); count_launch();
    return cudaGetLastError();
}

// Steady-state planning: A.start is the unrolled clock [2K + 1], the period and geometry arrays hold unrolled slots.
cudaError_t launch_plan_one_cyclic(const PlanArgs &A_in, const Workspace &w, cudaStream_t s)
{
    PlanArgs A = A_in;
    OneArgs O;
    BatchArgs B;
    B.variants = nullptr; B.P0 = nullptr; B.P_out = nullptr;
    O.done = w.one_done;
    O.smem_bytes = one_smem_budget<false, true>();
    cudaError_t e = cudaFuncSetAttribute((const void *)k_plan_one<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, O.smem_bytes);
    if (e != cudaSuccess) return e;
    k_plan_one<false, true><<<1, kOneThreads, (size_t)O.smem_bytes, s>>>(A, O, B); count_launch();
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Batch: one block per variant, then one block per variant again for the stability pairs.
// ---------------------------------------------------------------------------------------------
// stability[v] = (|M_v & M_0|, |M_v | M_0|) over the migrated periods of variant v and of variant 0; (-1, -1) if
// either plan is missing.  Also folds the call-wide status word (trace validation) into every variant's summary[7].
__global__ void __launch_bounds__(256) k_batch_finish(int64_t Pn_bound, const int64_t *Pn_dev, const g10_migration *out, int64_t out_cap,
                                                      int64_t *summary, int64_t *stability, const ull *status)
{
    extern __shared__ unsigned s_bits[];
    __shared__ int s_inter;
    const int v = blockIdx.x;
    const int64_t Pn = *Pn_dev < Pn_bound ? *Pn_dev : Pn_bound;
    const int words = (int)((Pn + 31) / 32);
    const int64_t n0 = summary[0] < out_cap ? summary[0] : out_cap, nv = summary[v * 8] < out_cap ? summary[v * 8] : out_cap;
    const bool ok = summary[2] >= 0 && summary[v * 8 + 2] >= 0;
    if (threadIdx.x == 0) s_inter = 0;
    for (int j = threadIdx.x; j < words; j += blockDim.x) s_bits[j] = 0;
    __syncthreads();
    if (ok) {
        for (int64_t j = threadIdx.x; j < n0; j += blockDim.x) { const int p = out[j].period; atomicOr(&s_bits[p >> 5], 1u << (p & 31)); }
        __syncthreads();
        int mine = 0;
        const g10_migration *mv = out + (size_t)v * out_cap;
        for (int64_t j = threadIdx.x; j < nv; j += blockDim.x) { const int p = mv[j].period; mine += (s_bits[p >> 5] >> (p & 31)) & 1u; }
        mine = __reduce_add_sync(0xffffffffu, mine);
        if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&s_inter, mine);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        stability[2 * v] = ok ? s_inter : -1;
        stability[2 * v + 1] = ok ? n0 + nv - s_inter : -1;
        summary[v * 8 + 7] |= (int64_t)*status;
    }
}

int batch_max_periods()          // periods whose bitmap fits the finishing kernel's shared memory
{
    return 200 * 1024 * 8;
}

static cudaError_t run_batch_finish(int64_t geo_stride, const int64_t *Pn_dev, const g10_migration *mig, int64_t out_cap, int64_t *summary,
                                    int V, int64_t *stability, const ull *status_word, cudaStream_t s)
{
    const int64_t bound = geo_stride < batch_max_periods() ? geo_stride : batch_max_periods();
    const size_t smem = (size_t)((bound + 31) / 32) * 4;
    cudaError_t e = cudaFuncSetAttribute((const void *)k_batch_finish, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_batch_finish<<<V, 256, smem, s>>>(bound, Pn_dev, mig, out_cap, summary, stability, status_word); count_launch();
    return cudaGetLastError();
}

cudaError_t launch_batch_finish(const DeviceTrace &t, const Workspace &w, const PlanParams &p, int V, int64_t *stability, const ull *status_word,
                                cudaStream_t s)
{
    return run_batch_finish(t.E > 0 ? t.E : 1, w.counts + 1, p.migrations, p.migrations_cap, p.summary, V, stability, status_word, s);
}

cudaError_t launch_plan_batch(const PlanArgs &A_in, const Workspace &w, int V, const BatchArgs &B, int64_t *stability, cudaStream_t s)
{
    PlanArgs A = A_in;
    OneArgs O;
    O.done = w.one_done;
    O.smem_bytes = one_smem_budget<true, false>();
    cudaError_t e = cudaFuncSetAttribute((const void *)k_plan_one<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, O.smem_bytes);
    if (e != cudaSuccess) return e;
    k_plan_one<true, false><<<V, kOneThreads, (size_t)O.smem_bytes, s>>>(A, O, B); count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    return run_batch_finish(A.geo_stride, A.Pn_dev, A.out, A.out_cap, A.summary, V, stability, A.status, s);
}

}  // namespace g10

// Algorithm 1 for traces whose timeline fits in shared memory (a few thousand kernels: every DNN-shaped
// configuration).  Each block keeps a private, identical copy of the planner state -- pressure and slot
// clock in shared memory, channel bookings and host occupancy in a private slice of global memory -- and
// owns a fixed share of the periods (period p belongs to block p mod G).  One iteration is then:
//   1. every block rescores those of its periods whose score can have changed (state STALE / DIRTY, as in
//      the large-trace planner), from shared memory;
//   2. block-local argmax, published with an iteration tag; every block polls all G tagged slots and reduces
//      them to the same global winner (this exchange is the only grid-wide synchronisation of the iteration);
//   3. every block applies the winner to its own copy of the state and reclassifies its own periods.
// Because all copies evolve identically no block ever reads another block's state, so no barrier separates
// the commit from the next scoring round.
#include "g10_planner.cuh"

namespace g10 {

enum { kFreshS = 1, kStaleS = 2, kDirtyS = 3 };

// A block's proposal travels as kXWords 64-bit words, each holding 32 bits of payload and the 32-bit
// iteration tag: a reader that finds the expected tag in a word knows the payload half next to it belongs
// to this iteration (64-bit accesses are single-copy atomic), so no fence is needed on either side.
constexpr int kXWords = 16;
struct XPayload {                // 64 bytes = 16 payload halves
    ull ben_lo, ben_hi;          // winner's benefit
    long long t;                 // transfer time (cost = 2 t)
    long long bytes;             // tensor size
    int idx, dest;               // period, destination (-1 = no candidate)
    int wa, wap, wbp, wb;        // evict slots [wa, wap-1], absent [wap, wbp], prefetch [wbp+1, wb]
    int tensor, pad;
};
static_assert(sizeof(XPayload) == 4 * kXWords, "payload must fill the exchange words");

struct SmallArgs {
    int64_t *busy_rep;      // [G][4][K]
    int64_t *hocc_rep;      // [G][K]
    ull *xwords;            // [2][G][kXWords] tagged proposals, then [2][G][kXWords] winner records, one copy per block
                            // (all start zeroed; tags start at 1)
    int cand_cap;           // periods a block can own
    const unsigned *done;   // non-zero: the single-block planner already produced the plan
};

// Static facts of an owned period, cached in shared memory for the whole run.
struct PeriodInfo {
    long long bytes;
    long long t[2];
    int a, b;                // inactive slots [a, b] = [u+1, v-1]
    int ap[2], bp[2];        // absent range per destination (ap < 0: unusable)
    int tensor, pad;
};

// busy + overlap <= dur over slots k0..k1 for the window [w0, w1), clock in shared memory; whole warp
__device__ __forceinline__ bool window_free_s(const int64_t *sStart, const int64_t *busy, int64_t w0, int64_t w1, int k0, int k1, int lane)
{
    bool ok = true;
#pragma unroll 1
    for (int k = k0 + lane; k <= k1; k += 32) {
        const int64_t s0 = sStart[k], s1 = sStart[k + 1];
        const int64_t lo = w0 > s0 ? w0 : s0, hi = w1 < s1 ? w1 : s1;
        const int64_t ov = hi > lo ? hi - lo : 0;
        if (__ldcg(&busy[k]) + ov > s1 - s0) ok = false;      // bookings are reductions performed at L2
    }
    return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void st_volatile_u64(ull *p, ull v)
{
    asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Half-warp poll: lanes 0-15 (or 16-31) of a warp each read one word of a record, so that a poll is one
// coalesced 128-byte request.  Returns when all 16 words carry `tag` (the payload word of every lane is then
// in *word); gives up (false) when the grid-wide error flag is raised or after kBarrierTimeoutNs, raising
// the flag itself.  `active` lanes must form complete half-warps; inactive lanes pass through.
__device__ __forceinline__ bool poll_record_halfwarp(const ull *rec, bool active, ull tag, unsigned *word, unsigned *error_flag)
{
    const int lane = threadIdx.x & 31;
    const unsigned half_mask = (lane < 16) ? 0x0000ffffu : 0xffff0000u;
    const unsigned act = __ballot_sync(0xffffffffu, active);
    unsigned polls = 0;
    ull t0 = 0;
    bool ok = true;
    for (;;) {
        bool mine_ok = true;
        if (active) {
            ull x;
            asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(x) : "l"(rec + (lane & 15)) : "memory");
            mine_ok = (x & 0xffffffff00000000ull) == tag;
            *word = (unsigned)x;
        }
        const unsigned good = __ballot_sync(0xffffffffu, mine_ok);
        // done when every active half-warp is complete
        const bool lo_done = ((act & 0x0000ffffu) == 0u) || ((good & 0x0000ffffu) == 0x0000ffffu);
        const bool hi_done = ((act & 0xffff0000u) == 0u) || ((good & 0xffff0000u) == 0xffff0000u);
        (void)half_mask;
        if (lo_done && hi_done) break;
        if ((++polls & 255u) == 0u) {
            if (t0 == 0) t0 = global_timer_ns();
            const bool stop = ld_acquire_u32(error_flag) || global_timer_ns() - t0 > kBarrierTimeoutNs;
            if (__any_sync(0xffffffffu, stop)) { ok = false; break; }
        }
    }
    if (!ok && lane == 0) atomicExch(error_flag, 1u);
    return ok;
}


// kFew: every block owns at most 256 periods (warp 0 alone finds the block's best candidate).
template <bool kFew>
__global__ void __launch_bounds__(kPlanThreads, 1) k_plan_small(PlanArgs A, SmallArgs S)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ Cand s_cand[kPlanWarps + 1];
    __shared__ BestScratch s_best;
    __shared__ XPayload s_pay;
    __shared__ __align__(16) unsigned char s_recs[kSmallMaxBlocks * sizeof(XPayload)];
    __shared__ int s_n_over;
    __shared__ unsigned s_err;
    if (*S.done) return;                  // same answer in every thread of the grid: written by an earlier launch
    const int G = gridDim.x, c = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int K = (int)A.K;
    const int64_t Pn = *A.Pn_dev < A.geo_stride ? *A.Pn_dev : A.geo_stride;
    const int64_t limit = (A.max_iterations <= 0 || A.max_iterations > Pn) ? Pn : A.max_iterations;
    const int n_local = (int)((Pn - c + G - 1) / G > 0 ? (Pn - c + G - 1) / G : 0);     // periods c, c + G, ...

    int64_t *sP = (int64_t *)smem_raw;
    int64_t *sStart = sP + K;
    int64_t *sDur = sStart + K + 1;
    ull *cben_lo = (ull *)(sDur + K);
    ull *cben_hi = cben_lo + S.cand_cap;
    double *ckey = (double *)(cben_hi + S.cand_cap);        // rounded benefit/cost of the cached score
    PeriodInfo *info = (PeriodInfo *)(ckey + S.cand_cap);
    unsigned char *cstate = (unsigned char *)(info + S.cand_cap);
    unsigned char *cskip = cstate + S.cand_cap;             // STALE period that cannot be this block's proposal in this iteration
    const int NT = (K + kTileO - 1) / kTileO;
    int64_t *tmin = (int64_t *)(((uintptr_t)(cskip + S.cand_cap) + 7) & ~(uintptr_t)7);   // [NT] smallest pressure per tile of 32 slots
    int64_t *tmax = tmin + NT;                                                             // [NT] largest
    int64_t *busy = S.busy_rep + (size_t)c * 4 * K;
    int64_t *hocc = S.hocc_rep + (size_t)c * K;

    if (threadIdx.x == 0) { s_n_over = 0; s_err = 0; }
    __syncthreads();
    {
        int over = 0;
#pragma unroll 1
        for (int k = threadIdx.x; k < K; k += kPlanThreads) {
            const int64_t pv = A.P[k];
            sP[k] = pv;
            if (pv > A.cap) ++over;
        }
#pragma unroll 1
        for (int k = threadIdx.x; k <= K; k += kPlanThreads) sStart[k] = A.start[k];
#pragma unroll 1
        for (int k = threadIdx.x; k < K; k += kPlanThreads) sDur[k] = A.dur[k];
#pragma unroll 1
        for (int li = threadIdx.x; li < n_local; li += kPlanThreads) {
            const int64_t p = (int64_t)li * G + c;
            PeriodInfo I;
            I.tensor = A.per_t[p];
            I.bytes = A.bytes[I.tensor];
            I.a = A.per_u[p] + 1; I.b = A.per_v[p] - 1;
#pragma unroll 1
            for (int X = 0; X < 2; ++X) {
                I.t[X] = A.geo_t[X * A.geo_stride + p];
                I.ap[X] = A.geo_a[X * A.geo_stride + p];
                I.bp[X] = A.geo_b[X * A.geo_stride + p];
            }
            I.pad = 0;
            info[li] = I;
            cstate[li] = (unsigned char)(kDirtyS << 2);
        }
#pragma unroll 1
        for (int k = threadIdx.x; k < 4 * K; k += kPlanThreads) busy[k] = 0;
        if (A.host_capacity != 0) for (int k = threadIdx.x; k < K; k += kPlanThreads) hocc[k] = 0;
        if (over) atomicAdd(&s_n_over, over);
    }
    __syncthreads();
    for (int t = warp; t < NT; t += kPlanWarps) tile_refresh_warp(sP, K, t, tmin, tmax, lane);
    __syncthreads();

    int64_t n_mig = 0, rounds = 0, bytes_ssd = 0, bytes_host = 0;
    int status = -1;
#pragma unroll 1
    for (int64_t it = 0;; ++it) {
        if (A.fits_always || s_n_over == 0) { status = n_mig == 0 ? G10_ALREADY_FITS : G10_FIT; break; }
        if (it >= limit) { status = limit < Pn ? G10_ITERATION_LIMIT : G10_EXHAUSTED; break; }
        rounds += 1;
        if (kFew) for (int li = threadIdx.x; li < n_local; li += kPlanThreads) cskip[li] = 0;
        // ---------------- 1. bring this block's periods up to date (one warp per period).  With few periods per
        // block only the DIRTY ones are done here (rare); STALE ones are rescored on demand in step 2.
#pragma unroll 1
        for (int li = warp; li < n_local; li += kPlanWarps) {
            const unsigned char st = cstate[li];
            if (st == 0 || (st >> 2) == kFreshS) continue;
            if (kFew && (st >> 2) == kStaleS) continue;
            const int a = info[li].a, b = info[li].b;
            const int64_t s = info[li].bytes;
            int d = (st & 3) - 1;
            if ((st >> 2) == kDirtyS) {
                const int64_t t_r = sStart[a], t_end = sStart[b + 1];
                d = -1;
#pragma unroll 1
                for (int X = 0; X < 2 && d < 0; ++X) {
                    const int ap = info[li].ap[X];
                    if (ap < 0) continue;
                    const int bp = info[li].bp[X];
                    const int64_t t = info[li].t[X];
                    if (!window_free_s(sStart, busy + (size_t)(2 * X) * K, t_r, t_r + t, a, ap - 1, lane)) continue;
                    if (!window_free_s(sStart, busy + (size_t)(2 * X + 1) * K, t_end - t, t_end, bp + 1, b, lane)) continue;
                    if (X == G10_DEST_HOST && A.host_capacity != 0) {
                        bool ok = true;
#pragma unroll 1
                        for (int k = a + lane; k <= b; k += 32)
                            if ((uint64_t)__ldcg(&hocc[k]) + (uint64_t)s > A.host_capacity) ok = false;
                        if (!__all_sync(0xffffffffu, ok)) continue;
                    }
                    d = X;
                }
                if (d < 0) { if (lane == 0) cstate[li] = 0; continue; }     // channels only fill up: gone for good
            }
            const int ap = info[li].ap[d], bp = info[li].bp[d];
            u128 acc = 0;
#pragma unroll 1
            for (int k = ap + lane; k <= bp; k += 32) {
                int64_t ex = sP[k] - A.cap;
                if (ex > 0) {
                    if (ex > s) ex = s;
                    acc += (u128)(ull)ex * (u128)(ull)sDur[k];
                }
            }
            acc = warp_sum_u128(acc);
            if (lane == 0) {
                Cand cd;
                cd.ben = acc; cd.cost = 2ull * (ull)info[li].t[d]; cd.idx = 0; cd.dest = d;
                cben_lo[li] = (ull)acc; cben_hi[li] = (ull)(acc >> 64);
                ckey[li] = acc == 0 ? 0.0 : cand_key(cd);
                cstate[li] = (unsigned char)((d + 1) | (kFreshS << 2));
            }
        }
        __syncthreads();
        // ---------------- 2. block-local argmax, published as tagged words
        const int par = (int)(it & 1);
        const ull tag = (ull)(unsigned)(it + 1) << 32;
        if (kFew) {
            // Few periods per block.  A STALE period's cached score is an upper bound (pressure only falls), so
            // only the STALE periods whose bound could still beat the best FRESH score are rescored, best bound
            // first, by warp 0 from the pressure tiles; the loop ends when the block's best is FRESH (exact).  Rounded ratios
            // (ckey) steer the search; anything within 1e-10 of a decision is settled by exact comparison.
            if (warp == 0) {
#pragma unroll 1
                for (;;) {
                    double kf = -1.0, ks = -1.0;
                    int lf = -1, ls = -1;
#pragma unroll 1
                    for (int li = lane; li < n_local; li += 32) {
                        const unsigned char st = cstate[li];
                        if (st == 0) continue;
                        const double key = ckey[li];
                        if (!(key > 0.0)) continue;                   // no benefit: never a winner
                        if ((st >> 2) == kFreshS) {
                            bool take = key > kf;
                            if (lf >= 0 && key >= kf * (1.0 - 1e-10) && kf >= key * (1.0 - 1e-10)) {
                                Cand x, y;                               // too close to call by rounding: exact
                                x.ben = ((u128)cben_hi[li] << 64) | cben_lo[li]; x.cost = 2ull * (ull)info[li].t[(st & 3) - 1];
                                x.idx = (int)((int64_t)li * G + c); x.dest = 0;
                                const unsigned char sf = cstate[lf];
                                y.ben = ((u128)cben_hi[lf] << 64) | cben_lo[lf]; y.cost = 2ull * (ull)info[lf].t[(sf & 3) - 1];
                                y.idx = (int)((int64_t)lf * G + c); y.dest = 0;
                                take = cand_beats(x, y);
                            }
                            if (take) { kf = key; lf = li; }
                        } else if (!cskip[li] && key > ks) { ks = key; ls = li; }
                    }
                    double mf = kf, ms = ks;
#pragma unroll 1
                    for (int o = 16; o > 0; o >>= 1) {
                        const double yf = __shfl_xor_sync(0xffffffffu, mf, o), ys = __shfl_xor_sync(0xffffffffu, ms, o);
                        if (yf > mf) mf = yf;
                        if (ys > ms) ms = ys;
                    }
                    // A STALE bound clearly above the best FRESH score has to be rescored; one within 1e-10 of it only
                    // if the bound can win exactly (benefit and cost of the cached score, ties to the lower index):
                    // otherwise the period cannot be this block's proposal in this iteration and is set aside.
                    const bool above = ls >= 0 && ks > 0.0 && (!(mf > 0.0) || ks > mf * (1.0 + 1e-10));
                    const bool near = ls >= 0 && ks > 0.0 && mf > 0.0 && !above && ks >= mf * (1.0 - 1e-10);
                    // the block's exact best FRESH period (near-ties between lanes settled exactly): needed to decide a
                    // near-tie and to publish, not when a bound is clearly above and gets rescored anyway
                    const bool any_near = __any_sync(0xffffffffu, near);
                    const bool need_best = any_near || !__any_sync(0xffffffffu, above);
                    int src = -1;
                    Cand best;
                    best.ben = 0; best.cost = 1; best.idx = -1; best.dest = -1;
                    if (need_best) {
                        const unsigned fin = __ballot_sync(0xffffffffu, lf >= 0 && kf >= mf * (1.0 - 1e-10));
                        if (lf >= 0) {
                            const unsigned char sf = cstate[lf];
                            best.ben = ((u128)cben_hi[lf] << 64) | cben_lo[lf]; best.dest = (sf & 3) - 1;
                            best.cost = 2ull * (ull)info[lf].t[best.dest]; best.idx = (int)((int64_t)lf * G + c);
                        }
                        if (__popc(fin) == 1) src = __ffs(fin) - 1;
                        else if (fin != 0u) {
                            // usual case of a tie: identical benefit and cost (repeated layers): the lowest index wins
                            const int f0 = __ffs(fin) - 1;
                            // (every lane takes part in the shuffles: no short-circuit around them)
                            const ull b0 = __shfl_sync(0xffffffffu, (ull)best.ben, f0);
                            const ull b1 = __shfl_sync(0xffffffffu, (ull)(best.ben >> 64), f0);
                            const ull c0 = __shfl_sync(0xffffffffu, best.cost, f0);
                            const bool same = !((fin >> lane) & 1u) || ((ull)best.ben == b0 && (ull)(best.ben >> 64) == b1 && best.cost == c0);
                            if (__all_sync(0xffffffffu, same)) {
                                const unsigned lowest = __reduce_min_sync(0xffffffffu, ((fin >> lane) & 1u) ? (unsigned)best.idx : 0xffffffffu);
                                src = __ffs(__ballot_sync(0xffffffffu, ((fin >> lane) & 1u) && (unsigned)best.idx == lowest)) - 1;
                            } else {
                            Cand z = best;
                            if (!((fin >> lane) & 1u)) z.idx = -1;
#pragma unroll 1
                            for (int o = 16; o > 0; o >>= 1) {
                                const Cand y = cand_shfl_xor(z, o);
                                if (cand_beats(y, z)) z = y;
                            }
                            src = __ffs(__ballot_sync(0xffffffffu, best.idx >= 0 && best.idx == z.idx)) - 1;
                            }
                        }
                    }
                    Cand zbest = best;
                    bool can = above, set_aside = false;
                    if (any_near) {
                        // (every lane needs the exact best: broadcast it from its lane)
                        const int from = src < 0 ? 0 : src;
                        zbest.ben = ((u128)__shfl_sync(0xffffffffu, (ull)(best.ben >> 64), from) << 64) | __shfl_sync(0xffffffffu, (ull)best.ben, from);
                        zbest.cost = __shfl_sync(0xffffffffu, best.cost, from);
                        zbest.idx = __shfl_sync(0xffffffffu, best.idx, from);
                        if (near) {
                            Cand x;
                            const unsigned char ss = cstate[ls];
                            x.ben = ((u128)cben_hi[ls] << 64) | cben_lo[ls]; x.cost = 2ull * (ull)info[ls].t[(ss & 3) - 1];
                            x.idx = (int)((int64_t)ls * G + c); x.dest = 0;
                            can = src < 0 || cand_beats(x, zbest);
                            if (!can) { cskip[ls] = 1; set_aside = true; }
                        }
                    }
                    int todo = -1;
                    const unsigned want = __ballot_sync(0xffffffffu, can);
                    if (want) {
                        double m2 = can ? ks : -1.0;
#pragma unroll 1
                        for (int o = 16; o > 0; o >>= 1) { const double y = __shfl_xor_sync(0xffffffffu, m2, o); if (y > m2) m2 = y; }
                        const unsigned who = __ballot_sync(0xffffffffu, can && ks == m2);
                        todo = __shfl_sync(0xffffffffu, ls, __ffs(who) - 1);
                    } else if (__any_sync(0xffffffffu, set_aside)) {
                        todo = -2;                                 // look again: a lane may hold further STALE periods
                    } else {
                        // the block's best is FRESH: build the record
                        if (src < 0) {
                            if (lane == 0) { s_pay.idx = -1; s_pay.dest = -1; s_pay.ben_lo = 0; s_pay.ben_hi = 0; s_pay.t = 0; }
                        } else if (lane == src) {
                            const PeriodInfo &I = info[lf];
                            XPayload q;
                            q.ben_lo = (ull)best.ben; q.ben_hi = (ull)(best.ben >> 64); q.idx = best.idx; q.dest = best.dest;
                            q.t = I.t[best.dest]; q.bytes = I.bytes; q.wa = I.a; q.wb = I.b; q.wap = I.ap[best.dest]; q.wbp = I.bp[best.dest];
                            q.tensor = I.tensor; q.pad = 0;
                            s_pay = q;
                        }
                        __syncwarp();
                        if (lane < kXWords)
                            st_volatile_u64(&S.xwords[((size_t)par * G + c) * kXWords + lane], tag | ((const unsigned *)&s_pay)[lane]);
                    }
                    if (todo == -1) break;                     // published
                    if (todo == -2) { __syncwarp(); continue; }
                    // warp 0 rescores period `todo` from the pressure tiles and looks again
                    {
                        const int li = todo;
                        const unsigned char st = cstate[li];
                        const int d = (st & 3) - 1;
                        const u128 tot = warp_sum_u128(benefit_tiles_warp(sP, sStart, tmin, tmax, A.cap, info[li].bytes, info[li].ap[d], info[li].bp[d], lane));
                        if (lane == 0) {
                            Cand cd;
                            cd.ben = tot; cd.cost = 2ull * (ull)info[li].t[d]; cd.idx = 0; cd.dest = d;
                            cben_lo[li] = (ull)tot; cben_hi[li] = (ull)(tot >> 64);
                            ckey[li] = tot == 0 ? 0.0 : cand_key(cd);
                            cstate[li] = (unsigned char)((d + 1) | (kFreshS << 2));
                        }
                        __syncwarp();
                    }
                }
            }
            __syncthreads();
        } else {
            Cand best;
            best.ben = 0; best.cost = 1; best.idx = -1; best.dest = -1;
#pragma unroll 1
            for (int li = threadIdx.x; li < n_local; li += kPlanThreads) {
                const unsigned char st = cstate[li];
                if (st == 0) continue;
                Cand x;
                x.ben = ((u128)cben_hi[li] << 64) | cben_lo[li];
                if (x.ben == 0) continue;
                x.dest = (st & 3) - 1;
                x.cost = 2ull * (ull)info[li].t[x.dest]; x.idx = (int)((int64_t)li * G + c);
                if (cand_beats(x, best)) best = x;
            }
            best = block_best_fast(best, &s_best, s_cand);
            if (threadIdx.x == 0) {
                XPayload q;
                q.ben_lo = (ull)best.ben; q.ben_hi = (ull)(best.ben >> 64); q.idx = best.idx; q.dest = best.dest;
                q.t = 0; q.bytes = 0; q.wa = q.wap = q.wbp = q.wb = 0; q.tensor = 0; q.pad = 0;
                if (best.idx >= 0) {
                    const PeriodInfo &I = info[best.idx / G];
                    q.t = I.t[best.dest]; q.bytes = I.bytes; q.wa = I.a; q.wb = I.b; q.wap = I.ap[best.dest]; q.wbp = I.bp[best.dest];
                    q.tensor = I.tensor;
                }
                s_pay = q;
            }
            __syncthreads();
            if (threadIdx.x < kXWords)
                st_volatile_u64(&S.xwords[((size_t)par * G + c) * kXWords + threadIdx.x], tag | ((const unsigned *)&s_pay)[threadIdx.x]);
            __syncthreads();                               // s_pay is reused for the winner's record below
        }
        // ---------------- block 0 reads all G proposals (one half-warp per record), reduces them and writes one
        // copy of the winner's record per block; every other block polls its own copy (no hot line)
        ull *win_words = &S.xwords[((size_t)2 * G + (size_t)par * G) * kXWords];      // [G] copies for this parity
        if (c == 0) {
            XPayload *recs = (XPayload *)s_recs;
#pragma unroll 1
            for (int j0 = 0; j0 < G; j0 += kPlanThreads / 16) {
                const int j = j0 + (threadIdx.x >> 4);
                unsigned word = 0;
                const bool active = j < G;
                if (!poll_record_halfwarp(&S.xwords[((size_t)par * G + (active ? j : 0)) * kXWords], active, tag, &word, &A.bar->error))
                    s_err = 1u;
                if (active) ((unsigned *)&recs[j])[threadIdx.x & 15] = word;
            }
            __syncthreads();
            Cand x;
            x.ben = 0; x.cost = 1; x.idx = -1; x.dest = -1;
#pragma unroll 1
            for (int j = threadIdx.x; j < G; j += kPlanThreads) {
                const XPayload &y = recs[j];
                if (y.idx < 0) continue;
                Cand cy;
                cy.ben = ((u128)y.ben_hi << 64) | y.ben_lo; cy.cost = 2ull * (ull)y.t; cy.idx = y.idx; cy.dest = y.dest;
                if (cand_beats(cy, x)) x = cy;
            }
            const Cand gw = block_best_fast(x, &s_best, s_cand);         // (its barriers also publish s_err)
            if (threadIdx.x == 0) {
                if (gw.idx < 0) { s_pay.idx = -1; s_pay.dest = -1; }
                else s_pay = recs[gw.idx % G];             // period p was proposed by block p mod G
            }
            __syncthreads();
            if (!s_err)
#pragma unroll 1
                for (int w = threadIdx.x; w < G * kXWords; w += kPlanThreads)
                    st_volatile_u64(&win_words[w], tag | ((const unsigned *)&s_pay)[w & (kXWords - 1)]);
        } else {
            if (warp == 0) {
                unsigned word = 0;
                const bool active = lane < 16;
                if (!poll_record_halfwarp(&win_words[(size_t)c * kXWords], active, tag, &word, &A.bar->error)) s_err = 1u;
                else if (active) ((unsigned *)&s_pay)[lane] = word;
            }
            __syncthreads();
        }
        if (s_err) { status = -2; break; }
        const XPayload win = s_pay;
        if (win.idx < 0) { status = G10_EXHAUSTED; break; }
        // ---------------- 3. apply the winner to this block's copy of the state
        {
            const int64_t p = win.idx;
            const int X = win.dest;
            const int wa = win.wa, wb = win.wb, wap = win.wap, wbp = win.wbp;
            const int64_t s = win.bytes, t = win.t;
            const int64_t t_r = sStart[wa], t_end = sStart[wb + 1];
            int64_t *bo = busy + (size_t)(2 * X) * K, *bi = busy + (size_t)(2 * X + 1) * K;
            // reclassify this block's periods against the winner's slot ranges; the bookings are not in `busy` yet
            // (the sums of the two shared boundary slots are formed here), so this runs before they are added
#pragma unroll 1
            for (int li = threadIdx.x; li < n_local; li += kPlanThreads) {
                const unsigned char st = cstate[li];
                if (st == 0) continue;
                if ((int64_t)li * G + c == p) { cstate[li] = 0; continue; }
                int state = st >> 2;
                if (state == kDirtyS) continue;
                const int d = (st & 3) - 1;
                const int qa = info[li].a, qb = info[li].b;
                if (!(qa <= wb && wa <= qb)) continue;
                const int ap = info[li].ap[d], bp = info[li].bp[d];
                bool hit = false;
                if (d == X) {
                    const bool meet_out = qa <= wap - 1 && wa <= ap - 1, meet_in = bp + 1 <= wb && wbp + 1 <= qb;
                    if (meet_out || meet_in) {
                        const int64_t tq = info[li].t[d];
                        const int64_t q_r = sStart[qa], q_end = sStart[qb + 1];
                        hit = (meet_out && window_conflict<false, true>(sStart, bo, wa, wap - 1, t_r, t_r + t, q_r, q_r + tq, qa, ap - 1)) ||
                              (meet_in && window_conflict<false, true>(sStart, bi, wbp + 1, wb, t_end - t, t_end, q_end - tq, q_end, bp + 1, qb));
                    }
                    if (!hit && d == G10_DEST_HOST && A.host_capacity != 0) hit = true;
                }
                if (hit) state = kDirtyS;
                else if (state == kFreshS && ap <= wbp && wap <= bp) state = kStaleS;
                cstate[li] = (unsigned char)((st & 3) | (state << 2));
            }
            __syncthreads();
            int fell = 0;
#pragma unroll 1
            for (int k = wap + threadIdx.x; k <= wbp; k += kPlanThreads) {
                const int64_t before = sP[k], after = before - s;
                sP[k] = after;
                if (before > A.cap && after <= A.cap) ++fell;
            }
            if (fell) atomicSub(&s_n_over, fell);
#pragma unroll 1
            for (int k = wa + threadIdx.x; k <= wap - 1; k += kPlanThreads) {
                const int64_t s0 = sStart[k], s1 = sStart[k + 1];
                const int64_t lo = t_r > s0 ? t_r : s0, hi = (t_r + t) < s1 ? (t_r + t) : s1;
                if (hi > lo) atomicAdd((ull *)&bo[k], (ull)(hi - lo));
            }
#pragma unroll 1
            for (int k = wbp + 1 + threadIdx.x; k <= wb; k += kPlanThreads) {
                const int64_t s0 = sStart[k], s1 = sStart[k + 1];
                const int64_t lo = (t_end - t) > s0 ? (t_end - t) : s0, hi = t_end < s1 ? t_end : s1;
                if (hi > lo) atomicAdd((ull *)&bi[k], (ull)(hi - lo));
            }
            if (X == G10_DEST_HOST && A.host_capacity != 0)
#pragma unroll 1
                for (int k = wa + threadIdx.x; k <= wb; k += kPlanThreads) atomicAdd((ull *)&hocc[k], (ull)s);
            if (c == 0 && threadIdx.x == 0) {
                if (n_mig < A.out_cap) {
                    g10_migration m;
                    m.period = (int32_t)p; m.tensor = win.tensor; m.dest = X; m.absent_first = wap; m.absent_last = wbp;
                    m.iteration = (int32_t)it; m.evict_issue_ns = t_r; m.prefetch_issue_ns = t_end - t; m.transfer_ns = t;
                    A.out[n_mig] = m;
                } else raise_status(A.status, G10_DEV_PLAN_OVERFLOW);
            }
            n_mig += 1;
            if (X == G10_DEST_SSD) bytes_ssd += s; else bytes_host += s;
            __syncthreads();                               // the pressure is updated: refresh the tiles the commit touched
            for (int tl = wap / kTileO + warp; tl <= wbp / kTileO; tl += kPlanWarps) tile_refresh_warp(sP, K, tl, tmin, tmax, lane);
        }
        __syncthreads();
    }
    // ---------------- epilogue: block 0 writes the final pressure and the summary
    if (c != 0) return;
    __syncthreads();

    long long pk = 0;
    int ps = -1;
#pragma unroll 1
    for (int k = threadIdx.x; k < K; k += kPlanThreads) {
        const long long pv = sP[k];
        A.P[k] = pv;
        if (ps < 0 || pv > pk) { pk = pv; ps = k; }      // k ascending per thread: first maximum kept
    }
    __shared__ long long s_pk[kPlanThreads];
    __shared__ int s_ps[kPlanThreads];
    s_pk[threadIdx.x] = pk; s_ps[threadIdx.x] = ps;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll 1
        for (int j = 1; j < kPlanThreads; ++j)
            if (s_ps[j] >= 0 && (ps < 0 || s_pk[j] > pk || (s_pk[j] == pk && s_ps[j] < ps))) { pk = s_pk[j]; ps = s_ps[j]; }
        if (status == -2) raise_status(A.status, G10_DEV_TIMEOUT);
        A.summary[0] = n_mig; A.summary[1] = rounds; A.summary[2] = status == -2 ? -1 : status;
        A.summary[3] = ps < 0 ? 0 : pk; A.summary[4] = ps;
        A.summary[5] = bytes_ssd; A.summary[6] = bytes_host;
    }
}

// Shared memory the small-trace planner needs for K slots and `cand_cap` periods per block.
static size_t small_smem_bytes(int64_t K, int cand_cap)
{
    return (size_t)(3 * K + 1) * 8 + (size_t)cand_cap * (24 + sizeof(PeriodInfo) + 2) + 16 + 8 + (size_t)((K + 31) / 32) * 16;
}

bool plan_small_fits(int64_t K, int64_t E, int G, int *cand_cap_out, size_t *smem_out)
{
    if (G < 1) return false;
    const int cand_cap = (int)((E + G - 1) / G) + 1;
    const size_t smem = small_smem_bytes(K, cand_cap);
    *cand_cap_out = cand_cap;
    *smem_out = smem;
    return smem <= 200 * 1024;
}

int plan_small_blocks()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return sms > kMaxPlanBlocks ? kMaxPlanBlocks : sms;
}

cudaError_t launch_plan_small(const PlanArgs &A_in, const Workspace &w, int G, int cand_cap, size_t smem, cudaStream_t s)
{
    PlanArgs A = A_in;
    SmallArgs S;
    S.busy_rep = w.busy_rep; S.hocc_rep = w.hocc_rep; S.xwords = w.xwords; S.cand_cap = cand_cap; S.done = w.one_done;
    const void *kernel = cand_cap <= 256 ? (const void *)k_plan_small<true> : (const void *)k_plan_small<false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    void *args[] = {&A, &S};
    return cudaLaunchCooperativeKernel(kernel, dim3(G), dim3(kPlanThreads), args, smem, s);
}

}  // namespace g10

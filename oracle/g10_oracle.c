/*
 * g10_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-threaded CPU restatement of the compile-time planning path of G10
 * (tensor vitality analysis, Section 4.2; GPU memory pressure, Section 4.3; the smart tensor
 * eviction loop, Algorithm 1).  It exists so that the CUDA library can be compared against
 * something written directly from the paper's definitions.  It shares no code, header, table or
 * helper with the CUDA path, and nothing outside tests / the smoke check / the benchmark's CPU
 * baseline may call it.
 *
 * Everything is integer.  Times are nanoseconds, sizes are bytes.  "u128" is an exact unsigned
 * 128-bit integer.  Where the paper leaves a point open the reading taken is stated next to the
 * code that implements it.
 *
 * Pins (tests that tie each function to something other than itself):
 *   g10o_slot_clock, g10o_vitality, g10o_pressure : dense kernel-by-tensor matrix brute force,
 *       closed forms for the MLP-chain trace, conservation of byte-slots.
 *   g10o_geometry : hand-worked examples, dense per-nanosecond brute force on toy traces.
 *   g10o_plan (plain tier) : three hand-worked traces, an independent arbitrary-precision Python
 *       restatement on random toy traces, plan invariants (excess-area identity, channel budgets,
 *       residency at every use).  The paper prints no numeric example of Algorithm 1 (its figures
 *       did not survive), so agreement with the paper's own numbers is "parity unpinned".
 *   g10o_plan (lazy tier) : must equal the plain tier bit for bit.
 *   g10o_schedule_prefetch : a hand-worked example, a dense slot-by-slot restatement on toy plans, invariants
 *       (capacity never exceeded by the pass, bytes added = size x slots regained, issue times only earlier).
 *   g10o_emit_instructions : the stream of hand-worked example A, a dense restatement on toy traces, structural
 *       invariants (one ALLOC per used tensor, one FREE per intermediate tensor, order inside a boundary).
 *   g10o_characterize : dense restatement on toy traces, closed forms on the MLP chain, conservation identities
 *       (sum of active bytes = sum of size x uses, active <= pressure, hidden-latency counts against the geometry).
 *   batched re-planning (g10_oracle.py, plan_batch: a loop of g10o_plan plus set arithmetic) : every variant against
 *       the dense brute force, the set identities of the stability pairs.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;

enum { DEST_SSD = 0, DEST_HOST = 1 };
enum { CH_SSD_OUT = 0, CH_SSD_IN = 1, CH_HOST_OUT = 2, CH_HOST_IN = 3 };
enum { ST_ALREADY_FITS = 0, ST_FIT = 1, ST_EXHAUSTED = 2, ST_ITERATION_LIMIT = 3 };

#define T_SATURATE ((int64_t)1 << 62)

typedef struct {
    int32_t period, tensor, dest;
    int32_t absent_first, absent_last;
    int32_t iteration;
    int64_t evict_issue_ns, prefetch_issue_ns, transfer_ns;
} g10o_migration;

/* ------------------------------------------------------------------------------------------
 * Slot clock (Section 4.2: kernel execution times measure the inactive periods).
 * Reading: kernels run back to back in trace order, so kernel k occupies [start[k], start[k+1]).
 * ---------------------------------------------------------------------------------------- */
void g10o_slot_clock(int64_t K, const int64_t *kernel_ns, int64_t *start /* [K+1] */)
{
    start[0] = 0;
    for (int64_t k = 0; k < K; ++k) start[k + 1] = start[k] + kernel_ns[k];
}

/* ------------------------------------------------------------------------------------------
 * Tensor vitality (Section 4.2).
 * A tensor is active while a kernel that lists it (input or output) runs.  U_i is the sorted set
 * of distinct kernels listing tensor i (a kernel that lists a tensor twice, as an in-place
 * operator does, uses it once).  Born at min U_i, dead after max U_i.  Between two consecutive
 * uses u < v with at least one kernel in between (v - u >= 2) the tensor is inactive and not
 * dead: one inactive period (i, u, v).  Periods are numbered by (tensor, u) ascending.
 * Returns 0, or -1 if uses_cap / periods_cap is too small (counts[] still holds the need).
 * ---------------------------------------------------------------------------------------- */
int32_t g10o_vitality(int64_t K, int64_t N, const int64_t *kernel_ptr, const int32_t *kernel_tensors,
                      int32_t *first_use, int32_t *last_use, int32_t *num_uses,
                      int64_t *use_ptr /* [N+1] */, int32_t *uses, int64_t uses_cap,
                      int64_t *period_ptr /* [N+1] */, int32_t *period_tensor, int32_t *period_prev_use,
                      int32_t *period_next_use, int64_t periods_cap, int64_t *counts /* [2] */)
{
    int32_t *seen = (int32_t *)malloc(sizeof(int32_t) * (size_t)(N > 0 ? N : 1));
    int64_t *fill = (int64_t *)malloc(sizeof(int64_t) * (size_t)(N > 0 ? N : 1));
    for (int64_t i = 0; i < N; ++i) { seen[i] = -1; num_uses[i] = 0; }
    /* |U_i| : kernels are visited in increasing order, so a repeat inside one kernel is caught
       by remembering the last kernel that listed the tensor. */
    for (int64_t k = 0; k < K; ++k)
        for (int64_t e = kernel_ptr[k]; e < kernel_ptr[k + 1]; ++e) {
            int32_t i = kernel_tensors[e];
            if (seen[i] != (int32_t)k) { seen[i] = (int32_t)k; num_uses[i] += 1; }
        }
    use_ptr[0] = 0;
    for (int64_t i = 0; i < N; ++i) use_ptr[i + 1] = use_ptr[i] + num_uses[i];
    counts[0] = use_ptr[N];
    int32_t rc = 0;
    if (use_ptr[N] > uses_cap) rc = -1;
    if (rc == 0) {
        for (int64_t i = 0; i < N; ++i) { seen[i] = -1; fill[i] = use_ptr[i]; }
        for (int64_t k = 0; k < K; ++k)
            for (int64_t e = kernel_ptr[k]; e < kernel_ptr[k + 1]; ++e) {
                int32_t i = kernel_tensors[e];
                if (seen[i] != (int32_t)k) { seen[i] = (int32_t)k; uses[fill[i]++] = (int32_t)k; }
            }
    }
    /* born / dead, and the inactive periods */
    int64_t np = 0;
    period_ptr[0] = 0;
    for (int64_t i = 0; i < N; ++i) {
        if (num_uses[i] == 0) { first_use[i] = -1; last_use[i] = -1; }
        else if (rc == 0) { first_use[i] = uses[use_ptr[i]]; last_use[i] = uses[use_ptr[i + 1] - 1]; }
        if (rc == 0)
            for (int64_t j = use_ptr[i]; j + 1 < use_ptr[i + 1]; ++j) {
                int32_t u = uses[j], v = uses[j + 1];
                if (v - u >= 2) {
                    if (np < periods_cap) { period_tensor[np] = (int32_t)i; period_prev_use[np] = u; period_next_use[np] = v; }
                    np += 1;
                }
            }
        period_ptr[i + 1] = np;
    }
    counts[1] = np;
    if (np > periods_cap) rc = -1;
    free(seen); free(fill);
    return rc;
}

/* ------------------------------------------------------------------------------------------
 * GPU memory pressure before any migration (Section 4.3: "the total size of non-evicted tensors
 * in GPU memory at time T").  Written as the definition: every tensor adds its size to every
 * slot it is alive in.  An intermediate tensor lives from its birth to its death; a global
 * tensor (weights) is allocated at the start of the program and is never freed, so it lives in
 * every slot, provided the trace uses it at all.  peak_slot is the lowest slot holding the peak
 * (-1 when there are no slots).
 * ---------------------------------------------------------------------------------------- */
void g10o_pressure(int64_t K, int64_t N, const int64_t *tensor_bytes, const uint8_t *tensor_global,
                   const int32_t *first_use, const int32_t *last_use,
                   int64_t *pressure /* [K] */, int64_t *peak_bytes, int32_t *peak_slot)
{
    for (int64_t k = 0; k < K; ++k) pressure[k] = 0;
    for (int64_t i = 0; i < N; ++i) {
        if (first_use[i] < 0) continue;
        int64_t lo = first_use[i], hi = last_use[i];
        if (tensor_global && tensor_global[i]) { lo = 0; hi = K - 1; }
        for (int64_t k = lo; k <= hi; ++k) pressure[k] += tensor_bytes[i];
    }
    int64_t pk = 0; int32_t ps = -1;
    for (int64_t k = 0; k < K; ++k) if (ps < 0 || pressure[k] > pk) { pk = pressure[k]; ps = (int32_t)k; }
    *peak_bytes = pk; *peak_slot = ps;
}

/* ------------------------------------------------------------------------------------------
 * Candidate geometry for one period and one destination.
 * Transfer time t = ceil(bytes * 1e9 / bandwidth) ns (Algorithm 1: tensor_size / BW), the same in
 * both directions.  The eviction starts when the period starts, t_r = end of kernel u (Algorithm 1
 * schedules the pre-eviction at t_r) and occupies [t_r, t_r + t).  The prefetch is issued at the
 * latest safe prefetch time t_end - t (Section 4.4), t_end = start of kernel v, and occupies
 * [t_end - t, t_end).  The tensor counts as absent from GPU memory exactly in the slots that lie
 * wholly between the two windows: from a' = first slot starting at or after t_r + t, to
 * b' = the slot before the one in which the prefetch window begins.  Invalid (never a candidate)
 * when the two transfers do not fit into the period (2t > L) or no whole slot is left (a' > b').
 * ---------------------------------------------------------------------------------------- */
static int64_t transfer_ns(int64_t bytes, uint64_t bw)
{
    u128 num = (u128)(uint64_t)bytes * (u128)1000000000u;
    u128 q = num / bw;
    if (q * bw != num) q += 1;
    if (q > (u128)T_SATURATE) return T_SATURATE;
    return (int64_t)q;
}

typedef struct { int64_t t; int32_t a_abs, b_abs; int valid; } geo_t;

static geo_t geometry_one(int64_t K, const int64_t *start, int64_t bytes, int32_t u, int32_t v, uint64_t bw)
{
    geo_t g; g.valid = 0; g.a_abs = -1; g.b_abs = -2;
    g.t = transfer_ns(bytes, bw);
    int64_t t_r = start[u + 1], t_end = start[v];
    int64_t L = t_end - t_r;
    if (g.t > L || 2 * g.t > L) return g;                 /* (first test keeps 2t from overflowing) */
    int64_t ap = u + 1;                                   /* first k in [0,K] with start[k] >= t_r + t */
    while (ap <= K && start[ap] < t_r + g.t) ++ap;
    int64_t j = v;                                        /* last j in [0,K] with start[j] <= t_end - t */
    while (j >= 0 && start[j] > t_end - g.t) --j;
    int64_t bp = j - 1;
    if (ap > bp) return g;
    g.valid = 1; g.a_abs = (int32_t)ap; g.b_abs = (int32_t)bp;
    return g;
}

/* transfer_ns[X*Pn+p], absent_first[X*Pn+p], absent_last[X*Pn+p] for X = 0 (SSD), 1 (HOST);
   an invalid pair has absent_first = -1, absent_last = -2. */
void g10o_geometry(int64_t K, int64_t Pn, const int64_t *start, const int64_t *tensor_bytes,
                   const int32_t *period_tensor, const int32_t *period_prev_use, const int32_t *period_next_use,
                   uint64_t host_bw, uint64_t ssd_bw,
                   int64_t *out_transfer_ns, int32_t *out_absent_first, int32_t *out_absent_last)
{
    for (int X = 0; X < 2; ++X)
        for (int64_t p = 0; p < Pn; ++p) {
            geo_t g = geometry_one(K, start, tensor_bytes[period_tensor[p]], period_prev_use[p], period_next_use[p],
                                   X == DEST_SSD ? ssd_bw : host_bw);
            out_transfer_ns[X * Pn + p] = g.t;
            out_absent_first[X * Pn + p] = g.a_abs;
            out_absent_last[X * Pn + p] = g.b_abs;
        }
}

/* ------------------------------------------------------------------------------------------
 * Planner state and scoring (Section 4.3, Algorithm 1).
 * ---------------------------------------------------------------------------------------- */
typedef struct {
    int64_t K, Pn;
    const int64_t *start, *dur, *bytes;
    const int32_t *per_tensor, *per_u, *per_v;
    geo_t *geo[2];
    int64_t *P;            /* current pressure per slot                                  */
    int64_t *busy[4];      /* ns of each slot already given to a transfer, per channel   */
    int64_t *hocc;         /* bytes parked in host memory per slot                       */
    int64_t cap;
    uint64_t host_capacity;
} plan_state;

/* overlap of the time window [w0, w1) with slot k */
static int64_t overlap(const plan_state *S, int64_t w0, int64_t w1, int64_t k)
{
    int64_t lo = w0 > S->start[k] ? w0 : S->start[k];
    int64_t hi = w1 < S->start[k + 1] ? w1 : S->start[k + 1];
    return hi > lo ? hi - lo : 0;
}

/* Bandwidth budget (Algorithm 1 tests whether the link to a device is saturated for the duration
   of the transfer).  Reading: each slot offers dur[k] ns of channel time per device and direction; a
   transfer may be booked iff, in every slot its window touches, the time already booked plus the
   window's overlap with that slot stays within dur[k]. */
static int channel_free(const plan_state *S, int ch, int64_t w0, int64_t w1, int64_t k0, int64_t k1)
{
    for (int64_t k = k0; k <= k1; ++k)
        if (S->busy[ch][k] + overlap(S, w0, w1, k) > S->dur[k]) return 0;
    return 1;
}

static int admissible(const plan_state *S, int64_t p, int X)
{
    const geo_t *g = &S->geo[X][p];
    if (!g->valid) return 0;
    int64_t a = S->per_u[p] + 1, b = S->per_v[p] - 1;
    int64_t t_r = S->start[a], t_end = S->start[b + 1];
    int out = X == DEST_SSD ? CH_SSD_OUT : CH_HOST_OUT, in = X == DEST_SSD ? CH_SSD_IN : CH_HOST_IN;
    if (!channel_free(S, out, t_r, t_r + g->t, a, g->a_abs - 1)) return 0;
    if (!channel_free(S, in, t_end - g->t, t_end, g->b_abs + 1, b)) return 0;
    if (X == DEST_HOST && S->host_capacity != 0) {
        /* host-capacity test of Algorithm 1: the tensor occupies host memory for the whole period */
        uint64_t s = (uint64_t)S->bytes[S->per_tensor[p]];
        for (int64_t k = a; k <= b; ++k)
            if ((uint64_t)S->hocc[k] + s > S->host_capacity) return 0;
    }
    return 1;
}

/* Benefit of evicting during the period with destination X: the part of the pressure curve above
   the capacity line that disappears (the shaded area of the paper's state-transition figure),
   in byte*ns: sum over absent slots of min(size, excess) * dur. */
static u128 benefit_of(const plan_state *S, int64_t p, int X)
{
    const geo_t *g = &S->geo[X][p];
    int64_t s = S->bytes[S->per_tensor[p]];
    u128 acc = 0;
    for (int64_t k = g->a_abs; k <= g->b_abs; ++k) {
        int64_t ex = S->P[k] - S->cap;
        if (ex <= 0) continue;
        if (ex > s) ex = s;
        acc += (u128)(uint64_t)ex * (u128)(uint64_t)S->dur[k];
    }
    return acc;
}

/* Destination rule: SSD first (large capacity); host memory only when the SSD cannot take the
   transfer (its channel is saturated in the window, or the tensor cannot go out and come back
   within the period) and the host link and host memory can.  Returns -1 if neither works. */
static int choose_destination(const plan_state *S, int64_t p)
{
    if (admissible(S, p, DEST_SSD)) return DEST_SSD;
    if (admissible(S, p, DEST_HOST)) return DEST_HOST;
    return -1;
}

/* p beats q iff benefit_p / cost_p > benefit_q / cost_q, exact; ties go to the lower index */
static int beats(u128 bp, int64_t cp, int64_t ip, u128 bq, int64_t cq, int64_t iq)
{
    u128 l = bp * (u128)(uint64_t)cq, r = bq * (u128)(uint64_t)cp;
    if (l != r) return l > r;
    return ip < iq;
}

static void commit(plan_state *S, int64_t p, int X)
{
    const geo_t *g = &S->geo[X][p];
    int64_t s = S->bytes[S->per_tensor[p]];
    int64_t a = S->per_u[p] + 1, b = S->per_v[p] - 1;
    int64_t t_r = S->start[a], t_end = S->start[b + 1];
    int out = X == DEST_SSD ? CH_SSD_OUT : CH_HOST_OUT, in = X == DEST_SSD ? CH_SSD_IN : CH_HOST_IN;
    for (int64_t k = g->a_abs; k <= g->b_abs; ++k) S->P[k] -= s;
    for (int64_t k = a; k <= g->a_abs - 1; ++k) S->busy[out][k] += overlap(S, t_r, t_r + g->t, k);
    for (int64_t k = g->b_abs + 1; k <= b; ++k) S->busy[in][k] += overlap(S, t_end - g->t, t_end, k);
    if (X == DEST_HOST) for (int64_t k = a; k <= b; ++k) S->hocc[k] += s;
}

static void peak_of(const int64_t *P, int64_t K, int64_t *pk, int64_t *ps)
{
    *pk = 0; *ps = -1;
    for (int64_t k = 0; k < K; ++k) if (*ps < 0 || P[k] > *pk) { *pk = P[k]; *ps = k; }
}

/* ---- a binary max-heap of (bound ratio, index) for the lazy tier --------------------------- */
typedef struct { u128 ben; int64_t cost; int64_t idx; int64_t ver; } hnode;
static int hbeats(const hnode *x, const hnode *y) { return beats(x->ben, x->cost, x->idx, y->ben, y->cost, y->idx); }
static void hpush(hnode *h, int64_t *n, hnode v)
{
    int64_t i = (*n)++; h[i] = v;
    while (i > 0) { int64_t par = (i - 1) / 2; if (!hbeats(&h[i], &h[par])) break; hnode t = h[i]; h[i] = h[par]; h[par] = t; i = par; }
}
static hnode hpop(hnode *h, int64_t *n)
{
    hnode top = h[0]; h[0] = h[--(*n)];
    int64_t i = 0;
    for (;;) {
        int64_t l = 2 * i + 1, r = l + 1, m = i;
        if (l < *n && hbeats(&h[l], &h[m])) m = l;
        if (r < *n && hbeats(&h[r], &h[m])) m = r;
        if (m == i) break;
        hnode t = h[i]; h[i] = h[m]; h[m] = t; i = m;
    }
    return top;
}

/* Lazy tier.  Pressure only falls and booked channel time / host occupancy only rise, so for a
   fixed destination a period's ratio can only fall: the ratio computed earlier is an upper bound
   of the current one, as long as the period's destination is still the one the rule picks.  The
   destination is therefore kept exact: after every commit, each live period whose transfer
   windows (or, with a finite host memory, whose whole period) share a slot with what the commit
   booked on the same device is re-examined at once.  slots_meet tells whether two slot ranges
   intersect. */
static int slots_meet(int64_t a0, int64_t a1, int64_t b0, int64_t b1) { return a0 <= b1 && b0 <= a1 && a0 <= a1 && b0 <= b1; }

/* ------------------------------------------------------------------------------------------
 * The planner (Algorithm 1).  Each iteration: stop if the peak fits; score every live period;
 * take the best benefit/cost ratio; book it; erase the period.  Stops EXHAUSTED when no live
 * period has a positive benefit ("no more beneficial eviction candidates").
 *   lazy = 0 : the definition (every live period is rescored every iteration).
 *   lazy = 1 : same result, periods rescored only when their earlier score (an upper bound) is on
 *              top of a heap; destinations are kept exact after every commit.
 * win_benefit (optional, 2 words per record: low, high) and win_cost (optional) report the
 * winner's score for the invariant tests.
 * summary[8] = { migrations, scoring rounds, exit status, final peak, final peak slot,
 *                bytes to SSD, bytes to host, 0 }.
 * Returns 0, or -1 if out_cap is too small (summary[0] then holds the number needed).
 * ---------------------------------------------------------------------------------------- */
int32_t g10o_plan(int64_t K, int64_t N, const int64_t *kernel_ptr, const int32_t *kernel_tensors,
                  const int64_t *tensor_bytes, const int64_t *kernel_ns, const uint8_t *tensor_global,
                  uint64_t gpu_capacity_bytes, uint64_t host_bw, uint64_t ssd_bw,
                  uint64_t host_capacity_bytes, int64_t max_iterations, int32_t lazy,
                  g10o_migration *out, int64_t out_cap, int64_t *final_pressure /* [K] */,
                  int64_t *summary /* [8] */, uint64_t *win_benefit, int64_t *win_cost)
{
    int64_t E = K > 0 ? kernel_ptr[K] : 0;
    size_t nN = (size_t)(N > 0 ? N : 1), nK = (size_t)(K > 0 ? K : 1), nE = (size_t)(E > 0 ? E : 1);
    int64_t *start = (int64_t *)malloc(sizeof(int64_t) * (nK + 1));
    int32_t *first = (int32_t *)malloc(4 * nN), *last = (int32_t *)malloc(4 * nN), *nuse = (int32_t *)malloc(4 * nN);
    int64_t *use_ptr = (int64_t *)malloc(8 * (nN + 1)), *per_ptr = (int64_t *)malloc(8 * (nN + 1));
    int32_t *uses = (int32_t *)malloc(4 * nE);
    int32_t *pt = (int32_t *)malloc(4 * nE), *pu = (int32_t *)malloc(4 * nE), *pv = (int32_t *)malloc(4 * nE);
    int64_t counts[2];
    g10o_slot_clock(K, kernel_ns, start);
    g10o_vitality(K, N, kernel_ptr, kernel_tensors, first, last, nuse, use_ptr, uses, E, per_ptr, pt, pu, pv, E, counts);
    int64_t Pn = counts[1];
    int64_t pk; int32_t ps32;
    g10o_pressure(K, N, tensor_bytes, tensor_global, first, last, final_pressure, &pk, &ps32);

    plan_state S;
    S.K = K; S.Pn = Pn; S.start = start; S.dur = kernel_ns; S.bytes = tensor_bytes;
    S.per_tensor = pt; S.per_u = pu; S.per_v = pv; S.P = final_pressure;
    S.host_capacity = host_capacity_bytes;
    size_t nP = (size_t)(Pn > 0 ? Pn : 1);
    for (int X = 0; X < 2; ++X) {
        S.geo[X] = (geo_t *)malloc(sizeof(geo_t) * nP);
        for (int64_t p = 0; p < Pn; ++p)
            S.geo[X][p] = geometry_one(K, start, tensor_bytes[pt[p]], pu[p], pv[p], X == DEST_SSD ? ssd_bw : host_bw);
    }
    for (int c = 0; c < 4; ++c) S.busy[c] = (int64_t *)calloc(nK, 8);
    S.hocc = (int64_t *)calloc(nK, 8);
    char *alive = (char *)malloc(nP);
    memset(alive, 1, nP);

    int64_t limit = (max_iterations <= 0 || max_iterations > Pn) ? Pn : max_iterations;
    int64_t n_mig = 0, n_rounds = 0, status = -1, bytes_to[2] = {0, 0};
    int32_t rc = 0;
    /* a capacity of 2^63 or more can never be exceeded by an int64 pressure */
    int fits_always = gpu_capacity_bytes >= ((uint64_t)1 << 63);
    S.cap = fits_always ? INT64_MAX : (int64_t)gpu_capacity_bytes;

    hnode *heap = NULL, *popped = NULL; int64_t hn = 0;
    int *dest = NULL; int64_t *ver = NULL;
    if (lazy) {
        /* every period enters the heap once, plus once per change of destination (at most two) */
        heap = (hnode *)malloc(sizeof(hnode) * (3 * nP + 1));
        popped = (hnode *)malloc(sizeof(hnode) * (3 * nP + 1));
        dest = (int *)malloc(sizeof(int) * nP);
        ver = (int64_t *)calloc(nP, sizeof(int64_t));
        for (int64_t p = 0; p < Pn; ++p) {
            dest[p] = choose_destination(&S, p);
            if (dest[p] < 0) { alive[p] = 0; continue; }
            hnode nd; nd.idx = p; nd.ver = 0;
            nd.ben = benefit_of(&S, p, dest[p]); nd.cost = 2 * S.geo[dest[p]][p].t;
            if (nd.ben > 0) hpush(heap, &hn, nd);
        }
    }

    for (int64_t it = 0;; ++it) {
        int64_t cur_peak, cur_slot;
        peak_of(S.P, K, &cur_peak, &cur_slot);
        if (fits_always || cur_peak <= S.cap) { status = n_mig == 0 ? ST_ALREADY_FITS : ST_FIT; break; }
        if (it >= limit) { status = limit < Pn ? ST_ITERATION_LIMIT : ST_EXHAUSTED; break; }
        n_rounds += 1;
        int64_t best = -1; int bestX = -1; u128 bestB = 0; int64_t bestC = 1;
        if (!lazy) {
            for (int64_t p = 0; p < Pn; ++p) {
                if (!alive[p]) continue;
                int X = choose_destination(&S, p);
                if (X < 0) continue;
                u128 b = benefit_of(&S, p, X);
                if (b == 0) continue;
                int64_t c = 2 * S.geo[X][p].t;
                if (best < 0 || beats(b, c, p, bestB, bestC, best)) { best = p; bestX = X; bestB = b; bestC = c; }
            }
        } else {
            /* Pop while the top bound could still beat the best exact score seen this iteration;
               every popped period is rescored against the current state.  What stays in the heap
               has bound <= best, hence score <= best. */
            int64_t npop = 0;
            while (hn > 0 && (best < 0 || beats(heap[0].ben, heap[0].cost, heap[0].idx, bestB, bestC, best))) {
                hnode top = hpop(heap, &hn);
                int64_t p = top.idx;
                if (!alive[p] || top.ver != ver[p]) continue;          /* superseded entry */
                hnode nd; nd.idx = p; nd.ver = ver[p];
                nd.ben = benefit_of(&S, p, dest[p]); nd.cost = 2 * S.geo[dest[p]][p].t;
                if (nd.ben == 0) continue;            /* stays out until its destination changes */
                popped[npop++] = nd;
                if (best < 0 || beats(nd.ben, nd.cost, p, bestB, bestC, best)) { best = p; bestX = dest[p]; bestB = nd.ben; bestC = nd.cost; }
            }
            for (int64_t j = 0; j < npop; ++j) if (popped[j].idx != best) hpush(heap, &hn, popped[j]);
        }
        if (best < 0) { status = ST_EXHAUSTED; break; }
        if (n_mig < out_cap) {
            const geo_t *g = &S.geo[bestX][best];
            g10o_migration *m = &out[n_mig];
            m->period = (int32_t)best; m->tensor = pt[best]; m->dest = bestX;
            m->absent_first = g->a_abs; m->absent_last = g->b_abs; m->iteration = (int32_t)it;
            m->evict_issue_ns = start[pu[best] + 1]; m->prefetch_issue_ns = start[pv[best]] - g->t; m->transfer_ns = g->t;
            if (win_benefit) { win_benefit[2 * n_mig] = (uint64_t)bestB; win_benefit[2 * n_mig + 1] = (uint64_t)(bestB >> 64); }
            if (win_cost) win_cost[n_mig] = bestC;
        } else rc = -1;
        commit(&S, best, bestX);
        alive[best] = 0;
        if (lazy) {
            /* keep every destination exact: re-examine the periods the new bookings can affect */
            const geo_t *gw = &S.geo[bestX][best];
            int64_t aw = pu[best] + 1, bw = pv[best] - 1;
            for (int64_t p = 0; p < Pn; ++p) {
                if (!alive[p] || dest[p] != bestX) continue;
                const geo_t *gp = &S.geo[bestX][p];
                int64_t ap_ = pu[p] + 1, bp_ = pv[p] - 1;
                int hit = slots_meet(ap_, gp->a_abs - 1, aw, gw->a_abs - 1) || slots_meet(gp->b_abs + 1, bp_, gw->b_abs + 1, bw);
                if (!hit && bestX == DEST_HOST && S.host_capacity != 0) hit = slots_meet(ap_, bp_, aw, bw);
                if (!hit) continue;
                int nd_ = choose_destination(&S, p);
                if (nd_ == dest[p]) continue;
                dest[p] = nd_; ver[p] += 1;
                if (nd_ < 0) { alive[p] = 0; continue; }
                hnode nn; nn.idx = p; nn.ver = ver[p];
                nn.ben = benefit_of(&S, p, nd_); nn.cost = 2 * S.geo[nd_][p].t;
                if (nn.ben > 0) hpush(heap, &hn, nn);
            }
        }
        bytes_to[bestX] += tensor_bytes[pt[best]];
        n_mig += 1;
    }
    int64_t fpk, fps;
    peak_of(S.P, K, &fpk, &fps);
    summary[0] = n_mig; summary[1] = n_rounds; summary[2] = status; summary[3] = fpk; summary[4] = fps;
    summary[5] = bytes_to[DEST_SSD]; summary[6] = bytes_to[DEST_HOST]; summary[7] = 0;

    free(start); free(first); free(last); free(nuse); free(use_ptr); free(per_ptr); free(uses);
    free(pt); free(pu); free(pv); free(S.geo[0]); free(S.geo[1]);
    for (int c = 0; c < 4; ++c) free(S.busy[c]);
    free(S.hocc); free(alive); free(heap); free(popped); free(dest); free(ver);
    return rc;
}

/* ------------------------------------------------------------------------------------------
 * Steady-state (cyclic) planning.  Section 4.2 notes that the inactive period of a global tensor (a
 * weight) may span two consecutive training iterations.  Readings taken here:
 *   (1) the traced iteration repeats unchanged, so the timeline is a cycle of K slots of length T =
 *       sum of the durations; slot k of the next iteration is slot k again.  Unrolled index k + K
 *       names slot k one iteration later, unrolled time start[k] + T;
 *   (2) every global tensor that is used has, besides its periods inside the iteration, one more
 *       inactive period from its last use to its first use in the next iteration, (i, last, first + K),
 *       provided at least one slot lies in between (first + K - last >= 2).  These wrap-around periods
 *       are numbered after the ordinary ones, by tensor id;
 *   (3) geometry, admissibility, benefit and commit are those of the ordinary planner on the unrolled
 *       clock; pressure, channel bookings and host occupancy belong to the physical slot k mod K (a
 *       wrap-around period covers at most K - 1 slots, so no slot is met twice);
 *   (4) records carry unrolled slot indices and times (absent_last and the prefetch time of a
 *       wrap-around period may lie in the next iteration).
 * Plain tier only (every live period rescored every iteration).  periods_out (optional, 3 * (E + N)
 * ints) receives the period list used: tensor, prev use, next use (unrolled).
 * ---------------------------------------------------------------------------------------- */
typedef struct {
    int64_t K, Pn;
    const int64_t *start2;          /* [2K + 1] unrolled clock */
    const int64_t *dur, *bytes;
    const int32_t *per_tensor, *per_u, *per_v;
    geo_t *geo[2];
    int64_t *P, *busy[4], *hocc;
    int64_t cap;
    uint64_t host_capacity;
} cyc_state;

static int64_t cyc_overlap(const cyc_state *S, int64_t w0, int64_t w1, int64_t k)      /* k unrolled */
{
    int64_t lo = w0 > S->start2[k] ? w0 : S->start2[k];
    int64_t hi = w1 < S->start2[k + 1] ? w1 : S->start2[k + 1];
    return hi > lo ? hi - lo : 0;
}

static int cyc_channel_free(const cyc_state *S, int ch, int64_t w0, int64_t w1, int64_t k0, int64_t k1)
{
    for (int64_t k = k0; k <= k1; ++k)
        if (S->busy[ch][k % S->K] + cyc_overlap(S, w0, w1, k) > S->dur[k % S->K]) return 0;
    return 1;
}

static int cyc_admissible(const cyc_state *S, int64_t p, int X)
{
    const geo_t *g = &S->geo[X][p];
    if (!g->valid) return 0;
    int64_t a = S->per_u[p] + 1, b = S->per_v[p] - 1;
    int64_t t_r = S->start2[a], t_end = S->start2[b + 1];
    int out = X == DEST_SSD ? CH_SSD_OUT : CH_HOST_OUT, in = X == DEST_SSD ? CH_SSD_IN : CH_HOST_IN;
    if (!cyc_channel_free(S, out, t_r, t_r + g->t, a, g->a_abs - 1)) return 0;
    if (!cyc_channel_free(S, in, t_end - g->t, t_end, g->b_abs + 1, b)) return 0;
    if (X == DEST_HOST && S->host_capacity != 0) {
        uint64_t s = (uint64_t)S->bytes[S->per_tensor[p]];
        for (int64_t k = a; k <= b; ++k)
            if ((uint64_t)S->hocc[k % S->K] + s > S->host_capacity) return 0;
    }
    return 1;
}

int32_t g10o_plan_cyclic(int64_t K, int64_t N, const int64_t *kernel_ptr, const int32_t *kernel_tensors,
                         const int64_t *tensor_bytes, const int64_t *kernel_ns, const uint8_t *tensor_global,
                         uint64_t gpu_capacity_bytes, uint64_t host_bw, uint64_t ssd_bw,
                         uint64_t host_capacity_bytes, int64_t max_iterations,
                         g10o_migration *out, int64_t out_cap, int64_t *final_pressure /* [K] */,
                         int64_t *summary /* [8] */, int32_t *periods_out, int64_t *num_periods_out)
{
    int64_t E = K > 0 ? kernel_ptr[K] : 0;
    size_t nN = (size_t)(N > 0 ? N : 1), nK = (size_t)(K > 0 ? K : 1), nE = (size_t)(E + N > 0 ? E + N : 1);
    int64_t *start = (int64_t *)malloc(8 * (nK + 1)), *start2 = (int64_t *)malloc(8 * (2 * nK + 1));
    int32_t *first = (int32_t *)malloc(4 * nN), *last = (int32_t *)malloc(4 * nN), *nuse = (int32_t *)malloc(4 * nN);
    int64_t *use_ptr = (int64_t *)malloc(8 * (nN + 1)), *per_ptr = (int64_t *)malloc(8 * (nN + 1));
    int32_t *uses = (int32_t *)malloc(4 * nE);
    int32_t *pt = (int32_t *)malloc(4 * nE), *pu = (int32_t *)malloc(4 * nE), *pv = (int32_t *)malloc(4 * nE);
    int64_t counts[2];
    g10o_slot_clock(K, kernel_ns, start);
    for (int64_t k = 0; k <= 2 * K; ++k) start2[k] = k <= K ? start[k] : start[k - K] + start[K];
    g10o_vitality(K, N, kernel_ptr, kernel_tensors, first, last, nuse, use_ptr, uses, E, per_ptr, pt, pu, pv, E, counts);
    int64_t Pn = counts[1];
    for (int64_t i = 0; i < N; ++i)                      /* the wrap-around periods of the global tensors */
        if (tensor_global && tensor_global[i] && first[i] >= 0 && first[i] + K - last[i] >= 2) {
            pt[Pn] = (int32_t)i; pu[Pn] = last[i]; pv[Pn] = (int32_t)(first[i] + K); Pn += 1;
        }
    int64_t pk; int32_t ps32;
    g10o_pressure(K, N, tensor_bytes, tensor_global, first, last, final_pressure, &pk, &ps32);

    cyc_state S;
    S.K = K; S.Pn = Pn; S.start2 = start2; S.dur = kernel_ns; S.bytes = tensor_bytes;
    S.per_tensor = pt; S.per_u = pu; S.per_v = pv; S.P = final_pressure; S.host_capacity = host_capacity_bytes;
    size_t nP = (size_t)(Pn > 0 ? Pn : 1);
    for (int X = 0; X < 2; ++X) {
        S.geo[X] = (geo_t *)malloc(sizeof(geo_t) * nP);
        for (int64_t p = 0; p < Pn; ++p)
            S.geo[X][p] = geometry_one(2 * K, start2, tensor_bytes[pt[p]], pu[p], pv[p], X == DEST_SSD ? ssd_bw : host_bw);
    }
    for (int c = 0; c < 4; ++c) S.busy[c] = (int64_t *)calloc(nK, 8);
    S.hocc = (int64_t *)calloc(nK, 8);
    unsigned char *alive = (unsigned char *)malloc(nP);
    for (int64_t p = 0; p < Pn; ++p) alive[p] = 1;
    int fits_always = gpu_capacity_bytes >= ((uint64_t)1 << 63);
    S.cap = fits_always ? INT64_MAX : (int64_t)gpu_capacity_bytes;
    int64_t limit = (max_iterations <= 0 || max_iterations > Pn) ? Pn : max_iterations;
    int64_t n_mig = 0, n_rounds = 0, status = -1, bytes_to[2] = {0, 0};
    int32_t rc = 0;
    for (int64_t it = 0;; ++it) {
        int64_t cur_peak, cur_slot;
        peak_of(S.P, K, &cur_peak, &cur_slot);
        if (fits_always || cur_peak <= S.cap) { status = n_mig == 0 ? ST_ALREADY_FITS : ST_FIT; break; }
        if (it >= limit) { status = limit < Pn ? ST_ITERATION_LIMIT : ST_EXHAUSTED; break; }
        n_rounds += 1;
        int64_t best = -1; int bestX = -1; u128 bestB = 0; int64_t bestC = 1;
        for (int64_t p = 0; p < Pn; ++p) {
            if (!alive[p]) continue;
            int X = cyc_admissible(&S, p, DEST_SSD) ? DEST_SSD : (cyc_admissible(&S, p, DEST_HOST) ? DEST_HOST : -1);
            if (X < 0) continue;
            const geo_t *g = &S.geo[X][p];
            int64_t s = tensor_bytes[pt[p]];
            u128 b = 0;
            for (int64_t k = g->a_abs; k <= g->b_abs; ++k) {
                int64_t ex = S.P[k % K] - S.cap;
                if (ex <= 0) continue;
                if (ex > s) ex = s;
                b += (u128)(uint64_t)ex * (u128)(uint64_t)kernel_ns[k % K];
            }
            if (b == 0) continue;
            int64_t c = 2 * g->t;
            if (best < 0 || beats(b, c, p, bestB, bestC, best)) { best = p; bestX = X; bestB = b; bestC = c; }
        }
        if (best < 0) { status = ST_EXHAUSTED; break; }
        const geo_t *g = &S.geo[bestX][best];
        int64_t s = tensor_bytes[pt[best]];
        int64_t a = pu[best] + 1, b = pv[best] - 1;
        int64_t t_r = start2[a], t_end = start2[b + 1];
        if (n_mig < out_cap) {
            g10o_migration *m = &out[n_mig];
            m->period = (int32_t)best; m->tensor = pt[best]; m->dest = bestX;
            m->absent_first = g->a_abs; m->absent_last = g->b_abs; m->iteration = (int32_t)it;
            m->evict_issue_ns = t_r; m->prefetch_issue_ns = t_end - g->t; m->transfer_ns = g->t;
        } else rc = -1;
        int outc = bestX == DEST_SSD ? CH_SSD_OUT : CH_HOST_OUT, inc = bestX == DEST_SSD ? CH_SSD_IN : CH_HOST_IN;
        for (int64_t k = g->a_abs; k <= g->b_abs; ++k) S.P[k % K] -= s;
        for (int64_t k = a; k <= g->a_abs - 1; ++k) S.busy[outc][k % K] += cyc_overlap(&S, t_r, t_r + g->t, k);
        for (int64_t k = g->b_abs + 1; k <= b; ++k) S.busy[inc][k % K] += cyc_overlap(&S, t_end - g->t, t_end, k);
        if (bestX == DEST_HOST) for (int64_t k = a; k <= b; ++k) S.hocc[k % K] += s;
        alive[best] = 0;
        bytes_to[bestX] += s;
        n_mig += 1;
    }
    int64_t fpk, fps;
    peak_of(S.P, K, &fpk, &fps);
    summary[0] = n_mig; summary[1] = n_rounds; summary[2] = status; summary[3] = fpk; summary[4] = fps;
    summary[5] = bytes_to[DEST_SSD]; summary[6] = bytes_to[DEST_HOST]; summary[7] = 0;
    if (periods_out) for (int64_t p = 0; p < Pn; ++p) { periods_out[3 * p] = pt[p]; periods_out[3 * p + 1] = pu[p]; periods_out[3 * p + 2] = pv[p]; }
    if (num_periods_out) *num_periods_out = Pn;
    free(start); free(start2); free(first); free(last); free(nuse); free(use_ptr); free(per_ptr); free(uses);
    free(pt); free(pu); free(pv); free(S.geo[0]); free(S.geo[1]);
    for (int c = 0; c < 4; ++c) free(S.busy[c]);
    free(S.hocc); free(alive);
    return rc;
}

/* ------------------------------------------------------------------------------------------
 * Smart tensor prefetching (Section 4.4).  The eviction loop above assumes every prefetch at its
 * latest safe prefetch time.  Afterwards the evicted periods are sorted by that time and visited in
 * order; for each one the search goes backward from the latest safe prefetch time to the earliest
 * time at which the GPU can hold the whole tensor with the space that is left, the prefetch is
 * rescheduled there and the pressure curve in between is updated.
 * Readings: (1) whole-slot granularity as in the eviction loop -- the tensor becomes resident again
 * in whole slots, so the search walks slot by slot from absent_last downwards while pressure + size
 * stays within capacity, never past absent_first; (2) ties in the sort go to the earlier plan
 * record; (3) only memory is examined, as the section says -- channel bookings are not revisited;
 * (4) a prefetch that moves is issued at the start of the first slot in which the tensor is resident
 * again; one that cannot move keeps its time.
 * Plans of the steady-state planner (g10o_plan_cyclic) are accepted too.  Readings for them: (5) their
 * records carry unrolled slots and times (reading (4) there); the pressure curve belongs to the physical
 * slots, so slot x stands for slot x mod K, and a prefetch that moves is issued at the unrolled time of
 * its first regained slot; (6) on the cycle no prefetch comes "first": the visiting order is that of the
 * position inside the iteration, i.e. of the latest safe prefetch time modulo the iteration's length T.
 * For an ordinary plan every slot is below K and every time below T, and nothing changes.
 * order[i] = plan record visited i-th; new_absent_last / new_issue_ns are indexed by plan record.
 * summary[4] = { prefetches moved, slots regained in total, peak pressure after, its lowest slot }.
 * ---------------------------------------------------------------------------------------- */
void g10o_schedule_prefetch(int64_t K, int64_t n, const g10o_migration *mig, const int64_t *start,
                            const int64_t *tensor_bytes, uint64_t gpu_capacity_bytes, int64_t *pressure /* [K] in/out */,
                            int32_t *order, int32_t *new_absent_last, int64_t *new_issue_ns, int64_t *summary)
{
    int64_t cap = gpu_capacity_bytes >= ((uint64_t)1 << 63) ? INT64_MAX : (int64_t)gpu_capacity_bytes;
    const int64_t T = K > 0 ? start[K] : 1;
    for (int64_t i = 0; i < n; ++i) order[i] = (int32_t)i;
    /* insertion sort by (latest safe prefetch time inside the iteration, record): plain and stable */
    for (int64_t i = 1; i < n; ++i) {
        int32_t x = order[i];
        int64_t j = i - 1;
        while (j >= 0 && (mig[order[j]].prefetch_issue_ns % T > mig[x].prefetch_issue_ns % T)) { order[j + 1] = order[j]; --j; }
        order[j + 1] = x;
    }
    int64_t moved = 0, regained = 0;
    for (int64_t i = 0; i < n; ++i) {
        const g10o_migration *m = &mig[order[i]];
        int64_t s = tensor_bytes[m->tensor];
        int64_t j = m->absent_last;
        while (j >= m->absent_first && pressure[j % K] <= cap - s) --j;  /* pressure + s <= cap, without overflow */
        for (int64_t k = j + 1; k <= m->absent_last; ++k) pressure[k % K] += s;
        new_absent_last[order[i]] = (int32_t)j;
        const int64_t first = j + 1;                                     /* first regained slot, unrolled */
        new_issue_ns[order[i]] = j < m->absent_last ? (first <= K ? start[first] : start[first - K] + T) : m->prefetch_issue_ns;
        if (j < m->absent_last) { moved += 1; regained += m->absent_last - j; }
    }
    int64_t pk, ps;
    peak_of(pressure, K, &pk, &ps);
    summary[0] = moved; summary[1] = regained; summary[2] = pk; summary[3] = ps;
}

/* ------------------------------------------------------------------------------------------
 * Code instrumentation (Section 4.4; the instrumented program of Figure 9): the list of
 * g10_alloc / g10_free / g10_pre_evict / g10_prefetch calls inserted between the kernels.
 * Boundary b (0 <= b <= K) is the gap before kernel b (b = K: after the last kernel).
 *   ALLOC     before the first kernel that uses the tensor; a global tensor (weights) is allocated
 *             at the beginning of the program: boundary 0.  (Figure 9: g10_alloc before Kernel 3.)
 *   FREE      right after the last kernel that uses an intermediate tensor: boundary last + 1;
 *             global tensors are never freed.  (Figure 9: g10_free right after Kernel 4.)
 *   PRE_EVICT at the start of the inactive period, t_r: the boundary whose time is t_r.
 *   PREFETCH  at its issue time; an instruction can only sit between kernels, so it goes to the
 *             last boundary at or before that time (earlier is safe, later is not).
 * Within one boundary the order is FREE, PRE_EVICT (tidy up after the previous kernel), ALLOC,
 * PREFETCH (get ready for the next), as in Figure 9; then by tensor id.  A tensor never has two
 * instructions of the same kind at one boundary, so the order is total.
 * new_issue_ns (optional): prefetch times from the eager prefetch pass, indexed by plan record.
 * A plan of the steady-state planner is accepted too: the stream is that of one iteration of the cycle, and a
 * prefetch whose time lies in the next iteration (a wrap-around period's) stands where the program is at
 * that moment of every iteration: its time is taken modulo the iteration's length, and so is its boundary.
 * Returns the number of instructions (records beyond out_cap are not written).
 * ---------------------------------------------------------------------------------------- */
enum { OP_FREE = 0, OP_PRE_EVICT = 1, OP_ALLOC = 2, OP_PREFETCH = 3 };

typedef struct {
    int32_t opcode, tensor, target, record;     /* target: destination of a pre-eviction, else -1; record: plan record, else -1 */
    int64_t bytes, time_ns;
} g10o_instruction;

typedef struct { int64_t boundary; g10o_instruction ins; } keyed_ins;

static int cmp_keyed(const void *x, const void *y)
{
    const keyed_ins *a = (const keyed_ins *)x, *b = (const keyed_ins *)y;
    if (a->boundary != b->boundary) return a->boundary < b->boundary ? -1 : 1;
    if (a->ins.opcode != b->ins.opcode) return a->ins.opcode < b->ins.opcode ? -1 : 1;
    if (a->ins.tensor != b->ins.tensor) return a->ins.tensor < b->ins.tensor ? -1 : 1;
    return 0;
}

int64_t g10o_emit_instructions(int64_t K, int64_t N, const int32_t *first_use, const int32_t *last_use,
                               const int64_t *tensor_bytes, const uint8_t *tensor_global, const int64_t *start,
                               int64_t n, const g10o_migration *mig, const int64_t *new_issue_ns,
                               int64_t *inst_ptr /* [K+2] */, g10o_instruction *out, int64_t out_cap)
{
    keyed_ins *list = (keyed_ins *)malloc(sizeof(keyed_ins) * (size_t)(2 * N + 2 * n + 1));
    int64_t m = 0;
    for (int64_t i = 0; i < N; ++i) {
        if (first_use[i] < 0) continue;
        int glob = tensor_global && tensor_global[i];
        keyed_ins a; a.boundary = glob ? 0 : first_use[i];
        a.ins.opcode = OP_ALLOC; a.ins.tensor = (int32_t)i; a.ins.target = -1; a.ins.record = -1;
        a.ins.bytes = tensor_bytes[i]; a.ins.time_ns = start[a.boundary];
        list[m++] = a;
        if (!glob) {
            keyed_ins f = a; f.boundary = (int64_t)last_use[i] + 1; f.ins.opcode = OP_FREE; f.ins.time_ns = start[f.boundary];
            list[m++] = f;
        }
    }
    for (int64_t r = 0; r < n; ++r) {
        keyed_ins e;
        int64_t b = 0;
        while (start[b] < mig[r].evict_issue_ns) ++b;            /* the boundary whose time is t_r */
        e.boundary = b; e.ins.opcode = OP_PRE_EVICT; e.ins.tensor = mig[r].tensor; e.ins.target = mig[r].dest;
        e.ins.record = (int32_t)r; e.ins.bytes = tensor_bytes[mig[r].tensor]; e.ins.time_ns = mig[r].evict_issue_ns;
        list[m++] = e;
        keyed_ins p = e;
        int64_t t = new_issue_ns ? new_issue_ns[r] : mig[r].prefetch_issue_ns;
        if (t >= start[K]) t -= start[K];                        /* (steady-state plans only: a time in the next iteration) */
        b = K;
        while (start[b] > t) --b;                                /* last boundary at or before the issue time */
        p.boundary = b; p.ins.opcode = OP_PREFETCH; p.ins.target = -1; p.ins.time_ns = t;
        list[m++] = p;
    }
    qsort(list, (size_t)m, sizeof(keyed_ins), cmp_keyed);
    int64_t j = 0;
    for (int64_t b = 0; b <= K; ++b) {
        inst_ptr[b] = j;
        while (j < m && list[j].boundary == b) { if (j < out_cap) out[j] = list[j].ins; ++j; }
    }
    inst_ptr[K + 1] = m;
    free(list);
    return m;
}

/* ------------------------------------------------------------------------------------------
 * Workload characterisation (Section 3): the statistics behind the paper's Figures 2-4, on a trace.
 *   active_bytes[k]   memory of the tensors kernel k uses (inputs and outputs, each once): the "active
 *                     tensors" of Figure 2; also the working set that must fit while kernel k runs.
 *   len_hist[b]       number of inactive periods whose length L = start[v] - start[u+1] (ns) has
 *                     floor(log2 L) = b: the distribution of Figure 3.
 *   size_len_hist     [41][45] periods by floor(log2 size) x floor(log2 L): the scatter of Figure 4.
 *   hide[2]           periods long enough to swap the tensor out and back in, 2 t <= L, over the SSD
 *                     and over the host link (Section 3: most periods can hide the swap latency).
 * ---------------------------------------------------------------------------------------- */
static int floor_log2_i64(int64_t x) { int b = 0; while (x > 1) { x >>= 1; ++b; } return b; }

void g10o_characterize(int64_t K, int64_t N, const int64_t *use_ptr, const int32_t *uses, const int64_t *tensor_bytes,
                       const int64_t *start, int64_t Pn, const int32_t *period_tensor, const int32_t *period_prev_use,
                       const int32_t *period_next_use, uint64_t host_bw, uint64_t ssd_bw,
                       int64_t *active_bytes /* [K] */, int64_t *len_hist /* [64] */, int64_t *size_len_hist /* [41*45] */,
                       int64_t *hide /* [2] */, int64_t *summary /* [2]: max active bytes, its lowest kernel */)
{
    for (int64_t k = 0; k < K; ++k) active_bytes[k] = 0;
    for (int64_t i = 0; i < N; ++i)
        for (int64_t j = use_ptr[i]; j < use_ptr[i + 1]; ++j) active_bytes[uses[j]] += tensor_bytes[i];
    for (int b = 0; b < 64; ++b) len_hist[b] = 0;
    for (int b = 0; b < 41 * 45; ++b) size_len_hist[b] = 0;
    hide[0] = hide[1] = 0;
    for (int64_t p = 0; p < Pn; ++p) {
        int64_t L = start[period_next_use[p]] - start[period_prev_use[p] + 1];
        int64_t s = tensor_bytes[period_tensor[p]];
        int bl = floor_log2_i64(L), bs = floor_log2_i64(s);
        len_hist[bl] += 1;
        size_len_hist[(bs > 40 ? 40 : bs) * 45 + (bl > 44 ? 44 : bl)] += 1;
        if (transfer_ns(s, ssd_bw) <= L / 2) hide[0] += 1;     /* 2 t <= L without overflow */
        if (transfer_ns(s, host_bw) <= L / 2) hide[1] += 1;
    }
    int64_t mx = 0, arg = -1;
    for (int64_t k = 0; k < K; ++k) if (arg < 0 || active_bytes[k] > mx) { mx = active_bytes[k]; arg = k; }
    summary[0] = mx; summary[1] = arg;
}

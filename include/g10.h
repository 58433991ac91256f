/*
 * g10.h -- C ABI of the B200-native planner for G10's compile-time tensor-migration analysis
 * (G10, MICRO '23: tensor vitality analysis, Section 4.2; GPU memory pressure and the smart tensor
 * eviction loop, Section 4.3 and Algorithm 1; latest safe prefetch time, Section 4.4).
 *
 * Conventions
 *   - All integers little-endian, all arrays contiguous.  Slots are kernels in trace order; slot k
 *     occupies the time [start[k], start[k+1]) ns, start being the prefix sum of kernel_ns.
 *   - Memory space: trace.mem says where EVERY array named by the trace and by the output struct of
 *     the same call lives.  G10_MEM_DEVICE: device pointers, the call only enqueues work on `stream`
 *     and returns; results are valid once the caller has synchronised the stream.  G10_MEM_HOST: host
 *     pointers (pinned memory recommended); the library stages the inputs into the workspace with
 *     cudaMemcpyAsync, runs the same kernels and copies the outputs back on the same stream; results
 *     are valid once the stream has been synchronised.
 *   - Ownership: the caller owns every buffer, the workspace and the stream.  The library allocates
 *     no device memory, keeps no state between calls and frees nothing.  The workspace `ws` is ALWAYS
 *     device memory, 256-byte aligned, of at least g10_workspace_bytes(...) bytes; its contents are
 *     scratch.  Two calls may run concurrently only on different workspaces.
 *   - Stream capture: a G10_MEM_DEVICE call of g10_vitality, g10_pressure_timeline, g10_candidate_geometry,
 *     g10_characterize or g10_emit_instructions enqueues only kernels and memsets (with programmatic
 *     dependencies between them) and may be captured in a CUDA graph, after one ordinary call of the same
 *     entry point (which sets kernel attributes).  The planner calls launch cooperative kernels and
 *     g10_plan_batch may synchronise: they are not meant for capture.
 *   - Errors: the return value is 0 (enqueued) or a negative G10_ERR_* found on the host before any
 *     launch.  Errors that depend on the data (tensor id out of range, non-monotone kernel_ptr,
 *     sizes or durations outside their limits, an output array too small, a grid barrier that timed
 *     out) are reported in a device status word (`counts[2]`, `summary[7]`, `*status`); outputs are
 *     then unspecified but every access stays in bounds.  FIT / EXHAUSTED / ALREADY_FITS are results,
 *     not errors.
 *   - Limits: 0 <= K, N, E < 2^31 - 1; 1 <= tensor_bytes < 2^40; kernel_ns >= 1; sum(kernel_ns) < 2^44.
 *     They make every benefit fit 84 bits and every benefit x cost product fit 128 bits.
 */
#ifndef G10_H_
#define G10_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define G10_VERSION 1

#define G10_MEM_DEVICE 0
#define G10_MEM_HOST 1

/* host-side return codes */
#define G10_OK 0
#define G10_ERR_ARG (-1)        /* NULL pointer, negative size, zero bandwidth, unknown enum       */
#define G10_ERR_LIMIT (-2)      /* K, N or E beyond the limits above                               */
#define G10_ERR_WORKSPACE (-3)  /* workspace NULL, misaligned or too small                         */
#define G10_ERR_CUDA (-4)       /* a CUDA runtime call failed (launch, copy, attribute query)      */

/* bits of the device status word (0 = no error) */
#define G10_DEV_BAD_TENSOR_ID 0x1    /* kernel_tensors entry outside [0, N)                       */
#define G10_DEV_BAD_KERNEL_PTR 0x2   /* kernel_ptr not nondecreasing from 0 to E                  */
#define G10_DEV_BAD_BYTES 0x4        /* tensor_bytes outside [1, 2^40)                            */
#define G10_DEV_BAD_DURATION 0x8     /* kernel_ns < 1 or sum >= 2^44                              */
#define G10_DEV_USES_OVERFLOW 0x10   /* uses_cap too small (counts[0] holds the need)             */
#define G10_DEV_PERIODS_OVERFLOW 0x20 /* periods_cap too small (counts[1] holds the need)         */
#define G10_DEV_PLAN_OVERFLOW 0x40   /* migrations_cap too small (summary[0] holds the need)      */
#define G10_DEV_TIMEOUT 0x80         /* an internal wait gave up; the kernel returned early       */
#define G10_DEV_BAD_FIRST_LAST 0x200 /* first_use / last_use handed to g10_pressure_timeline: last < first or last >= K (tensor skipped) */
#define G10_DEV_BATCH_UNFIT 0x100    /* internal: the trace does not fit one SM (g10_plan_batch then plans the variants one by one) */

/* exit status of the planner (summary[2]) */
#define G10_ALREADY_FITS 0      /* unplanned peak pressure <= capacity, empty plan                 */
#define G10_FIT 1               /* peak pressure brought down to <= capacity                       */
#define G10_EXHAUSTED 2         /* no remaining inactive period relieves any pressure above capacity */
#define G10_ITERATION_LIMIT 3   /* options.max_iterations reached first                            */

#define G10_DEST_SSD 0
#define G10_DEST_HOST 1

/* The kernel execution trace (Section 4.2; the instrumented program of Figure 9 shows its shape:
   an ordered list of kernels, each with its tensor arguments; a tensor may appear twice in one
   kernel, as the in-place ReLU does). CSR: kernel k lists kernel_tensors[kernel_ptr[k] .. kernel_ptr[k+1]). */
typedef struct g10_trace {
    int64_t num_kernels;            /* K                                                            */
    int64_t num_tensors;            /* N                                                            */
    int64_t num_events;             /* E = kernel_ptr[K]                                            */
    const int64_t *kernel_ptr;      /* [K+1]                                                        */
    const int32_t *kernel_tensors;  /* [E]                                                          */
    const int64_t *tensor_bytes;    /* [N]                                                          */
    const int64_t *kernel_ns;       /* [K] profiled execution time of each kernel                   */
    const uint8_t *tensor_global;   /* [N] 1 = global tensor (weights: allocated at program start,
                                       never freed), 0 = intermediate; NULL = all intermediate      */
    int32_t mem;                    /* G10_MEM_DEVICE or G10_MEM_HOST                               */
} g10_trace;

/* Tensor vitality (Section 4.2).  uses: per tensor the sorted distinct kernels that list it
   (use_ptr CSR).  A tensor is born at its first use and dead after its last (-1 / -1 / 0 uses if the
   trace never lists it).  One inactive period (tensor, prev_use u, next_use v) for every two
   consecutive uses with v - u >= 2; periods are ordered by (tensor, u); period_ptr is the CSR by tensor. */
typedef struct g10_vitality_out {
    int32_t *first_use, *last_use, *num_uses;   /* [N]                                              */
    int64_t *use_ptr;                           /* [N+1]                                            */
    int32_t *uses;                              /* [uses_cap]   (E always suffices)                 */
    int64_t uses_cap;
    int64_t *period_ptr;                        /* [N+1]                                            */
    int32_t *period_tensor, *period_prev_use, *period_next_use;   /* [periods_cap] (E always suffices) */
    int64_t periods_cap;
    int64_t *counts;                            /* [3]: number of uses E', number of periods Pn, device status word */
    /* Optional (NULL = no): the memory-pressure timeline of the same trace from the same call (workspace
       G10_WS_ANALYSIS; with a host trace the trace is staged once for both).  The kernel that writes first / last use books every tensor's size
       on the way, so that S1 - S3 walk the events once and only the slot clock and the pressure scan are
       left.  Its first_use / last_use inputs must be NULL; its outputs and status word are those of
       g10_pressure_timeline. */
    struct g10_timeline_out *timeline;
} g10_vitality_out;

/* Memory-pressure timeline (Section 4.3: pressure = total size of the tensors resident in GPU memory
   at a time).  pressure[k] = bytes alive during slot k before any migration: an intermediate tensor
   from first to last use, a global tensor in every slot if it is used at all. */
typedef struct g10_timeline_out {
    int64_t *kernel_start_ns;   /* [K+1] exclusive prefix sum of kernel_ns                          */
    int64_t *pressure;          /* [K]                                                              */
    int64_t *peak_bytes;        /* [1] max pressure (0 if K = 0)                                    */
    int32_t *peak_slot;         /* [1] lowest slot attaining it (-1 if K = 0)                       */
    int64_t *status;            /* [1] device status word                                           */
    /* Optional INPUTS (both or neither; device traces only): first / last use of every tensor as
       g10_vitality returned them ([N], -1 = unused).  A caller that runs the vitality analysis anyway
       hands them over and the timeline call does not walk kernel_tensors a second time: it books every
       tensor's size at the slots given (a pair with last < first or last >= K sets
       G10_DEV_BAD_FIRST_LAST and is skipped).  Without them the call derives both from the trace. */
    const int32_t *first_use;
    const int32_t *last_use;
} g10_timeline_out;

/* Candidate geometry of a period for one destination (Algorithm 1: t = tensor_size / BW; Section 4.4:
   prefetch at the latest safe prefetch time).  t = ceil(bytes * 1e9 / bw) ns (saturated at 2^62).
   Eviction runs in [t_r, t_r + t), t_r = end of kernel u; prefetch in [t_end - t, t_end), t_end =
   start of kernel v.  The tensor counts as absent in the slots lying wholly between the two windows,
   absent_first .. absent_last.  A pair that cannot be used (2t > period length, or no whole slot
   left) has absent_first = -1, absent_last = -2.  Index [X * Pn + p], X = G10_DEST_SSD / G10_DEST_HOST. */
typedef struct g10_geometry_out {
    int64_t *transfer_ns;       /* [2 * Pn]                                                         */
    int32_t *absent_first;      /* [2 * Pn]                                                         */
    int32_t *absent_last;       /* [2 * Pn]                                                         */
} g10_geometry_out;

/* One committed migration (the step of Algorithm 1 that schedules a tensor's pre-eviction to its destination
   at the start of the period; the matching prefetch is issued at prefetch_issue_ns).  Records appear in commit order. */
typedef struct g10_migration {
    int32_t period, tensor, dest;
    int32_t absent_first, absent_last;
    int32_t iteration;
    int64_t evict_issue_ns, prefetch_issue_ns, transfer_ns;
} g10_migration;                /* 48 bytes */

typedef struct g10_plan_out {
    g10_migration *migrations;  /* [migrations_cap] (the number of periods always suffices; E bounds it) */
    int64_t migrations_cap;
    int64_t *final_pressure;    /* [K] pressure after every committed migration                     */
    int64_t *summary;           /* [8]: migrations, scoring rounds, exit status, final peak bytes,
                                   final peak slot, bytes sent to SSD, bytes sent to host, device status word */
} g10_plan_out;

typedef struct g10_options {
    uint64_t host_capacity_bytes;   /* host memory available for evicted tensors; 0 = unlimited      */
    int64_t max_iterations;         /* 0 = as many as there are periods                              */
    uint32_t flags;                 /* G10_FLAG_*                                                    */
    void **stage_events;            /* optional: num_stage_events cudaEvent_t handles owned by the caller; the
                                       planner records them on `stream` at its stage boundaries, in order:
                                       start, after slot clock + vitality, after the pressure timeline,
                                       after candidate geometry, after the greedy loop (extra handles unused) */
    int32_t num_stage_events;
} g10_options;

#define G10_NUM_PLAN_STAGES 5

#define G10_FLAG_RESCORE_ALL 0x1    /* the plain formulation of every stage: every live period rescored every
                                       iteration (Algorithm 1 as printed), use lists built with global atomics
                                       instead of shared-memory buckets; identical results, slower           */

#define G10_FLAG_GLOBAL_STATE 0x2   /* keep the planner state in global memory even when the timeline would fit
                                       in shared memory (the path large traces take); same plan              */

#define G10_FLAG_MULTI_BLOCK 0x4    /* never let a single block run the greedy loop out of its shared memory (the path
                                       the smallest traces take); same plan                                  */

#ifdef G10_TEST_HOOKS
/* Honoured only by the test build of the library (compiled with -DG10_TEST_HOOKS, never shipped): one block of the
   planner's cooperative grid skips its first grid-barrier arrival and every barrier wait of the call is limited to a
   millisecond, so that the give-up path of the bounded waits can be exercised: the call returns with
   G10_DEV_TIMEOUT in summary[7].  The product build ignores the bit. */
#define G10_FLAG_TEST_SKIP_ARRIVAL 0x40000000
#endif

#define G10_WS_VITALITY 0
#define G10_WS_TIMELINE 1
#define G10_WS_PLAN 2
#define G10_WS_GEOMETRY 3
#define G10_WS_EMIT 4
#define G10_WS_BATCH 5
#define G10_WS_PREFETCH 6
#define G10_WS_ANALYSIS 7   /* g10_vitality with its `timeline` output */

/* Section 4.2, tensor vitality analysis.  Device-found errors land in counts[2]; with G10_DEV_BAD_KERNEL_PTR every
   tensor is reported unused (no uses, no periods), with G10_DEV_BAD_TENSOR_ID the offending entries are skipped. */
int32_t g10_vitality(const g10_trace *trace, g10_vitality_out *out, void *ws, size_t ws_bytes, void *stream);

/* Section 4.3, GPU memory pressure over time (difference array of signed sizes + prefix scan). */
int32_t g10_pressure_timeline(const g10_trace *trace, g10_timeline_out *out, void *ws, size_t ws_bytes, void *stream);

/* Algorithm 1 / Section 4.4: transfer times and absent-slot ranges of every period for both
   destinations.  All pointers are DEVICE pointers; kernel_start_ns [K+1] and the period arrays come
   from the two calls above.  Needs no workspace. */
int32_t g10_candidate_geometry(int64_t num_kernels, int64_t num_periods, const int64_t *kernel_start_ns,
                               const int64_t *tensor_bytes, const int32_t *period_tensor,
                               const int32_t *period_prev_use, const int32_t *period_next_use,
                               uint64_t host_bw, uint64_t ssd_bw, g10_geometry_out *out, void *stream);

/* Algorithm 1, smart tensor eviction: vitality, pressure, geometry, then the greedy loop -- until the
   peak pressure fits gpu_capacity_bytes or no period relieves pressure above it: score every live
   period (destination SSD first, host when the SSD channel is booked or too slow; benefit = pressure
   above capacity removed, in byte*ns; cost = eviction + prefetch time), take the best benefit/cost
   ratio (exact comparison, ties to the lowest period index), commit it (pressure, channel time, host
   occupancy) and erase the period.  Bandwidths in bytes per second. */
int32_t g10_plan_migrations(const g10_trace *trace, uint64_t gpu_capacity_bytes, uint64_t host_bw, uint64_t ssd_bw,
                            const g10_options *options /* NULL = defaults */, g10_plan_out *out,
                            void *ws, size_t ws_bytes, void *stream);

/* Section 4.4, smart tensor prefetching: visits the committed migrations in the order of their latest safe
   prefetch time (ties: the earlier plan record) and moves each prefetch back to the earliest slot from which
   pressure + size stays within gpu_capacity_bytes up to the old prefetch slot (never past absent_first), adding
   the tensor's size to the slots it becomes resident in again.  Only memory is examined (the section says nothing
   of bandwidth); a prefetch that moves is issued at the start of its first newly resident slot.
   All pointers are DEVICE pointers.  `pressure` [K] is the final pressure of the eviction plan on entry and the
   pressure after the pass on return; order [n] receives the visiting order; new_absent_last [n] and
   new_prefetch_issue_ns [n] are indexed by plan record; summary [5] = prefetches moved, slots regained, new peak,
   its lowest slot, device status word (0, or G10_DEV_TIMEOUT when a wait between thread blocks ran out: the other
   outputs are then not valid).
   `ws` (optional; G10_WS_PREFETCH, with the number of migrations in place of E; contents are scratch): with it, a
   timeline too long for one SM's shared memory (more than 15 360 slots, up to about 25 000 slots per SM of the GPU;
   at most 262 144 migrations) is cut into slices, one per thread block of a cooperative launch, and every block walks the records in visiting
   order, waiting only for the records that can still reach its slice; the result is that of the sequential pass.
   With ws == NULL (ws_bytes ignored) one block does the whole pass, record by record.
   Records of g10_plan_cyclic are accepted as they are: a slot beyond K stands for the same slot of the cycle (the
   pressure curve has K slots), a moved prefetch is issued at the unrolled time of its first regained slot, and the
   visiting order is that of the prefetch's moment inside the iteration (its time modulo the iteration's length);
   records that wrap around are always visited by one block.  For an ordinary plan nothing changes. */
typedef struct g10_prefetch_out {
    int64_t *pressure;
    int32_t *order;
    int32_t *new_absent_last;
    int64_t *new_prefetch_issue_ns;
    int64_t *summary;
} g10_prefetch_out;
int32_t g10_schedule_prefetch(int64_t num_kernels, int64_t num_migrations, const g10_migration *migrations,
                              const int64_t *kernel_start_ns, const int64_t *tensor_bytes, uint64_t gpu_capacity_bytes,
                              g10_prefetch_out *out, void *ws, size_t ws_bytes, void *stream);

/* Section 4.4, code instrumentation (the instrumented program of Figure 9): the g10_alloc / g10_free /
   g10_pre_evict / g10_prefetch calls to insert between the kernels.  Boundary b (0 <= b <= K) is the gap before
   kernel b (b = K: after the last kernel).  ALLOC sits before the first kernel using the tensor (boundary 0 for a
   global tensor), FREE right after the last kernel using an intermediate tensor (global tensors are never freed),
   PRE_EVICT at the boundary whose time is the period start t_r, PREFETCH at the last boundary at or before its
   issue time.  Inside a boundary: FREE, PRE_EVICT, ALLOC, PREFETCH (as in Figure 9), then by tensor id.
   inst_ptr [K + 2] is the CSR by boundary; counts [2] = number of instructions, device status word
   (G10_DEV_PLAN_OVERFLOW if instructions_cap is too small).  new_prefetch_issue_ns (optional) are the times from
   g10_schedule_prefetch.  All pointers are DEVICE pointers; `ws` as for the other calls (G10_WS_EMIT, with the
   number of migrations in place of E).  Limits: K + 1 <= 4096 * 4096 boundaries.
   Records of g10_plan_cyclic are accepted as they are: the stream is that of one iteration of the cycle, and the
   prefetch of a wrap-around period, whose time lies in the next iteration, stands at the same moment of this one
   (time and boundary modulo the iteration). */
#define G10_OP_FREE 0
#define G10_OP_PRE_EVICT 1
#define G10_OP_ALLOC 2
#define G10_OP_PREFETCH 3
typedef struct g10_instruction {
    int32_t opcode, tensor;
    int32_t target;                 /* destination of a pre-eviction (G10_DEST_*), else -1 */
    int32_t record;                 /* plan record of a pre-eviction / prefetch, else -1   */
    int64_t bytes, time_ns;
} g10_instruction;                  /* 32 bytes */
typedef struct g10_emit_out {
    int64_t *inst_ptr;
    g10_instruction *instructions;
    int64_t instructions_cap;       /* 2 * N + 2 * num_migrations always suffices */
    int64_t *counts;
} g10_emit_out;
int32_t g10_emit_instructions(int64_t num_kernels, int64_t num_tensors, const int32_t *first_use, const int32_t *last_use,
                              const int64_t *tensor_bytes, const uint8_t *tensor_global, const int64_t *kernel_start_ns,
                              int64_t num_migrations, const g10_migration *migrations, const int64_t *new_prefetch_issue_ns,
                              g10_emit_out *out, void *ws, size_t ws_bytes, void *stream);

/* Steady-state planning on the cyclic timeline.  Section 4.2 notes that the inactive period of a global tensor (a
   weight) may span two consecutive training iterations.  Here the traced iteration is taken to repeat unchanged:
   the timeline is a cycle of K slots, unrolled slot k + K is slot k one iteration later (unrolled time + the length
   of the iteration).  Besides the ordinary periods, every used global tensor has one wrap-around period from its
   last use to its first use of the next iteration, (tensor, last, first + K), if at least one slot lies in between;
   these are numbered after the ordinary periods, by tensor id.  Geometry, scoring and commits are those of
   g10_plan_migrations on the unrolled clock, while pressure, channel bookings and host occupancy belong to the
   physical slot k mod K.  Records carry unrolled slots and times (absent_last may be >= K, the prefetch time may lie
   in the next iteration).  Same arguments, outputs and workspace (G10_WS_PLAN) as g10_plan_migrations; of the
   options only host_capacity_bytes and max_iterations are used.  g10_schedule_prefetch and g10_emit_instructions take
   the records as they are.
   A trace whose pressure, clock, bookings and periods fit the shared memory of one SM (K <= 32000) is planned by one
   thread block; a larger one by the multi-block formulation of Algorithm 1 as printed (every live period rescored
   every iteration: the same plan, slower). */
int32_t g10_plan_cyclic(const g10_trace *trace, uint64_t gpu_capacity_bytes, uint64_t host_bw, uint64_t ssd_bw,
                        const g10_options *options /* NULL = defaults */, g10_plan_out *out,
                        void *ws, size_t ws_bytes, void *stream);

/* Section 5's sensitivity studies seen from the planner: the same trace planned under V variants at once -- other
   kernel durations (profiling error), SSD / host bandwidths, GPU capacity, host capacity -- one thread block per
   variant, all variants running concurrently.  Every variant's result is exactly what g10_plan_migrations gives for
   the trace with that variant's durations and parameters.  `variants` is a HOST array (copied before the call
   returns); its kernel_ns pointers are DEVICE pointers.  Outputs are DEVICE pointers: migrations [V][migrations_cap],
   final_pressure [V][K], summary [V][8] (as in g10_plan_out; summary[8 v + 7] holds the status bits of variant v),
   stability [V][2] = (|M_v & M_0|, |M_v | M_0|) over the sets of migrated periods of variant v and variant 0 (their
   quotient is the Jaccard index; (-1, -1) when a plan is missing).
   Limits: the trace has to be device resident (G10_MEM_DEVICE); 1 <= V <= 1024.
   One block per variant requires that pressure, clock, bookings and the periods of the trace fit the shared memory of
   one SM (the DNN-shaped traces of a few thousand kernels do).  Only the device can tell, so the call reads variant
   0's summary back (one small copy and a synchronisation of `stream`: unlike the other calls this one returns with
   its kernels finished); if the trace did not fit, the variants are then planned one after the other by the planners
   that use the whole GPU -- the same results, V times the time of one plan.
   Workspace: G10_WS_BATCH. */
typedef struct g10_variant {
    const int64_t *kernel_ns;       /* [K] device pointer, or NULL: the trace's own durations */
    uint64_t gpu_capacity_bytes;
    uint64_t host_bw, ssd_bw;       /* bytes per second */
    uint64_t host_capacity_bytes;   /* 0 = unlimited */
} g10_variant;
typedef struct g10_batch_out {
    g10_migration *migrations;
    int64_t migrations_cap;         /* records per variant */
    int64_t *final_pressure;
    int64_t *summary;
    int64_t *stability;
} g10_batch_out;
int32_t g10_plan_batch(const g10_trace *trace, int32_t num_variants, const g10_variant *variants, int64_t max_iterations,
                       g10_batch_out *out, void *ws, size_t ws_bytes, void *stream);

/* Section 3, workload characterisation (the statistics of Figures 2-4) from the results of g10_vitality and the
   slot clock of g10_pressure_timeline.  active_bytes [K]: bytes of the tensors kernel k uses, each once (the
   working set that has to fit while k runs).  len_hist [64]: inactive periods by floor(log2 L), L = the period's
   length in ns.  size_len_hist [41 * 45], row-major: periods by min(floor(log2 size), 40) x min(floor(log2 L), 44).
   hide [2]: periods with 2 * transfer time <= L for the SSD and for the host link (indexed by G10_DEST_*).
   summary [2]: max of active_bytes and its lowest kernel (0, -1 for K = 0).  All pointers are DEVICE pointers;
   use_ptr [N + 1] / uses are the CSR of distinct uses; the call zeroes its outputs itself.  Needs no workspace. */
#define G10_STATS_LEN_BINS 64
#define G10_STATS_SIZE_BINS 41
#define G10_STATS_LEN2_BINS 45
typedef struct g10_stats_out {
    int64_t *active_bytes;
    int64_t *len_hist;
    int64_t *size_len_hist;
    int64_t *hide;
    int64_t *summary;
} g10_stats_out;
int32_t g10_characterize(int64_t num_kernels, int64_t num_tensors, const int64_t *use_ptr, const int32_t *uses,
                         const int64_t *tensor_bytes, const int64_t *kernel_start_ns, int64_t num_periods,
                         const int32_t *period_tensor, const int32_t *period_prev_use, const int32_t *period_next_use,
                         uint64_t host_bw, uint64_t ssd_bw, g10_stats_out *out, void *stream);

/* The paper has no counterpart for this entry point: it is g10_pressure_timeline for callers that cannot
   allocate device memory when they need a timeline (a host whose device memory is wholly owned by its own
   pool, or a code path where cudaMalloc / cudaFree are ruled out because they may synchronise the device).
   It takes no workspace: its scratch is a fixed 1.5 MiB array inside the library image, present on every GPU
   that loads the library until the process exits.  Consequences the caller must know:
     - device pointers only (trace->mem must be G10_MEM_DEVICE); same outputs, same device status word and the
       same stream semantics as g10_pressure_timeline (the optional first_use / last_use inputs of the output
       struct are not looked at: first and last use always come from the trace);
     - traces up to G10_STATIC_MAX_KERNELS kernels and G10_STATIC_MAX_TENSORS tensors; anything larger is
       refused with G10_ERR_LIMIT before any work is enqueued;
     - the first call on each device looks the array's address up (cudaGetSymbolAddress, with that device
       current); make that first call outside any stream capture.  The address is remembered for the life of the
       process: after cudaDeviceReset() (or any teardown of the device's primary context) it is stale and this
       entry point must not be called again in that process;
     - all calls on a device share the one array, which keeps the previous call's contents (the call clears
       what it needs zeroed); two calls that overlap on the GPU -- different streams, or one stream per thread --
       race on it and give wrong results, so serialise them;
     - it never calls cudaMalloc, cudaFree or any allocating library routine. */
#define G10_STATIC_MAX_KERNELS 32768
#define G10_STATIC_MAX_TENSORS 131072
int32_t g10_pressure_timeline_static(const g10_trace *trace, g10_timeline_out *out, void *stream);

/* Bytes of device workspace the call `which` (G10_WS_*) needs for a trace of K kernels, N tensors,
   E events whose arrays live in `mem`. */
int32_t g10_workspace_bytes(int32_t which, int64_t num_kernels, int64_t num_tensors, int64_t num_events,
                            int32_t mem, size_t *out_bytes);

const char *g10_strerror(int32_t code);
int32_t g10_version(void);
/* Diagnostic: kernels this library has launched in the process so far (a benchmark reads it before and after its timed
   region to say how many of the library's own kernels ran there). */
uint64_t g10_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* G10_H_ */

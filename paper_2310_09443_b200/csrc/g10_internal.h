// Host-side declarations shared by the translation units of the library: workspace layout and the
// launchers of each pass.  Everything here works on DEVICE pointers.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "g10.h"

namespace g10 {

typedef unsigned long long ull;

// Kernels this library has launched in the process so far (every launch site counts itself; read through
// g10_launch_count, which benchmarks use to report how many of the library's kernels ran inside a timed region).
extern ull g_launch_count;
inline void count_launch() { __atomic_fetch_add(&g_launch_count, 1ull, __ATOMIC_RELAXED); }
}  // namespace g10
#define cudaLaunchKernelEx(...) (g10::count_launch(), ::cudaLaunchKernelEx(__VA_ARGS__))
#define cudaLaunchCooperativeKernel(...) (g10::count_launch(), ::cudaLaunchCooperativeKernel(__VA_ARGS__))
namespace g10 {

constexpr size_t kAlign = 256;
constexpr int kHeavyThreshold = 32;      // tensors with more raw uses than this are sorted by a whole block

// Multiprocessors of the current device (0 if the query fails).  Asked every time: a process may use several devices.
inline int current_sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return sms > 0 ? sms : 0;
}

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline int64_t tiles_of(int64_t n, int64_t tile) { return n <= 0 ? 1 : (n + tile - 1) / tile; }

// One scan's look-back state inside the zero-initialised part of the workspace.
struct ScanSlot {
    unsigned *ticket;
    unsigned *done;
    unsigned *flag;
    long long *agg;
    long long *incl;
};

struct Proposal {          // a block's best candidate of one scoring round (32 bytes)
    ull ben_lo, ben_hi;
    ull cost;
    int idx;               // -1 = none
    int dest;
};

// Large-trace planner: what a block publishes after a pass over its periods (best FRESH candidate, best STALE
// bounds) and the sizes of its joint rescoring rounds.
constexpr int kLazyMaxBlocks = 256;
constexpr int kTopT = 4;
constexpr int kRoundM = 512;      // periods rescored together in one round, at most
constexpr int kDirtyPool = 256;   // DIRTY periods of one commit that join a round (more: rescored at once, shared out)
constexpr int kFirstM = 8;        // ... in the first round of an iteration (best bounds first)
struct __align__(16) LazyProp {
    ull ben_lo, ben_hi, cost;
    int idx, dest;
    double skey[kTopT];
    int sidx[kTopT];
};

// One variant of a batched re-planning call (device copy of g10_variant with the defaults filled in).
struct BatchVariant {
    const int64_t *kernel_ns;
    uint64_t cap, host_bw, ssd_bw, host_capacity;
};
struct BatchArgs {
    const BatchVariant *variants;     // [V]
    const int64_t *P0;                // [K] unplanned pressure, shared by all variants
    int64_t *P_out;                   // [V][K]
};
constexpr int kMaxVariants = 1024;

// Device views of a trace and of the intermediate arrays; filled by carve() in g10_api.cu.
struct Workspace {
    // --- zero-initialised region (one memset per call) ---
    char *zero_begin;
    size_t zero_bytes;
    size_t state_bytes;          // bytes of busy + hocc + dead (contiguous)
    ull *status;                 // device status word
    unsigned *heavy_count;
    int *peak_key;               // K - lowest peak slot (0 = none), reduced with atomicMax
    void *barrier;               // GridBarrier
    ScanSlot clock_scan, count_scan, emit_scan, pressure_scan;
    int32_t *cnt;                // [N] raw use counts, then scatter cursor, then heavy slot index
    int64_t *diff;               // [K+1] signed-size difference array
    int64_t *busy;               // [4*K] booked channel time per slot
    int64_t *hocc;               // [K] host-memory occupancy per slot
    unsigned char *dead;         // [E] period erased
    unsigned *wl_count;          // [2] lengths of the two DIRTY work lists
    unsigned *one_done;          // [1] the single-block planner produced the plan
    ull *event_budget;           // [1] events booked by the blocks of the first / last pass (at most E for a valid trace)
    unsigned *bk_count, *bk_cursor;   // [4096] events per tensor bucket, scatter cursors
    ull *bk_words;               // [2 * 4096] tagged per-bucket totals
    long long *bk_carry;         // [4] distinct uses and periods of all tensors before the current pass (two copies used in turn)
    ull *xwords;                 // [2][kSmallMaxBlocks][16] tagged words of the proposal exchange
    ull *seg_words, *seg_words2; // [blocks * 16] each: tagged segment sums of the slot-clock scan and of the pressure scan, one 128-byte line per block
    // --- uninitialised region ---
    int32_t *raw_ptr;            // [N+1]
    int32_t *raw_uses;           // [E]
    int32_t *heavy_list;         // [E/33+1] tensor ids
    int32_t *heavy_info;         // [2*(E/33+1)] distinct uses, periods
    int64_t *tile_max;           // [tiles(K)]
    int32_t *tile_slot;          // [tiles(K)]
    int64_t *tl_point;           // [K] bytes of the tensors alive in one slot only (timeline call)
    int *tl_pair;                // [2 * N] first / last use of every tensor, encoded (timeline call)
    // vitality / timeline outputs when the caller did not ask for them (planner) or passed host memory
    int32_t *first_use, *last_use, *num_uses;
    int64_t *use_ptr, *period_ptr;
    int32_t *uses, *period_tensor, *period_prev_use, *period_next_use;
    int64_t *counts;             // [3]
    int64_t *start;              // [K+1]
    int64_t *start2;             // [2K+1] unrolled clock (cyclic planning)
    int64_t *pressure;           // [K]
    int64_t *peak_bytes;         // [1]
    int32_t *peak_slot;          // [1]
    int64_t *geo_t;              // [2*E]
    int32_t *geo_a, *geo_b;      // [2*E]
    Proposal *proposals;         // [max blocks]
    Proposal *prop_stale;        // [max blocks]
    LazyProp *lazy_props;        // [2][kLazyMaxBlocks]
    ull *lazy_partials;          // [2][kRoundM][kLazyMaxBlocks][2]
    int64_t *lazy_tmin, *lazy_tmax; // [tiles of 1024 slots]
    unsigned char *c_state;      // [E] per-period state of the lazy planner
    ull *c_ben_lo, *c_ben_hi, *c_cost;   // [E] cached benefit and cost
    double *c_key;               // [E] rounded benefit / cost
    int2 *c_rng;                 // [E] absent range of the current destination
    int *worklist;               // [2*E]
    ull *bk_pairs;               // [E] events as (tensor in bucket, kernel) keys, bucket after bucket
    int64_t *busy_rep, *hocc_rep; // per-block copies of the channel bookings / host occupancy (small-trace planner)
    int64_t *peak_part;          // [max blocks]
    g10_migration *migrations;   // host mode only
    int64_t *summary;            // [8]
    BatchVariant *batch_variants; // [kMaxVariants]
    // staged copies of the trace (host mode only)
    int64_t *s_kernel_ptr, *s_tensor_bytes, *s_kernel_ns;
    int32_t *s_kernel_tensors;
    uint8_t *s_tensor_global;
};

struct DeviceTrace {
    int64_t K, N, E;
    const int64_t *kernel_ptr;
    const int32_t *kernel_tensors;
    const int64_t *tensor_bytes;
    const int64_t *kernel_ns;
    const uint8_t *tensor_global;
};

struct VitalityBuffers {
    int32_t *first_use, *last_use, *num_uses;
    int64_t *use_ptr;
    int32_t *uses;
    int64_t uses_cap;
    int64_t *period_ptr;
    int32_t *period_tensor, *period_prev_use, *period_next_use;
    int64_t periods_cap;
    int64_t *counts;   // [3]
    // When the caller wants the pressure timeline from the same call (bucketed formulation only): the kernel that writes
    // first / last use also books every tensor's size into the difference array [K + 1] and the point masses [K] (both
    // cleared beforehand), so that only the scan is left to do.  All null otherwise.
    ull *tl_diff = nullptr, *tl_point = nullptr;
    bool tl_cleared = false;     // tl_diff and tl_point have been cleared by an earlier kernel of the stream
    const int64_t *tl_bytes = nullptr;
    const uint8_t *tl_glob = nullptr;
    int64_t tl_K = 0;
};

struct PlanParams {
    uint64_t gpu_capacity_bytes, host_bw, ssd_bw, host_capacity_bytes;
    int64_t max_iterations;
    uint32_t flags;
    g10_migration *migrations;
    int64_t migrations_cap;
    int64_t *final_pressure;
    int64_t *summary;
};

constexpr int kMaxPlanBlocks = 1024;
constexpr int kSmallMaxBlocks = 160;       // blocks of the small-trace planner (one per SM, at most)
constexpr int64_t kSmallMaxSlots = 12000;  // largest K whose pressure + clock fit in shared memory

// passes (g10_passes.cu)
// (zero_diff [K + 1], zero_point [K]: arrays the kernel clears on its way, for a later kernel of the same call)
cudaError_t launch_slot_clock(const DeviceTrace &t, const Workspace &w, int64_t *start, cudaStream_t s, bool check_kernel_ptr = true,
                              int64_t *zero_diff = nullptr, int64_t *zero_point = nullptr);
cudaError_t launch_vitality(const DeviceTrace &t, const Workspace &w, const VitalityBuffers &out, cudaStream_t s);
// bucketed formulation (g10_vitality_buckets.cu); 4096 buckets of 4096 tensors per pass over the events, up to 16 passes
bool vitality_buckets_supported(int64_t N, int64_t E);
// (status_out, if not null, receives the device status word when the last block of the last kernel finishes)
// (pdl_first: the first kernel may start while its predecessor in the stream, which has released its dependents, still runs)
cudaError_t launch_vitality_buckets(const DeviceTrace &t, const Workspace &w, const VitalityBuffers &out, cudaStream_t s, int64_t *status_out = nullptr,
                                    bool pdl_first = false);
// the pressure scan alone (difference array and point masses are complete when its predecessor in the stream is)
cudaError_t launch_pressure_scan(const DeviceTrace &t, const Workspace &w, const int64_t *point, int64_t *pressure, int64_t *peak_bytes,
                                 int32_t *peak_slot, int64_t *status_out, cudaStream_t s);
cudaError_t launch_first_last(const DeviceTrace &t, const Workspace &w, int32_t *first_use, int32_t *last_use, cudaStream_t s);
cudaError_t launch_pressure(const DeviceTrace &t, const Workspace &w, const int32_t *first_use, const int32_t *last_use, bool encoded,
                            int64_t *pressure, int64_t *peak_bytes, int32_t *peak_slot, cudaStream_t s);
cudaError_t launch_geometry(int64_t K, int64_t Pn_bound, const int64_t *Pn_dev, const int64_t *start, const int64_t *tensor_bytes,
                            const int32_t *per_t, const int32_t *per_u, const int32_t *per_v, uint64_t host_bw, uint64_t ssd_bw,
                            int64_t stride, int64_t *geo_t, int32_t *geo_a, int32_t *geo_b, cudaStream_t s);
// timeline call: slot clock, pressure, peak from the trace alone (g10_passes.cu)
cudaError_t launch_timeline_pairs(const DeviceTrace &t, const Workspace &w, int64_t *start, int32_t *pair, int64_t *point, int64_t *pressure,
                                  int64_t *peak_bytes, int32_t *peak_slot, int64_t *status_out /* receives the device status word */, cudaStream_t s);
// timeline call with first / last use handed over by the caller (g10_passes.cu)
cudaError_t launch_timeline_given(const DeviceTrace &t, const Workspace &w, int64_t *start, const int32_t *first_use, const int32_t *last_use,
                                  int64_t *point, int64_t *pressure, int64_t *peak_bytes, int32_t *peak_slot, int64_t *status_out, cudaStream_t s);
// eager prefetch pass (g10_prefetch.cu)
constexpr int kPfMaxBlocks = 2048;         // most blocks the many-block form of the pass may use (one slice of the timeline each)
// Scratch of the many-block form, carved from the caller's workspace (all null: the call came without one).
struct PrefetchScratch {
    ull *status;              // device status word                                      }
    unsigned *ticket;         // blocks that have finished                               } cleared before the launch
    unsigned *fallback;       // set when the records need the one-block form after all  }
    unsigned *word;           // [n] where each record's search stands                   }
    unsigned *rank;           // [n] position of each record in the visiting order       }
    int32_t *first, *last;    // [n] absent_first / absent_last in visiting order
    int64_t *size;            // [n] tensor size in visiting order
    int64_t *block_max;       // [kPfMaxBlocks] largest pressure of each block's slice ...
    int32_t *block_slot;      // [kPfMaxBlocks] ... and its lowest slot
};
cudaError_t launch_schedule_prefetch(int64_t K, int64_t n, const g10_migration *mig, const int64_t *start, const int64_t *bytes,
                                     uint64_t gpu_capacity_bytes, int64_t *P, int32_t *order, int32_t *new_last, int64_t *new_issue,
                                     int64_t *summary, const PrefetchScratch &scratch, cudaStream_t s);
// instruction-stream emission (g10_emit.cu)
constexpr int kEmitMaxBlocks = 1024;       // most blocks the counting and the scatter kernel run with
struct EmitLaunch {
    int64_t K, N, n;
    const int32_t *first_use, *last_use;
    const int64_t *bytes;
    const uint8_t *glob;
    const int64_t *start;
    const g10_migration *mig;
    const int64_t *new_issue;
    unsigned *bucket_count, *bucket_cursor, *ticket;
    unsigned *block_count;       // [4096][kEmitMaxBlocks] instructions of each bucket seen by each block of the counting kernel
    ull *keys;
    int32_t *payload;
    ull *status;
    int64_t *inst_ptr;
    g10_instruction *inst;
    int64_t inst_cap;
    int64_t *counts;
};
bool emit_choose_buckets(int64_t K, int64_t total_items, int sms, int *bw, int *nb, ull *magic);
cudaError_t launch_emit(const EmitLaunch &L, cudaStream_t s);
cudaError_t launch_characterize(int64_t K, int64_t N, const int64_t *use_ptr, const int32_t *uses, const int64_t *bytes, const int64_t *start,
                                int64_t Pn, const int32_t *per_t, const int32_t *per_u, const int32_t *per_v, uint64_t host_bw, uint64_t ssd_bw,
                                int64_t *active, int64_t *len_hist, int64_t *size_len_hist, int64_t *hide, int64_t *summary, cudaStream_t s);
// planner (g10_planner.cu)
cudaError_t launch_plan_loop(const DeviceTrace &t, const Workspace &w, const PlanParams &p, cudaStream_t s);
cudaError_t launch_cyclic_prepare(const DeviceTrace &t, const Workspace &w, cudaStream_t s);
cudaError_t launch_plan_cyclic(const DeviceTrace &t, const Workspace &w, const PlanParams &p, cudaStream_t s);
cudaError_t launch_plan_variants(const DeviceTrace &t, const Workspace &w, const PlanParams &p, int V, int64_t *stability, cudaStream_t s);
// stability pairs of V finished plans against plan 0; ORs *status_word into every plan's summary[7]
cudaError_t launch_batch_finish(const DeviceTrace &t, const Workspace &w, const PlanParams &p, int V, int64_t *stability, const ull *status_word,
                                cudaStream_t s);
int plan_loop_max_blocks();
bool plan_keeps_state_on_chip(int64_t K, int64_t E, uint32_t flags);   // true: the small-trace planner will run
cudaError_t launch_publish_status(const Workspace &w, int64_t *dst, cudaStream_t s);
cudaError_t launch_publish_status_or(const Workspace &w, int64_t *dst, cudaStream_t s);

}  // namespace g10

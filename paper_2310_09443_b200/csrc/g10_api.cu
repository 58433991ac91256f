// The C ABI: argument checks, workspace layout, host-buffer staging and the launch sequence of each call.
#include <cstring>
#include <vector>

#include "g10_device.cuh"
#include "g10_internal.h"

namespace g10 {
ull g_launch_count = 0;
namespace {

struct Sizes {
    int64_t K, N, E;
    bool host;
};

// Lays the workspace out; with base == nullptr only measures it.
struct Carver {
    char *base;
    size_t off = 0;
    explicit Carver(void *b) : base((char *)b) {}
    template <typename T>
    T *take(size_t count)
    {
        off = align_up(off);
        T *p = base ? (T *)(base + off) : nullptr;
        off += sizeof(T) * (count ? count : 1);
        return p;
    }
};

void carve_scan(Carver &c, ScanSlot &s, int64_t tiles, int nv)
{
    s.ticket = c.take<unsigned>(1);
    s.done = c.take<unsigned>(1);
    s.flag = c.take<unsigned>((size_t)tiles);
    s.agg = c.take<long long>((size_t)tiles * nv);
    s.incl = c.take<long long>((size_t)tiles * nv);
}

// `which` (G10_WS_*) decides what is laid out: the timeline call needs neither the partition scratch of the vitality
// call nor the planner's state, the vitality call no timeline arrays; the planner calls need everything.
size_t carve(void *base, const Sizes &z, Workspace &w, int32_t which)
{
    std::memset(&w, 0, sizeof(w));
    Carver c(base);
    const bool vit = which != G10_WS_TIMELINE, tl = which != G10_WS_VITALITY;
    const bool plan = which != G10_WS_TIMELINE && which != G10_WS_VITALITY && which != G10_WS_ANALYSIS;
    const bool inner = plan || z.host;             // results of the analysis calls kept inside the workspace
    const size_t K = (size_t)z.K, N = (size_t)z.N, E = (size_t)z.E;
    const size_t heavy = E / (kHeavyThreshold + 1) + 1;
    const int64_t ktiles = tiles_of(z.K, 2048), ntiles = tiles_of(z.N, 2048), etiles = tiles_of(z.N, 1024);
    // zero-initialised region
    w.zero_begin = c.base ? c.base : nullptr;
    w.status = c.take<ull>(1);
    w.heavy_count = c.take<unsigned>(1);
    w.peak_key = c.take<int>(1);
    w.barrier = c.take<unsigned>(4);
    carve_scan(c, w.clock_scan, ktiles, 1);
    carve_scan(c, w.count_scan, vit ? ntiles : 1, 1);
    carve_scan(c, w.emit_scan, vit ? etiles : 1, 2);
    carve_scan(c, w.pressure_scan, ktiles, 1);
    w.wl_count = c.take<unsigned>(4);           // (two list lengths, two overflow flags)
    w.one_done = c.take<unsigned>(1);
    w.event_budget = c.take<ull>(1);
    w.bk_count = c.take<unsigned>(vit ? 4096 : 1);
    w.bk_cursor = c.take<unsigned>(vit ? 4096 : 1);
    w.bk_words = c.take<ull>(vit ? 2 * 4096 : 1);
    w.bk_carry = c.take<long long>(4);
    w.xwords = c.take<ull>(plan ? (2 * kSmallMaxBlocks + 2 * kSmallMaxBlocks) * 16 : 1);
    w.seg_words = c.take<ull>(512 * 16);
    w.seg_words2 = c.take<ull>(512 * 16);
    w.zero_bytes = align_up(c.off);
    // arrays that must start at zero, cleared only by the calls that use them (the difference array sits right behind
    // the zero-initialised region, so that one memset covers both)
    if (which == G10_WS_TIMELINE) {
        // (the first / last pairs right behind the zero-initialised region: one memset covers both; the difference array and
        // the point masses are cleared by the kernel that fills the pairs)
        w.tl_pair = c.take<int>(2 * N);
        w.diff = c.take<int64_t>(K + 1);
        w.tl_point = c.take<int64_t>(K);
    } else {
        w.diff = c.take<int64_t>(tl ? K + 1 : 1);
        w.tl_point = c.take<int64_t>(which == G10_WS_ANALYSIS ? K : 1);   // (right behind the difference array: one memset)
        w.tl_pair = c.take<int>(1);
    }
    w.cnt = c.take<int32_t>(vit ? N : 1);
    const size_t state_begin = align_up(c.off);
    w.busy = c.take<int64_t>(plan ? 4 * K : 1);       // busy, hocc and dead are contiguous: one memset
    w.hocc = c.take<int64_t>(plan ? K : 1);
    w.dead = c.take<unsigned char>(plan ? E : 1);
    w.state_bytes = align_up(c.off) - state_begin;
    // scratch
    w.raw_ptr = c.take<int32_t>(vit ? N + 1 : 1);
    w.raw_uses = c.take<int32_t>(vit ? E : 1);
    w.heavy_list = c.take<int32_t>(vit ? heavy : 1);
    w.heavy_info = c.take<int32_t>(vit ? 2 * heavy : 1);
    w.tile_max = c.take<int64_t>((size_t)ktiles);
    w.tile_slot = c.take<int32_t>((size_t)ktiles);
    w.first_use = c.take<int32_t>(vit && inner ? N : 1);
    w.last_use = c.take<int32_t>(vit && inner ? N : 1);
    w.num_uses = c.take<int32_t>(vit && inner ? N : 1);
    w.use_ptr = c.take<int64_t>(vit && inner ? N + 1 : 1);
    w.period_ptr = c.take<int64_t>(vit && inner ? N + 1 : 1);
    w.uses = c.take<int32_t>(vit && inner ? E : 1);
    w.period_tensor = c.take<int32_t>(vit && inner ? E : 1);
    w.period_prev_use = c.take<int32_t>(vit && inner ? E : 1);
    w.period_next_use = c.take<int32_t>(vit && inner ? E : 1);
    w.counts = c.take<int64_t>(4);
    w.start = c.take<int64_t>(tl && inner ? K + 1 : 1);
    w.start2 = c.take<int64_t>(plan ? 2 * K + 1 : 1);
    w.pressure = c.take<int64_t>(tl && inner ? K : 1);
    w.peak_bytes = c.take<int64_t>(1);
    w.peak_slot = c.take<int32_t>(2);
    w.geo_t = c.take<int64_t>(plan ? 2 * E : 1);
    w.geo_a = c.take<int32_t>(plan ? 2 * E : 1);
    w.geo_b = c.take<int32_t>(plan ? 2 * E : 1);
    w.proposals = c.take<Proposal>(plan ? kMaxPlanBlocks : 1);
    w.prop_stale = c.take<Proposal>(plan ? kMaxPlanBlocks : 1);
    w.lazy_props = c.take<LazyProp>(plan ? 2 * kLazyMaxBlocks : 1);
    w.lazy_partials = c.take<ull>(plan ? (size_t)2 * kRoundM * kLazyMaxBlocks * 2 : 1);
    w.lazy_tmin = c.take<int64_t>(plan ? (size_t)tiles_of(z.K, 1024) : 1);
    w.lazy_tmax = c.take<int64_t>(plan ? (size_t)tiles_of(z.K, 1024) : 1);
    w.c_state = c.take<unsigned char>(plan ? E : 1);
    w.c_ben_lo = c.take<ull>(plan ? E : 1);
    w.c_ben_hi = c.take<ull>(plan ? E : 1);
    w.c_cost = c.take<ull>(plan ? E : 1);
    w.c_key = c.take<double>(plan ? E : 1);
    w.c_rng = c.take<int2>(plan ? E : 1);
    w.worklist = c.take<int>(plan ? 2 * E : 1);
    w.bk_pairs = c.take<ull>(vit ? E : 1);
    if (plan && z.K <= kSmallMaxSlots) {
        w.busy_rep = c.take<int64_t>((size_t)kSmallMaxBlocks * 4 * K);
        w.hocc_rep = c.take<int64_t>((size_t)kSmallMaxBlocks * K);
    }
    w.peak_part = c.take<int64_t>(plan ? kMaxPlanBlocks : 1);
    w.summary = c.take<int64_t>(8);
    w.batch_variants = c.take<BatchVariant>(which == G10_WS_BATCH ? kMaxVariants : 1);
    if (z.host) {
        w.migrations = c.take<g10_migration>(plan ? E : 1);
        w.s_kernel_ptr = c.take<int64_t>(K + 1);
        w.s_kernel_tensors = c.take<int32_t>(E);
        w.s_tensor_bytes = c.take<int64_t>(N);
        w.s_kernel_ns = c.take<int64_t>(K);
        w.s_tensor_global = c.take<uint8_t>(N);
    }
    return align_up(c.off);
}

int32_t check_trace(const g10_trace *t)
{
    if (!t) return G10_ERR_ARG;
    if (t->num_kernels < 0 || t->num_tensors < 0 || t->num_events < 0) return G10_ERR_ARG;
    if (t->mem != G10_MEM_DEVICE && t->mem != G10_MEM_HOST) return G10_ERR_ARG;
    const int64_t lim = ((int64_t)1 << 31) - 1;
    if (t->num_kernels >= lim || t->num_tensors >= lim || t->num_events >= lim) return G10_ERR_LIMIT;
    if (!t->kernel_ptr) return G10_ERR_ARG;
    if (t->num_events > 0 && !t->kernel_tensors) return G10_ERR_ARG;
    if (t->num_tensors > 0 && !t->tensor_bytes) return G10_ERR_ARG;
    if (t->num_kernels > 0 && !t->kernel_ns) return G10_ERR_ARG;
    if (t->num_events > 0 && (t->num_kernels == 0 || t->num_tensors == 0)) return G10_ERR_ARG;
    return G10_OK;
}

int32_t check_ws(int32_t which, const g10_trace *t, void *ws, size_t ws_bytes)
{
    size_t need = 0;
    const int32_t rc = g10_workspace_bytes(which, t->num_kernels, t->num_tensors, t->num_events, t->mem, &need);
    if (rc != G10_OK) return rc;
    if (!ws || ((uintptr_t)ws % kAlign) != 0 || ws_bytes < need) return G10_ERR_WORKSPACE;
    return G10_OK;
}

#define CU(x)                                   \
    do {                                        \
        if ((x) != cudaSuccess) return G10_ERR_CUDA; \
    } while (0)

// Prepares the workspace and returns the device view of the trace (staging it first in host mode).
enum { kZeroCounts = 1, kZeroDiff = 2, kZeroState = 4, kZeroPairs = 8, kZeroDiffPoint = 16 };

int32_t begin_call(int32_t which, const g10_trace *t, void *ws, Workspace &w, DeviceTrace &d, cudaStream_t s, int zero_mask)
{
    Sizes z{t->num_kernels, t->num_tensors, t->num_events, t->mem == G10_MEM_HOST};
    carve(ws, z, w, which);
    {
        size_t head = w.zero_bytes;
        if (zero_mask & kZeroDiff) head = (size_t)((char *)(w.diff + z.K + 1) - w.zero_begin);
        if (zero_mask & kZeroPairs) head = (size_t)((char *)(w.tl_pair + 2 * z.N) - w.zero_begin);
        if (zero_mask & kZeroDiffPoint) head = (size_t)((char *)(w.tl_point + z.K) - w.zero_begin);
        CU(cudaMemsetAsync(w.zero_begin, 0, head, s));
    }
    if ((zero_mask & kZeroCounts) && z.N > 0) CU(cudaMemsetAsync(w.cnt, 0, sizeof(int32_t) * (size_t)z.N, s));
    if (zero_mask & kZeroState) CU(cudaMemsetAsync(w.busy, 0, w.state_bytes, s));
    d.K = z.K; d.N = z.N; d.E = z.E;
    if (!z.host) {
        d.kernel_ptr = t->kernel_ptr; d.kernel_tensors = t->kernel_tensors; d.tensor_bytes = t->tensor_bytes;
        d.kernel_ns = t->kernel_ns; d.tensor_global = t->tensor_global;
    } else {
        CU(cudaMemcpyAsync(w.s_kernel_ptr, t->kernel_ptr, sizeof(int64_t) * (size_t)(z.K + 1), cudaMemcpyHostToDevice, s));
        if (z.E) CU(cudaMemcpyAsync(w.s_kernel_tensors, t->kernel_tensors, sizeof(int32_t) * (size_t)z.E, cudaMemcpyHostToDevice, s));
        if (z.N) CU(cudaMemcpyAsync(w.s_tensor_bytes, t->tensor_bytes, sizeof(int64_t) * (size_t)z.N, cudaMemcpyHostToDevice, s));
        if (z.K) CU(cudaMemcpyAsync(w.s_kernel_ns, t->kernel_ns, sizeof(int64_t) * (size_t)z.K, cudaMemcpyHostToDevice, s));
        if (z.N && t->tensor_global)
            CU(cudaMemcpyAsync(w.s_tensor_global, t->tensor_global, (size_t)z.N, cudaMemcpyHostToDevice, s));
        d.kernel_ptr = w.s_kernel_ptr; d.kernel_tensors = w.s_kernel_tensors; d.tensor_bytes = w.s_tensor_bytes;
        d.kernel_ns = w.s_kernel_ns; d.tensor_global = t->tensor_global ? w.s_tensor_global : nullptr;
    }
    return G10_OK;
}

template <typename T>
cudaError_t d2h(T *dst, const T *src, size_t count, cudaStream_t s)
{
    if (count == 0 || dst == nullptr) return cudaSuccess;
    return cudaMemcpyAsync(dst, src, sizeof(T) * count, cudaMemcpyDeviceToHost, s);
}

size_t carve_emit(void *base, int64_t N, int64_t n, EmitLaunch &L, char **zero_begin, size_t *zero_bytes)
{
    Carver c(base);
    const size_t total = (size_t)(2 * N + 2 * n) + 1;
    *zero_begin = c.base;
    L.status = c.take<ull>(1);
    L.ticket = c.take<unsigned>(1);
    L.bucket_count = c.take<unsigned>(4096);
    L.bucket_cursor = c.take<unsigned>(4096);
    *zero_bytes = align_up(c.off);
    L.keys = c.take<ull>(total);
    L.payload = c.take<int32_t>(total);
    L.block_count = c.take<unsigned>((size_t)4096 * kEmitMaxBlocks);
    return align_up(c.off);
}

// Scratch of the eager prefetch pass (many-block form): what must start at zero first.
size_t carve_prefetch(void *base, int64_t n, PrefetchScratch &p, size_t *zero_bytes)
{
    Carver c(base);
    p.status = c.take<ull>(1);
    p.ticket = c.take<unsigned>(1);
    p.fallback = c.take<unsigned>(1);
    p.word = c.take<unsigned>((size_t)n);
    p.rank = c.take<unsigned>((size_t)n);
    *zero_bytes = align_up(c.off);
    p.first = c.take<int32_t>((size_t)n);
    p.last = c.take<int32_t>((size_t)n);
    p.size = c.take<int64_t>((size_t)n);
    p.block_max = c.take<int64_t>(kPfMaxBlocks);
    p.block_slot = c.take<int32_t>(kPfMaxBlocks);
    return align_up(c.off);
}

}  // namespace
}  // namespace g10

using namespace g10;

extern "C" {

int32_t g10_version(void) { return G10_VERSION; }

uint64_t g10_launch_count(void) { return __atomic_load_n(&g_launch_count, __ATOMIC_RELAXED); }

const char *g10_strerror(int32_t code)
{
    switch (code) {
        case G10_OK: return "ok";
        case G10_ERR_ARG: return "invalid argument";
        case G10_ERR_LIMIT: return "trace dimensions beyond the supported limits";
        case G10_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case G10_ERR_CUDA: return "a CUDA runtime call failed";
        default: return "unknown error code";
    }
}

int32_t g10_workspace_bytes(int32_t which, int64_t K, int64_t N, int64_t E, int32_t mem, size_t *out_bytes)
{
    if (!out_bytes || K < 0 || N < 0 || E < 0) return G10_ERR_ARG;
    if (which < G10_WS_VITALITY || which > G10_WS_ANALYSIS) return G10_ERR_ARG;
    if (mem != G10_MEM_DEVICE && mem != G10_MEM_HOST) return G10_ERR_ARG;
    const int64_t lim = ((int64_t)1 << 31) - 1;
    if (K >= lim || N >= lim || E >= lim) return G10_ERR_LIMIT;
    if (which == G10_WS_GEOMETRY) { *out_bytes = 0; return G10_OK; }
    if (which == G10_WS_EMIT) {                    // E stands for the number of migrations here
        EmitLaunch L;
        char *zb = nullptr;
        size_t zbytes = 0;
        *out_bytes = carve_emit(nullptr, N, E, L, &zb, &zbytes);
        return G10_OK;
    }
    if (which == G10_WS_PREFETCH) {                // E stands for the number of migrations here
        PrefetchScratch p;
        size_t zbytes = 0;
        *out_bytes = carve_prefetch(nullptr, E, p, &zbytes);
        return G10_OK;
    }
    Workspace w;
    Sizes z{K, N, E, mem == G10_MEM_HOST};
    *out_bytes = carve(nullptr, z, w, which);
    return G10_OK;
}

int32_t g10_vitality(const g10_trace *trace, g10_vitality_out *out, void *ws, size_t ws_bytes, void *stream)
{
    int32_t rc = check_trace(trace);
    if (rc != G10_OK) return rc;
    if (!out || !out->first_use || !out->last_use || !out->num_uses || !out->use_ptr || !out->period_ptr || !out->counts)
        return G10_ERR_ARG;
    if (out->uses_cap < 0 || out->periods_cap < 0) return G10_ERR_ARG;
    if ((out->uses_cap > 0 && !out->uses) ||
        (out->periods_cap > 0 && (!out->period_tensor || !out->period_prev_use || !out->period_next_use)))
        return G10_ERR_ARG;
    g10_timeline_out *to = out->timeline;                  // the pressure timeline from the same call, if wanted
    if (to) {
        if (to->first_use || to->last_use) return G10_ERR_ARG;
        if (!to->kernel_start_ns || !to->peak_bytes || !to->peak_slot || !to->status || (trace->num_kernels > 0 && !to->pressure)) return G10_ERR_ARG;
    }
    const int32_t wsk = to ? G10_WS_ANALYSIS : G10_WS_VITALITY;
    rc = check_ws(wsk, trace, ws, ws_bytes);
    if (rc != G10_OK) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w;
    DeviceTrace d;
    const bool buckets = vitality_buckets_supported(trace->num_tensors, trace->num_events);
    // (bucketed formulation with the timeline: its counting kernel clears the difference array and the point masses itself)
    rc = begin_call(wsk, trace, ws, w, d, s, (buckets ? 0 : kZeroCounts) | (to && !buckets ? kZeroDiffPoint : 0));
    if (rc != G10_OK) return rc;
    const bool host = trace->mem == G10_MEM_HOST;
    VitalityBuffers vb;
    if (!host) {
        vb = VitalityBuffers{out->first_use, out->last_use, out->num_uses, out->use_ptr, out->uses, out->uses_cap, out->period_ptr,
                             out->period_tensor, out->period_prev_use, out->period_next_use, out->periods_cap, out->counts};
    } else {
        const int64_t ucap = out->uses_cap < d.E ? out->uses_cap : d.E, pcap = out->periods_cap < d.E ? out->periods_cap : d.E;
        vb = VitalityBuffers{w.first_use, w.last_use, w.num_uses, w.use_ptr, w.uses, ucap, w.period_ptr,
                             w.period_tensor, w.period_prev_use, w.period_next_use, pcap, w.counts};
    }
    // (host traces: the timeline's results stay in the workspace too and are copied out below)
    int64_t *tl_start = to ? (host ? w.start : to->kernel_start_ns) : nullptr, *tl_P = to ? (host ? w.pressure : to->pressure) : nullptr;
    int64_t *tl_pk = to ? (host ? w.peak_bytes : to->peak_bytes) : nullptr, *tl_st = to ? (host ? w.counts + 3 : to->status) : nullptr;
    int32_t *tl_ps = to ? (host ? w.peak_slot : to->peak_slot) : nullptr;
    if (to && buckets) {
        // slot clock; beside it the vitality kernels, the last of which books the tensors' sizes; then the pressure scan alone
        // (k_bk_hist, which runs whenever there are events, checks kernel_ptr; the slot clock, the lighter of the two, clears
        // the difference array and the point masses for the bookings of k_bk_emit)
        CU(launch_slot_clock(d, w, tl_start, s, !(d.E > 0 && d.K > 0), w.diff, w.tl_point));
        vb.tl_cleared = true;
        vb.tl_diff = (ull *)w.diff; vb.tl_point = (ull *)w.tl_point; vb.tl_bytes = d.tensor_bytes; vb.tl_glob = d.tensor_global; vb.tl_K = d.K;
        CU(launch_vitality_buckets(d, w, vb, s, vb.counts + 2, true));
        CU(launch_pressure_scan(d, w, w.tl_point, tl_P, tl_pk, tl_ps, tl_st, s));
    } else if (buckets) CU(launch_vitality_buckets(d, w, vb, s, vb.counts + 2));     // (its last block publishes the status word)
    else {
        CU(launch_vitality(d, w, vb, s));
        CU(launch_publish_status(w, vb.counts + 2, s));
        if (to) CU(launch_timeline_given(d, w, tl_start, vb.first_use, vb.last_use, w.tl_point, tl_P, tl_pk, tl_ps, tl_st, s));
    }
    if (host) {
        int64_t counts[3];
        CU(cudaMemcpyAsync(counts, w.counts, sizeof(counts), cudaMemcpyDeviceToHost, s));
        CU(cudaStreamSynchronize(s));
        std::memcpy(out->counts, counts, sizeof(counts));
        const size_t N = (size_t)d.N;
        const size_t nu = (size_t)(counts[0] < vb.uses_cap ? counts[0] : vb.uses_cap);
        const size_t np = (size_t)(counts[1] < vb.periods_cap ? counts[1] : vb.periods_cap);
        CU(d2h(out->first_use, w.first_use, N, s));
        CU(d2h(out->last_use, w.last_use, N, s));
        CU(d2h(out->num_uses, w.num_uses, N, s));
        CU(d2h(out->use_ptr, w.use_ptr, N + 1, s));
        CU(d2h(out->period_ptr, w.period_ptr, N + 1, s));
        CU(d2h(out->uses, w.uses, nu, s));
        CU(d2h(out->period_tensor, w.period_tensor, np, s));
        CU(d2h(out->period_prev_use, w.period_prev_use, np, s));
        CU(d2h(out->period_next_use, w.period_next_use, np, s));
        if (to) {
            CU(d2h(to->kernel_start_ns, w.start, (size_t)d.K + 1, s));
            CU(d2h(to->pressure, w.pressure, (size_t)d.K, s));
            CU(d2h(to->peak_bytes, w.peak_bytes, 1, s));
            CU(d2h(to->peak_slot, w.peak_slot, 1, s));
            CU(d2h(to->status, w.counts + 3, 1, s));
        }
        CU(cudaStreamSynchronize(s));
    }
    return G10_OK;
}

int32_t g10_pressure_timeline(const g10_trace *trace, g10_timeline_out *out, void *ws, size_t ws_bytes, void *stream)
{
    int32_t rc = check_trace(trace);
    if (rc != G10_OK) return rc;
    if (!out || !out->kernel_start_ns || !out->peak_bytes || !out->peak_slot || !out->status) return G10_ERR_ARG;
    if (trace->num_kernels > 0 && !out->pressure) return G10_ERR_ARG;
    rc = check_ws(G10_WS_TIMELINE, trace, ws, ws_bytes);
    if (rc != G10_OK) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w;
    DeviceTrace d;
    if ((out->first_use == nullptr) != (out->last_use == nullptr)) return G10_ERR_ARG;
    const bool given = out->first_use != nullptr;          // first / last use from the caller's vitality analysis
    if (given && trace->mem != G10_MEM_DEVICE) return G10_ERR_ARG;
    rc = begin_call(G10_WS_TIMELINE, trace, ws, w, d, s, given ? 0 : kZeroPairs);
    if (rc != G10_OK) return rc;
    const bool host = trace->mem == G10_MEM_HOST;
    int64_t *start = host ? w.start : out->kernel_start_ns;
    int64_t *P = host ? w.pressure : out->pressure;
    int64_t *pk = host ? w.peak_bytes : out->peak_bytes;
    int32_t *ps = host ? w.peak_slot : out->peak_slot;
    int64_t *st = host ? w.counts + 2 : out->status;
    if (given) {
        // (difference array and point masses sit next to each other: one memset; the pair array is not used)
        CU(cudaMemsetAsync(w.diff, 0, (size_t)((char *)(w.tl_point + d.K) - (char *)w.diff), s));
        CU(launch_timeline_given(d, w, start, out->first_use, out->last_use, w.tl_point, P, pk, ps, st, s));
    } else {
        CU(launch_timeline_pairs(d, w, start, w.tl_pair, w.tl_point, P, pk, ps, st, s));  // (its last block publishes the status word)
    }
    if (host) {
        CU(d2h(out->kernel_start_ns, w.start, (size_t)d.K + 1, s));
        CU(d2h(out->pressure, w.pressure, (size_t)d.K, s));
        CU(d2h(out->peak_bytes, w.peak_bytes, 1, s));
        CU(d2h(out->peak_slot, w.peak_slot, 1, s));
        CU(d2h(out->status, w.counts + 2, 1, s));
        CU(cudaStreamSynchronize(s));
    }
    return G10_OK;
}

int32_t g10_candidate_geometry(int64_t K, int64_t Pn, const int64_t *kernel_start_ns, const int64_t *tensor_bytes,
                               const int32_t *period_tensor, const int32_t *period_prev_use, const int32_t *period_next_use,
                               uint64_t host_bw, uint64_t ssd_bw, g10_geometry_out *out, void *stream)
{
    if (K < 0 || Pn < 0 || host_bw == 0 || ssd_bw == 0 || !out) return G10_ERR_ARG;
    if (Pn == 0) return G10_OK;
    if (!kernel_start_ns || !tensor_bytes || !period_tensor || !period_prev_use || !period_next_use) return G10_ERR_ARG;
    if (!out->transfer_ns || !out->absent_first || !out->absent_last) return G10_ERR_ARG;
    CU(launch_geometry(K, Pn, nullptr, kernel_start_ns, tensor_bytes, period_tensor, period_prev_use, period_next_use, host_bw, ssd_bw,
                       Pn, out->transfer_ns, out->absent_first, out->absent_last, (cudaStream_t)stream));
    return G10_OK;
}

int32_t g10_emit_instructions(int64_t K, int64_t N, const int32_t *first_use, const int32_t *last_use, const int64_t *tensor_bytes,
                              const uint8_t *tensor_global, const int64_t *kernel_start_ns, int64_t n, const g10_migration *migrations,
                              const int64_t *new_prefetch_issue_ns, g10_emit_out *out, void *ws, size_t ws_bytes, void *stream)
{
    if (K < 0 || N < 0 || n < 0 || !out || !out->inst_ptr || !out->counts || !kernel_start_ns) return G10_ERR_ARG;
    const int64_t lim = ((int64_t)1 << 31) - 1;
    if (K >= lim || N >= lim || n >= lim) return G10_ERR_LIMIT;
    if (N > 0 && (!first_use || !last_use || !tensor_bytes)) return G10_ERR_ARG;
    if (n > 0 && !migrations) return G10_ERR_ARG;
    if (out->instructions_cap < 0 || (out->instructions_cap > 0 && !out->instructions)) return G10_ERR_ARG;
    int bw = 0, nb = 0;
    ull magic = 0;
    if (!emit_choose_buckets(K, 2 * N + 2 * n, 0, &bw, &nb, &magic)) return G10_ERR_LIMIT;
    EmitLaunch L;
    char *zb = nullptr;
    size_t zbytes = 0;
    const size_t need = carve_emit(nullptr, N, n, L, &zb, &zbytes);
    if (!ws || ((uintptr_t)ws % kAlign) != 0 || ws_bytes < need) return G10_ERR_WORKSPACE;
    carve_emit(ws, N, n, L, &zb, &zbytes);
    cudaStream_t s = (cudaStream_t)stream;
    CU(cudaMemsetAsync(zb, 0, zbytes, s));
    L.K = K; L.N = N; L.n = n; L.first_use = first_use; L.last_use = last_use; L.bytes = tensor_bytes; L.glob = tensor_global;
    L.start = kernel_start_ns; L.mig = migrations; L.new_issue = new_prefetch_issue_ns;
    L.inst_ptr = out->inst_ptr; L.inst = out->instructions; L.inst_cap = out->instructions_cap; L.counts = out->counts;
    CU(launch_emit(L, s));
    Workspace w;
    std::memset(&w, 0, sizeof(w));
    w.status = L.status;
    CU(launch_publish_status(w, out->counts + 1, s));
    return G10_OK;
}

int32_t g10_characterize(int64_t K, int64_t N, const int64_t *use_ptr, const int32_t *uses, const int64_t *tensor_bytes,
                         const int64_t *kernel_start_ns, int64_t Pn, const int32_t *period_tensor, const int32_t *period_prev_use,
                         const int32_t *period_next_use, uint64_t host_bw, uint64_t ssd_bw, g10_stats_out *out, void *stream)
{
    if (K < 0 || N < 0 || Pn < 0 || host_bw == 0 || ssd_bw == 0 || !out) return G10_ERR_ARG;
    const int64_t lim = ((int64_t)1 << 31) - 1;
    if (K >= lim || N >= lim || Pn >= lim) return G10_ERR_LIMIT;
    if (!out->len_hist || !out->size_len_hist || !out->hide || !out->summary || (K > 0 && !out->active_bytes)) return G10_ERR_ARG;
    if (N > 0 && (!use_ptr || !tensor_bytes)) return G10_ERR_ARG;
    if (Pn > 0 && (!kernel_start_ns || !tensor_bytes || !period_tensor || !period_prev_use || !period_next_use)) return G10_ERR_ARG;
    CU(launch_characterize(K, N, use_ptr, uses, tensor_bytes, kernel_start_ns, Pn, period_tensor, period_prev_use, period_next_use,
                           host_bw, ssd_bw, out->active_bytes, out->len_hist, out->size_len_hist, out->hide, out->summary,
                           (cudaStream_t)stream));
    return G10_OK;
}

int32_t g10_schedule_prefetch(int64_t K, int64_t n, const g10_migration *migrations, const int64_t *kernel_start_ns,
                              const int64_t *tensor_bytes, uint64_t gpu_capacity_bytes, g10_prefetch_out *out, void *ws, size_t ws_bytes,
                              void *stream)
{
    if (K < 0 || n < 0 || !out || !out->summary) return G10_ERR_ARG;
    if (K >= (((int64_t)1 << 31) - 1) || n >= (((int64_t)1 << 31) - 1)) return G10_ERR_LIMIT;
    if (K > 0 && !out->pressure) return G10_ERR_ARG;
    if (n > 0 && (!migrations || !kernel_start_ns || !tensor_bytes || !out->order || !out->new_absent_last || !out->new_prefetch_issue_ns))
        return G10_ERR_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    PrefetchScratch p{};
    if (ws) {                                      // (without a workspace one block does the pass)
        if (((uintptr_t)ws & (kAlign - 1)) != 0) return G10_ERR_WORKSPACE;
        PrefetchScratch probe;
        size_t zbytes = 0;
        if (carve_prefetch(nullptr, n, probe, &zbytes) > ws_bytes) return G10_ERR_WORKSPACE;
        carve_prefetch(ws, n, p, &zbytes);
        CU(cudaMemsetAsync(ws, 0, zbytes, s));
    }
    CU(launch_schedule_prefetch(K, n, migrations, kernel_start_ns, tensor_bytes, gpu_capacity_bytes, out->pressure, out->order,
                                out->new_absent_last, out->new_prefetch_issue_ns, out->summary, p, s));
    return G10_OK;
}

int32_t g10_plan_cyclic(const g10_trace *trace, uint64_t gpu_capacity_bytes, uint64_t host_bw, uint64_t ssd_bw,
                        const g10_options *options, g10_plan_out *out, void *ws, size_t ws_bytes, void *stream)
{
    int32_t rc = check_trace(trace);
    if (rc != G10_OK) return rc;
    if (host_bw == 0 || ssd_bw == 0 || !out || !out->summary) return G10_ERR_ARG;
    if (out->migrations_cap < 0 || (out->migrations_cap > 0 && !out->migrations)) return G10_ERR_ARG;
    if (trace->num_kernels > 0 && !out->final_pressure) return G10_ERR_ARG;
    if (options && options->max_iterations < 0) return G10_ERR_ARG;
    rc = check_ws(G10_WS_PLAN, trace, ws, ws_bytes);
    if (rc != G10_OK) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w;
    DeviceTrace d;
    const bool buckets = vitality_buckets_supported(trace->num_tensors, trace->num_events);
    // (the planner state in global memory is cleared too: a trace too large for the single-block planner is planned there)
    rc = begin_call(G10_WS_PLAN, trace, ws, w, d, s, (buckets ? 0 : kZeroCounts) | kZeroDiff | kZeroState);
    if (rc != G10_OK) return rc;
    VitalityBuffers vb{w.first_use, w.last_use, w.num_uses, w.use_ptr, w.uses, d.E, w.period_ptr,
                       w.period_tensor, w.period_prev_use, w.period_next_use, d.E, w.counts};
    PlanParams pp;
    pp.gpu_capacity_bytes = gpu_capacity_bytes; pp.host_bw = host_bw; pp.ssd_bw = ssd_bw;
    pp.host_capacity_bytes = options ? options->host_capacity_bytes : 0;
    pp.max_iterations = options ? options->max_iterations : 0;
    pp.flags = 0;
    const bool host = trace->mem == G10_MEM_HOST;
    pp.migrations = host ? w.migrations : out->migrations;
    pp.migrations_cap = host ? (out->migrations_cap < d.E ? out->migrations_cap : d.E) : out->migrations_cap;
    pp.final_pressure = host ? w.pressure : out->final_pressure;
    pp.summary = host ? w.summary : out->summary;
    CU(launch_slot_clock(d, w, w.start, s));
    CU(buckets ? launch_vitality_buckets(d, w, vb, s) : launch_vitality(d, w, vb, s));
    CU(launch_pressure(d, w, w.first_use, w.last_use, false, pp.final_pressure, w.peak_bytes, w.peak_slot, s));
    CU(launch_cyclic_prepare(d, w, s));
    CU(launch_geometry(2 * d.K, d.E, w.counts + 1, w.start2, d.tensor_bytes, w.period_tensor, w.period_prev_use, w.period_next_use,
                       host_bw, ssd_bw, d.E > 0 ? d.E : 1, w.geo_t, w.geo_a, w.geo_b, s));
    CU(launch_plan_cyclic(d, w, pp, s));
    CU(launch_publish_status_or(w, pp.summary + 7, s));
    if (host) {
        int64_t summary[8];
        CU(cudaMemcpyAsync(summary, w.summary, sizeof(summary), cudaMemcpyDeviceToHost, s));
        CU(cudaStreamSynchronize(s));
        std::memcpy(out->summary, summary, sizeof(summary));
        const size_t nm = (size_t)(summary[0] < pp.migrations_cap ? (summary[0] > 0 ? summary[0] : 0) : pp.migrations_cap);
        CU(d2h(out->migrations, w.migrations, nm, s));
        CU(d2h(out->final_pressure, w.pressure, (size_t)d.K, s));
        CU(cudaStreamSynchronize(s));
    }
    return G10_OK;
}

int32_t g10_plan_batch(const g10_trace *trace, int32_t V, const g10_variant *variants, int64_t max_iterations, g10_batch_out *out,
                       void *ws, size_t ws_bytes, void *stream)
{
    int32_t rc = check_trace(trace);
    if (rc != G10_OK) return rc;
    if (trace->mem != G10_MEM_DEVICE || !variants || !out || !out->summary || !out->stability || max_iterations < 0) return G10_ERR_ARG;
    if (V < 1 || V > kMaxVariants) return G10_ERR_LIMIT;
    if (out->migrations_cap < 0 || (out->migrations_cap > 0 && !out->migrations)) return G10_ERR_ARG;
    if (trace->num_kernels > 0 && !out->final_pressure) return G10_ERR_ARG;
    std::vector<BatchVariant> bv((size_t)V);
    for (int32_t v = 0; v < V; ++v) {
        if (variants[v].host_bw == 0 || variants[v].ssd_bw == 0) return G10_ERR_ARG;
        bv[v].kernel_ns = variants[v].kernel_ns ? variants[v].kernel_ns : trace->kernel_ns;
        bv[v].cap = variants[v].gpu_capacity_bytes; bv[v].host_bw = variants[v].host_bw; bv[v].ssd_bw = variants[v].ssd_bw;
        bv[v].host_capacity = variants[v].host_capacity_bytes;
    }
    rc = check_ws(G10_WS_BATCH, trace, ws, ws_bytes);
    if (rc != G10_OK) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w;
    DeviceTrace d;
    const bool buckets = vitality_buckets_supported(trace->num_tensors, trace->num_events);
    rc = begin_call(G10_WS_BATCH, trace, ws, w, d, s, (buckets ? 0 : kZeroCounts) | kZeroDiff);
    if (rc != G10_OK) return rc;
    CU(cudaMemcpyAsync(w.batch_variants, bv.data(), sizeof(BatchVariant) * (size_t)V, cudaMemcpyHostToDevice, s));
    VitalityBuffers vb{w.first_use, w.last_use, w.num_uses, w.use_ptr, w.uses, d.E, w.period_ptr,
                       w.period_tensor, w.period_prev_use, w.period_next_use, d.E, w.counts};
    PlanParams pp;
    pp.gpu_capacity_bytes = 0; pp.host_bw = 1; pp.ssd_bw = 1; pp.host_capacity_bytes = 0;      // per variant, on the device
    pp.max_iterations = max_iterations; pp.flags = 0;
    pp.migrations = out->migrations; pp.migrations_cap = out->migrations_cap;
    pp.final_pressure = out->final_pressure; pp.summary = out->summary;
    CU(launch_slot_clock(d, w, w.start, s));                    // validates kernel_ptr and the trace's own durations
    CU(buckets ? launch_vitality_buckets(d, w, vb, s) : launch_vitality(d, w, vb, s));
    CU(launch_pressure(d, w, w.first_use, w.last_use, false, w.pressure, w.peak_bytes, w.peak_slot, s));
    CU(launch_plan_variants(d, w, pp, V, out->stability, s));
    // One block per variant needs the trace to fit the shared memory of one SM, which only the device can tell (the
    // number of periods is counted there).  Variant 0 says so: if it could not be planned, the variants are planned one
    // after the other by the planners that use the whole GPU.  Asking costs one small copy and a synchronisation.
    int64_t first[8];
    CU(cudaMemcpyAsync(first, out->summary, sizeof(first), cudaMemcpyDeviceToHost, s));
    CU(cudaStreamSynchronize(s));
    if (!(first[2] == -1 && (first[7] & G10_DEV_BATCH_UNFIT))) return G10_OK;
    CU(launch_publish_status(w, w.counts + 3, s));              // what trace validation found: folded into every variant at the end
    for (int32_t v = 0; v < V; ++v) {
        CU(cudaMemsetAsync(w.zero_begin, 0, w.zero_bytes, s));
        CU(cudaMemsetAsync(w.busy, 0, w.state_bytes, s));
        DeviceTrace dv = d;
        dv.kernel_ns = bv[v].kernel_ns;
        PlanParams pv;
        pv.gpu_capacity_bytes = bv[v].cap; pv.host_bw = bv[v].host_bw; pv.ssd_bw = bv[v].ssd_bw; pv.host_capacity_bytes = bv[v].host_capacity;
        pv.max_iterations = max_iterations; pv.flags = 0;
        pv.migrations = out->migrations ? out->migrations + (size_t)v * (size_t)out->migrations_cap : nullptr;
        pv.migrations_cap = out->migrations_cap;
        pv.final_pressure = out->final_pressure + (size_t)v * (size_t)d.K;
        pv.summary = out->summary + (size_t)v * 8;
        CU(launch_slot_clock(dv, w, w.start, s));               // this variant's clock (and the check of its durations)
        if (d.K > 0) CU(cudaMemcpyAsync(pv.final_pressure, w.pressure, sizeof(int64_t) * (size_t)d.K, cudaMemcpyDeviceToDevice, s));
        CU(launch_geometry(d.K, d.E, w.counts + 1, w.start, d.tensor_bytes, w.period_tensor, w.period_prev_use, w.period_next_use,
                           pv.host_bw, pv.ssd_bw, d.E > 0 ? d.E : 1, w.geo_t, w.geo_a, w.geo_b, s));
        CU(launch_plan_loop(dv, w, pv, s));
        CU(launch_publish_status(w, pv.summary + 7, s));
    }
    CU(launch_batch_finish(d, w, pp, V, out->stability, (const ull *)(w.counts + 3), s));
    return G10_OK;
}

int32_t g10_plan_migrations(const g10_trace *trace, uint64_t gpu_capacity_bytes, uint64_t host_bw, uint64_t ssd_bw,
                            const g10_options *options, g10_plan_out *out, void *ws, size_t ws_bytes, void *stream)
{
    int32_t rc = check_trace(trace);
    if (rc != G10_OK) return rc;
    if (host_bw == 0 || ssd_bw == 0 || !out || !out->summary) return G10_ERR_ARG;
    if (out->migrations_cap < 0 || (out->migrations_cap > 0 && !out->migrations)) return G10_ERR_ARG;
    if (trace->num_kernels > 0 && !out->final_pressure) return G10_ERR_ARG;
    if (options && options->max_iterations < 0) return G10_ERR_ARG;
    rc = check_ws(G10_WS_PLAN, trace, ws, ws_bytes);
    if (rc != G10_OK) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w;
    DeviceTrace d;
    const uint32_t flags = options ? options->flags : 0;
    const bool buckets = !(flags & G10_FLAG_RESCORE_ALL) && vitality_buckets_supported(trace->num_tensors, trace->num_events);
    rc = begin_call(G10_WS_PLAN, trace, ws, w, d, s, (buckets ? 0 : kZeroCounts) | kZeroDiff | (plan_keeps_state_on_chip(trace->num_kernels, trace->num_events, flags) ? 0 : kZeroState));
    if (rc != G10_OK) return rc;
    const bool host = trace->mem == G10_MEM_HOST;
#ifdef G10_TEST_HOOKS
    if (flags & G10_FLAG_TEST_SKIP_ARRIVAL) {        // (test build: block 1 skips its first barrier arrival, waits give up after 1 ms)
        static const unsigned hook = 2u;
        CU(cudaMemcpyAsync(&((GridBarrier *)w.barrier)->pad, &hook, sizeof(hook), cudaMemcpyHostToDevice, s));
    }
#endif
    VitalityBuffers vb{w.first_use, w.last_use, w.num_uses, w.use_ptr, w.uses, d.E, w.period_ptr,
                       w.period_tensor, w.period_prev_use, w.period_next_use, d.E, w.counts};
    PlanParams pp;
    pp.gpu_capacity_bytes = gpu_capacity_bytes; pp.host_bw = host_bw; pp.ssd_bw = ssd_bw;
    pp.host_capacity_bytes = options ? options->host_capacity_bytes : 0;
    pp.max_iterations = options ? options->max_iterations : 0;
    pp.flags = options ? options->flags : 0;
    pp.migrations = host ? w.migrations : out->migrations;
    pp.migrations_cap = host ? (out->migrations_cap < d.E ? out->migrations_cap : d.E) : out->migrations_cap;
    pp.final_pressure = host ? w.pressure : out->final_pressure;
    pp.summary = host ? w.summary : out->summary;
    // optional caller-owned events at the stage boundaries
    auto mark = [&](int stage) -> cudaError_t {
        if (options && options->stage_events && stage < options->num_stage_events && options->stage_events[stage])
            return cudaEventRecord((cudaEvent_t)options->stage_events[stage], s);
        return cudaSuccess;
    };
    CU(mark(0));
    CU(launch_slot_clock(d, w, w.start, s));
    CU(buckets ? launch_vitality_buckets(d, w, vb, s) : launch_vitality(d, w, vb, s));
    CU(mark(1));
    CU(launch_pressure(d, w, w.first_use, w.last_use, false, pp.final_pressure, w.peak_bytes, w.peak_slot, s));
    CU(mark(2));
    CU(launch_geometry(d.K, d.E, w.counts + 1, w.start, d.tensor_bytes, w.period_tensor, w.period_prev_use, w.period_next_use,
                       host_bw, ssd_bw, d.E > 0 ? d.E : 1, w.geo_t, w.geo_a, w.geo_b, s));
    CU(mark(3));
    CU(launch_plan_loop(d, w, pp, s));
    CU(mark(4));
    CU(launch_publish_status(w, pp.summary + 7, s));
    if (host) {
        int64_t summary[8];
        CU(cudaMemcpyAsync(summary, w.summary, sizeof(summary), cudaMemcpyDeviceToHost, s));
        CU(cudaStreamSynchronize(s));
        std::memcpy(out->summary, summary, sizeof(summary));
        const size_t nm = (size_t)(summary[0] < pp.migrations_cap ? summary[0] : pp.migrations_cap);
        CU(d2h(out->migrations, w.migrations, nm, s));
        CU(d2h(out->final_pressure, w.pressure, (size_t)d.K, s));
        CU(cudaStreamSynchronize(s));
    }
    return G10_OK;
}

}  // extern "C"

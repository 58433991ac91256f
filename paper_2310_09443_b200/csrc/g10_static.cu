// g10_pressure_timeline_static: the pressure-timeline call for hosts that must not allocate.
//
// Some programs that embed this library cannot give it a workspace at the moment they need a timeline:
// a process that handed all device memory to its own pool at start-up and exposes no allocator to plug-ins,
// or a code path on which cudaMalloc / cudaFree are off limits because both may synchronise the whole
// device.  For those callers the scratch memory of the timeline pass lives in the library image itself, in
// the fixed-size device array below.  Every GPU that loads the library carries that array (1.5 MiB) until
// the process exits, whether or not this entry point is ever called.
#include <mutex>

#include "g10_internal.h"

namespace g10 {
namespace {

constexpr size_t kStaticScratchBytes = 1536 * 1024;
constexpr int kMaxDevices = 64;

// File-scope scratch.  In host code this name is only a handle for cudaGetSymbolAddress; it is not a
// device address and must never be handed to a kernel as one.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// The layout of the call below at the documented maxima, bounded from above (every array rounded up to the workspace
// alignment): it has to fit the array, so that G10_ERR_LIMIT can only mean "trace larger than the documented maxima".
constexpr size_t au(size_t bytes) { return (bytes + kAlign - 1) / kAlign * kAlign; }
constexpr size_t static_layout_bound(size_t K, size_t N)
{
    const size_t tiles = (K + 2047) / 2048 + 1;
    return 2 * au(8)                                                      // status word, event budget
         + 2 * (2 * au(4) + au(4 * tiles) + 2 * au(8 * tiles))           // the two scans' slots
         + 2 * au(8 * 16 * (tiles + 1))                                   // their tagged words, one line per block
         + au(8 * (K + 1)) + 2 * au(4 * N)                                // difference array, first / last use
         + au(8 * tiles) + au(4 * tiles);                                 // per-block maxima
}
static_assert(static_layout_bound(G10_STATIC_MAX_KERNELS, G10_STATIC_MAX_TENSORS) <= kStaticScratchBytes,
              "the static scratch array is too small for the documented maxima");

std::mutex g_setup_mutex;
// Device address of g_static_scratch on each device, once looked up.  It belongs to the context it was looked up in: after
// cudaDeviceReset() (or any other teardown of the primary context) the remembered address is stale, and this entry
// point must not be called again in that process (documented in g10.h).
void *g_scratch_addr[kMaxDevices];

// Looks the array's device address up once per device (with that device current) and remembers it.
cudaError_t scratch_address(void **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (p == nullptr) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

struct Bump {
    char *base;
    size_t off = 0;
    template <typename T>
    T *take(size_t count)
    {
        off = align_up(off);
        T *p = (T *)(base + off);
        off += sizeof(T) * (count ? count : 1);
        return p;
    }
};

void take_scan(Bump &b, ScanSlot &s, size_t tiles)
{
    s.ticket = b.take<unsigned>(1);
    s.done = b.take<unsigned>(1);
    s.flag = b.take<unsigned>(tiles);
    s.agg = b.take<long long>(tiles);
    s.incl = b.take<long long>(tiles);
}

}  // namespace
}  // namespace g10

using namespace g10;

extern "C" int32_t g10_pressure_timeline_static(const g10_trace *trace, g10_timeline_out *out, void *stream)
{
    if (!trace || !out) return G10_ERR_ARG;
    if (trace->mem != G10_MEM_DEVICE) return G10_ERR_ARG;
    const int64_t K = trace->num_kernels, N = trace->num_tensors, E = trace->num_events;
    if (K < 0 || N < 0 || E < 0) return G10_ERR_ARG;
    if (K > G10_STATIC_MAX_KERNELS || N > G10_STATIC_MAX_TENSORS || E >= (((int64_t)1 << 31) - 1)) return G10_ERR_LIMIT;
    if (!trace->kernel_ptr || (E > 0 && !trace->kernel_tensors) || (N > 0 && !trace->tensor_bytes) || (K > 0 && !trace->kernel_ns))
        return G10_ERR_ARG;
    if (E > 0 && (K == 0 || N == 0)) return G10_ERR_ARG;
    if (!out->kernel_start_ns || !out->peak_bytes || !out->peak_slot || !out->status || (K > 0 && !out->pressure)) return G10_ERR_ARG;

    void *base = nullptr;
    if (scratch_address(&base) != cudaSuccess) return G10_ERR_CUDA;

    // Lay the pass's scratch out inside the static array: what must start at zero first.
    Workspace w{};
    Bump b{(char *)base};
    const size_t ktiles = (size_t)tiles_of(K, 2048);
    w.zero_begin = (char *)base;
    w.status = b.take<ull>(1);
    w.event_budget = b.take<ull>(1);
    take_scan(b, w.clock_scan, ktiles);
    take_scan(b, w.pressure_scan, ktiles);
    w.seg_words = b.take<ull>((ktiles + 1) * 16);        // (the scans run at most one block per 4096 kernels: fewer than ktiles)
    w.seg_words2 = b.take<ull>((ktiles + 1) * 16);
    w.diff = b.take<int64_t>((size_t)K + 1);
    w.zero_bytes = align_up(b.off);
    w.first_use = b.take<int32_t>((size_t)N);
    w.last_use = b.take<int32_t>((size_t)N);
    w.tile_max = b.take<int64_t>(ktiles);
    w.tile_slot = b.take<int32_t>(ktiles);
    if (align_up(b.off) > kStaticScratchBytes) return G10_ERR_LIMIT;

    cudaStream_t s = (cudaStream_t)stream;
    // The array still holds whatever the previous call left: clear the part that counts from zero.
    if (cudaMemsetAsync(w.zero_begin, 0, w.zero_bytes, s) != cudaSuccess) return G10_ERR_CUDA;
    DeviceTrace d{K, N, E, trace->kernel_ptr, trace->kernel_tensors, trace->tensor_bytes, trace->kernel_ns, trace->tensor_global};
    if (launch_slot_clock(d, w, out->kernel_start_ns, s) != cudaSuccess) return G10_ERR_CUDA;
    if (launch_first_last(d, w, w.first_use, w.last_use, s) != cudaSuccess) return G10_ERR_CUDA;
    if (launch_pressure(d, w, w.first_use, w.last_use, true, out->pressure, out->peak_bytes, out->peak_slot, s) != cudaSuccess) return G10_ERR_CUDA;
    if (launch_publish_status(w, out->status, s) != cudaSuccess) return G10_ERR_CUDA;
    return G10_OK;
}

// rr_route_noalloc: rr_route for callers that cannot allocate device memory.
//
// rr_route needs a few MB of scratch (per-token candidates, per-tile counters, nominee lists)
// which its caller normally allocates.  Some callers cannot: code that runs inside a
// stream-ordered or real-time section where cudaMalloc's implicit synchronisation is not
// acceptable, plug-ins that are handed tensors but no allocator, or processes whose memory pool
// is already fully committed.  For them the scratch lives in a fixed array inside the library
// image.  Every GPU that loads librr.so holds these kStaticScratchBytes until the process exits.
//
// Host code must not pass the array's name to a kernel: on the host that name is only a
// stand-in for the symbol.  Its device address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and that address is what the kernels get.
#include <mutex>

#include "rr_common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 4u << 20;  // 4 MiB, e.g. T = 65536, E = 64, k = 2 fits
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_route_scratch[kStaticScratchBytes];

std::mutex g_mutex;
void *g_scratch_addr[kMaxDevices];  // device address of g_route_scratch on each device, once known

// Device address of the static scratch on the current device (looked up on first use).
cudaError_t static_scratch(void **ptr)
{
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        err = cudaGetSymbolAddress(&p, g_route_scratch);
        if (err != cudaSuccess) return err;
        g_scratch_addr[dev] = p;
    }
    *ptr = g_scratch_addr[dev];
    return cudaSuccess;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" rr_status rr_route_noalloc(const float *logits, int T, int E, int k, int capacity, int G, unsigned mode,
                                      const rr_route_tables *out, void *status, void *stream)
{
    // the argument rules of rr_route; the modes that change the scratch layout per call are left out
    rr_status rc = rr::check_route_shape(T, E, k, capacity, G, mode);
    if (rc) return rc;
    if (mode & ~(RR_IR | RR_FR)) return RR_ERR_INVALID_ARG;
    rc = rr::check_route_tables(out);
    if (rc) return rc;
    if ((T > 0 && !logits) || !aligned16(logits) || !aligned16(status)) return RR_ERR_INVALID_ARG;

    rr::RouteScratch s;
    if (rr::route_scratch_layout(nullptr, T, E, k, &s, mode, G) > kStaticScratchBytes) return RR_ERR_STATIC_SCRATCH_EXCEEDED;

    void *base = nullptr;
    if (static_scratch(&base) != cudaSuccess) return RR_ERR_CUDA;
    rr::route_scratch_layout(base, T, E, k, &s, mode, G);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (status) {
        s.status = static_cast<int *>(status);  // only this one word of the caller's buffer is touched
    } else if (cudaMemsetAsync(base, 0, sizeof(int), st) != cudaSuccess) {
        // The array keeps the previous call's contents.  What must start at zero: the status word
        // (cleared here when the caller passes none) and the barrier words of the routing kernel, which
        // the kernel itself puts back to zero before it ends; everything else is written before it is read.
        return RR_ERR_CUDA;
    }
    cudaError_t err = rr::launch_route(logits, T, E, k, capacity, G, mode, *out, s, st);
    return err == cudaSuccess ? RR_OK : RR_ERR_CUDA;
}

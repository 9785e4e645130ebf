// st_agreement_noalloc — the agreement measurement (confusion matrix + mean IoU of two one-byte masks)
// for callers that must not allocate device memory.
//
// Who cannot allocate: a serving process that handed all of HBM to its own memory pool at start-up
// (cudaMalloc then simply fails), a latency-critical loop that cannot afford the device-wide
// synchronisation cudaMalloc/cudaFree imply, and code that runs while another thread is capturing a
// CUDA graph in a mode that forbids allocation calls.  The ordinary st_agreement needs a context, and
// creating a context allocates; this variant needs neither.
//
// The 64-bit counters the confusion kernel accumulates into live in a file-scope __device__ array
// instead of cudaMalloc'ed memory.  Every GPU that loads the library holds that array (about 33 KB)
// until the process exits.  All calls share it: it is cleared at the start of every call, and two
// calls whose work overlaps on the GPU (different streams, no ordering between them) would race on it.
#include "../../include/shadowtutor.h"
#include "st_internal.h"

#include <mutex>

namespace {

constexpr int kMaxClasses = ST_NOALLOC_MAX_CLASSES;
constexpr int kMaxDevices = 64;
constexpr size_t kCounters = (size_t)kMaxClasses * kMaxClasses;

// counters [kMaxClasses * kMaxClasses] followed by one word that counts skipped pixels
static __device__ __align__(256) unsigned long long g_agreement_scratch[kCounters + 4];

// In host code `g_agreement_scratch` is only a handle for the runtime, not a device address; the
// address a kernel can use has to be asked for, per device, with that device current.
unsigned long long* g_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_scratch_mutex;

cudaError_t scratch_for_current_device(unsigned long long** out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_agreement_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = (unsigned long long*)ptr;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" st_status st_agreement_noalloc(const uint8_t* pred, const uint8_t* label, int64_t n_pixels,
                                          int32_t n_classes, void* cuda_stream, int64_t* conf_out,
                                          double* miou_out)
{
    if (!pred || !label || !conf_out || !miou_out) return ST_ERR_INVALID_ARG;
    if (n_pixels < 0 || n_classes < 2) return ST_ERR_INVALID_ARG;
    if (n_classes > kMaxClasses) return ST_ERR_UNSUPPORTED;   // beyond the fixed scratch
    unsigned long long* scratch = nullptr;
    if (scratch_for_current_device(&scratch) != cudaSuccess) { cudaGetLastError(); return ST_ERR_CUDA; }
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const size_t cc = (size_t)n_classes * n_classes;
    // the array keeps the previous call's counts: clear what this call accumulates into
    if (cudaMemsetAsync(scratch, 0, (cc + 4) * sizeof(unsigned long long), s) != cudaSuccess) return ST_ERR_CUDA;
    st::launch_confusion(label, pred, n_pixels, n_classes, scratch, (unsigned int*)(scratch + cc), s);
    st::launch_miou(scratch, n_classes, miou_out, s);
    if (cudaGetLastError() != cudaSuccess) return ST_ERR_CUDA;
    if (cudaMemcpyAsync(conf_out, scratch, cc * sizeof(unsigned long long), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return ST_ERR_CUDA;
    return ST_OK;
}

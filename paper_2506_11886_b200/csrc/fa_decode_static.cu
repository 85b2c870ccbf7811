// fa_decode_attention_static: the decode call for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at all: a serving engine that
// hands its whole HBM budget to the KV-cache pool at start-up and gives plug-ins no
// scratch, or a latency-critical decode loop in which an allocation (which
// synchronises the device) is forbidden after warm-up.  For them the split / merge
// scratch of fa_decode_attention lives here, in a fixed array that is part of the
// loaded module: every GPU that loads the library holds kStaticWsBytes of it until
// the process exits.
//
// The array's name is a host-side stand-in in host code, not a device address, so
// the address is asked for with cudaGetSymbolAddress, once per device with that
// device current, and that pointer is what the kernels receive.
#include <mutex>

#include "fa_common.cuh"

namespace fa {

constexpr size_t kStaticWsBytes = size_t(8) << 20;   // 8 MiB per GPU
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

static std::mutex g_static_mu;
static char* g_static_ptr[kMaxDevices] = {nullptr};

// Device address of g_static_ws on the current device (looked up on first use).
static cudaError_t static_ws_of_current_device(char** out) {
    int dev = -1;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        err = cudaGetSymbolAddress(&p, g_static_ws);
        if (err != cudaSuccess) return err;
        if (!p) return cudaErrorInvalidSymbol;
        g_static_ptr[dev] = static_cast<char*>(p);
    }
    *out = g_static_ptr[dev];
    return cudaSuccess;
}

}  // namespace fa

extern "C" {

size_t fa_static_workspace_limit(void) { return fa::kStaticWsBytes; }

fa_status fa_decode_attention_static(const fa_layout* layout, const fa_cache* cache, const void* q, void* out,
                                     void* stream) {
    size_t need = 0;
    fa_status st = fa_workspace_bytes(layout, &need);      // also validates the layout; host only
    if (st != FA_OK) return st;
    if (need > fa::kStaticWsBytes) return FA_ERR_WORKSPACE; // this layout needs more scratch than the fixed array has
    char* ws = nullptr;
    if (fa::static_ws_of_current_device(&ws) != cudaSuccess) return FA_ERR_CUDA;
    // The barrier counters at the head of the scratch (its first 4 KiB) must be zero when the decode
    // kernels start.  A call that ends normally leaves them zero, a call that gave up on a bounded wait
    // (FA_ERR_TIMEOUT) does not, and the caller has no pointer to this array to clear it with
    // fa_workspace_init: so every call clears them itself, in stream order, in front of its kernels.
    // A memset allocates nothing.  Everything else in the array is written before it is read.
    if (cudaMemsetAsync(ws, 0, 4096, static_cast<cudaStream_t>(stream)) != cudaSuccess) return FA_ERR_CUDA;
    return fa_decode_attention(layout, cache, q, out, ws, fa::kStaticWsBytes, stream);
}

}  // extern "C"

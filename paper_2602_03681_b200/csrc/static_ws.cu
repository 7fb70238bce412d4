// natsl_hybrid_fwd_static: the forward of the layer for callers that must not allocate.
//
// Some hosts of this library cannot obtain device memory themselves: a plug-in running inside
// an inference server whose memory pool it does not own, or code on a latency-critical path
// where a cudaMalloc (which synchronises the device) is not acceptable.  For them the scratch
// memory the forward needs lives in a fixed array inside this library instead of a caller
// workspace.  The price: the array has a modest fixed size, so only small problems fit, and it
// is shared by every call on the device.
#include <mutex>

#include "natsl_internal.h"

namespace {

// Scratch of the forward for problems whose natsl_workspace_size(NATSL_OP_FWD) fits.  Every GPU
// that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_ws[NATSL_STATIC_WS_BYTES];

constexpr int kMaxDevices = 64;
void *g_static_ws_ptr[kMaxDevices] = {};   // device address of g_static_ws, per device
std::mutex g_static_ws_mu;

// In host code `g_static_ws` is only a handle for the runtime, not an address a kernel may use:
// the device address has to be asked for, once per device, with that device current.
// (The array of the CURRENT device: the caller's stream and tensors must belong to it.)
int static_ws_address(void **ptr) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NATSL_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_ws_mu);
    if (!g_static_ws_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) return NATSL_ERR_CUDA;
        g_static_ws_ptr[dev] = p;
    }
    *ptr = g_static_ws_ptr[dev];
    return NATSL_OK;
}

}  // namespace

extern "C" int natsl_hybrid_fwd_static(const void *q, const void *k, const void *v, const float *g,
                                       const float *beta, const uint8_t *route, void *out,
                                       const natsl_params *p, void *stream) {
    size_t need = 0;
    int rc = natsl_workspace_size(p, NATSL_OP_FWD, &need);   // validates shapes, host only
    if (rc != NATSL_OK) return rc;
    if (need > (size_t)NATSL_STATIC_WS_BYTES) return NATSL_ERR_TOO_LARGE;
    void *ws = nullptr;
    rc = static_ws_address(&ws);
    if (rc != NATSL_OK) return rc;
    // natsl_hybrid_fwd clears the status word at the head of the workspace and overwrites every
    // other scratch region before reading it, so stale contents of an earlier call are harmless.
    natsl_params ps = *p;
    ps.flags |= NATSL_SINGLE_STREAM;     // no library-owned stream: nothing is created by this call
    return natsl_hybrid_fwd(q, k, v, g, beta, route, out, &ps, ws, (size_t)NATSL_STATIC_WS_BYTES, stream);
}

// The status word of the built-in scratch of the current device: what natsl_device_status reads
// from a caller's workspace.  Allocates nothing.
extern "C" int natsl_static_status(void *stream) {
    void *ws = nullptr;
    const int rc = static_ws_address(&ws);
    if (rc != NATSL_OK) return rc;
    return natsl_device_status(ws, stream);
}

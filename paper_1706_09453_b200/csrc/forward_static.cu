// bnn_forward_static: the whole forward pass for callers that cannot allocate device memory.
//
// bnn_forward needs scratch (two ping-pong buffers for the activations between layers) and
// expects the caller to bring it.  Some callers cannot: a decoder thread that must never
// block (cudaMalloc synchronises the whole device), a plug-in inside a host program whose
// memory budget is fixed at start-up, a process that has handed all device memory to another
// pool.  For them the scratch lives here, in a fixed array inside the library image: every
// GPU that loads the library holds these bytes until the process exits, whether or not this
// entry point is ever called, which is why the array is kept modest.
#include "bnn_common.cuh"

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime, not a device
// address: the address is obtained once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_workspace[BNN_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
void* g_workspace_addr[kMaxDevices] = {};

// Device address of the array on the current device (nullptr on failure).
void* static_workspace_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    if (!g_workspace_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess) return nullptr;
        g_workspace_addr[dev] = p;
    }
    return g_workspace_addr[dev];
}

}  // namespace

extern "C" int bnn_forward_static(const bnn_model* model, const float* X, int ldx, int M,
                                  float* logp, int ldo, void* stream) {
    if (!model) return BNN_ERR_NULL;
    if (M < 1) return BNN_ERR_SHAPE;
    const size_t need = bnn_forward_min_workspace_bytes(model, M);
    // need == 0 means the model itself is invalid: bnn_forward reports which way.
    if (need > (size_t)BNN_STATIC_WORKSPACE_BYTES) return BNN_ERR_WORKSPACE;
    void* ws = static_workspace_for_current_device();
    if (!ws) return BNN_ERR_CUDA;
    // Nothing has to be cleared: every word of the scratch a layer reads was written by the
    // layer before it within this same call (readers ignore pitch words and pad bits).
    return bnn_forward(model, X, ldx, M, logp, ldo, ws, BNN_STATIC_WORKSPACE_BYTES, nullptr, stream);
}

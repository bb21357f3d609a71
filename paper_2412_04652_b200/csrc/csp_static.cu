// csp_prune_layer_static: Algorithm 1 for callers that cannot provide scratch memory of their own.
//
// The scratch that csp_prune_layer takes as a caller-allocated workspace (status word, the two score
// vectors, the index list) lives here in a fixed array that is part of the library image, so the
// call needs no allocator at all.  Every GPU that loads the library holds kStaticWorkspaceBytes of
// device memory for it until the process exits.
#include <mutex>

#include "csp_internal.cuh"

namespace {

constexpr size_t kStaticWorkspaceBytes = size_t(8) << 20;   // 8 MiB

// Device-side storage.  In host code this name is only a handle for cudaGetSymbolAddress, never a
// device address to hand to a kernel.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

constexpr int kMaxDevices = 64;
void* g_device_address[kMaxDevices] = {};
std::mutex g_setup_mutex;

// Looks up, once per device and with that device current, where the array lives on it.  The address is
// remembered for the life of the process; a cudaDeviceReset, which unloads the library's device image,
// is not supported between calls.
csp_status static_workspace(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return CSP_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_device_address[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || !ptr) { cudaGetLastError(); return CSP_ERR_CUDA; }
        g_device_address[dev] = ptr;
    }
    *out = g_device_address[dev];
    return CSP_OK;
}

}  // namespace

extern "C" {

size_t csp_static_workspace_limit(void) { return kStaticWorkspaceBytes; }

csp_status csp_prune_layer_static(const csp_params* p, csp_tensor q_win, csp_tensor k, csp_tensor v,
                                  const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                                  const int32_t* seq_lens, const int32_t* budgets,
                                  const int32_t* total_budget_or_null, const float* lse_or_null,
                                  csp_tensor k_out, csp_tensor v_out, uint8_t* mod_out, int32_t* n_out,
                                  int32_t* dev_status_out_or_null, void* cuda_stream) {
    // Everything the host can reject is rejected before the address lookup and before anything is enqueued:
    // parameters, null pointers, alignment, the architecture, then the size of the scratch.
    csp_status st = csp::check_prune_layer_args(p, q_win, k, v, modality, seq_lens, budgets, k_out, v_out, n_out);
    if (st != CSP_OK) return st;
    const size_t need = csp_workspace_bytes(p);
    if (need == 0) return CSP_ERR_UNSUPPORTED;
    if (need > kStaticWorkspaceBytes) return CSP_ERR_WORKSPACE;   // shapes beyond the built-in scratch
    void* ws = nullptr;
    st = static_workspace(&ws);
    if (st != CSP_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps whatever the previous call left: the status area must start at zero
    if (cudaMemsetAsync(ws, 0, csp::kStatusBytes, stream) != cudaSuccess) { cudaGetLastError(); return CSP_ERR_CUDA; }
    st = csp_prune_layer(p, q_win, k, v, modality, mod_stride_b, mod_stride_h, seq_lens, budgets,
                         total_budget_or_null, lse_or_null, k_out, v_out, mod_out, n_out, nullptr, nullptr, nullptr,
                         ws, need, cuda_stream);
    if (st != CSP_OK) return st;
    if (dev_status_out_or_null &&
        cudaMemcpyAsync(dev_status_out_or_null, ws, sizeof(int32_t), cudaMemcpyDeviceToDevice, stream) != cudaSuccess) {
        cudaGetLastError();
        return CSP_ERR_CUDA;
    }
    return CSP_OK;
}

}  // extern "C"

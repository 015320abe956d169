// Allocation-free variant of the W4A4 linear: the scratch the linear needs (the expanded int8
// activations and the per-row bias sums) lives in a fixed array inside the library image instead of
// a caller-provided workspace.
#include <mutex>

#include "common.cuh"

namespace sqap {

// The scratch itself. Every GPU that loads the library carries one copy until the process exits.
static __device__ __align__(256) unsigned char g_static_workspace[SQAP_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
static void* g_static_ptr[kMaxDevices] = {};
static std::mutex g_static_mutex;

// In host code `g_static_workspace` is only a stand-in for the symbol, not an address a kernel can
// use; the device address has to be asked for, once per device, with that device current.
static sqap_status static_workspace_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        note_cuda_error(e);
        return SQAP_ERR_CUDA;
    }
    if (dev < 0 || dev >= kMaxDevices) return SQAP_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_workspace);
        if (e != cudaSuccess || !p) {
            note_cuda_error(e);
            return SQAP_ERR_CUDA;
        }
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return SQAP_OK;
}

}  // namespace sqap

extern "C" sqap_status sqap_w4a4_linear_static(const uint8_t* q_packed, const float* act_scales, int M,
                                               const sqap_weights* w, const sqap_weights* w_up, void* out, int64_t ldo,
                                               int out_dtype, uint32_t flags, void* stream) {
    using namespace sqap;
    if (!w || M < 0) return SQAP_ERR_INVALID;
    if (flags & SQAP_L_REUSE_EXPANDED) return SQAP_ERR_INVALID;  // the shared scratch may have been overwritten
    if (sqap_workspace_bytes(M, w->N, w->K, flags) > static_cast<size_t>(SQAP_STATIC_WORKSPACE_BYTES))
        return SQAP_ERR_TOO_LARGE;
    void* scratch = nullptr;
    sqap_status st = static_workspace_address(&scratch);
    if (st != SQAP_OK) return st;
    // Nothing in the scratch has to start at zero: the expand pass writes every byte the GEMM reads.
    return sqap_w4a4_linear(q_packed, act_scales, M, w, w_up, out, ldo, out_dtype, flags, scratch,
                            SQAP_STATIC_WORKSPACE_BYTES, stream);
}

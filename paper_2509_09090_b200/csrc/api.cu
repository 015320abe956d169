// Status plumbing and the host-only helpers of the C ABI.
#include <atomic>
#include <cmath>

#include "common.cuh"

namespace sqap {

static thread_local int t_last_cuda_error = 0;
static std::atomic<int64_t> g_launches{0};

// One status word per device that loads the library; kernels OR an error code into it.
__device__ int g_device_status = 0;

void note_cuda_error(cudaError_t e) { t_last_cuda_error = static_cast<int>(e); }
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

sqap_status check_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        note_cuda_error(e);
        return SQAP_ERR_CUDA;
    }
    return SQAP_OK;
}

static PerDevice<DeviceProps> g_props;

const DeviceProps* device_props() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
        cudaGetLastError();
        return nullptr;
    }
    const DeviceProps* props = nullptr;
    const sqap_status st = g_props.run(
        [dev](DeviceProps* p) {
            cudaError_t e = cudaDeviceGetAttribute(&p->sms, cudaDevAttrMultiProcessorCount, dev);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->cc_major, cudaDevAttrComputeCapabilityMajor, dev);
            // in host code the symbol's name is not a device address: ask for it, with this device current
            if (e == cudaSuccess) e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p->status_word), g_device_status);
            if (e != cudaSuccess) {
                note_cuda_error(e);
                cudaGetLastError();
                return SQAP_ERR_CUDA;
            }
            return SQAP_OK;
        },
        &props);
    return st == SQAP_OK ? props : nullptr;
}

int sm_count() {
    const DeviceProps* p = device_props();
    return (p && p->sms > 0) ? p->sms : 148;
}

int* device_status_word() {
    const DeviceProps* p = device_props();
    return p ? p->status_word : nullptr;
}

}  // namespace sqap

extern "C" {

sqap_status sqap_device_status(void* stream) {
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        sqap::note_cuda_error(e);
        return SQAP_ERR_CUDA;
    }
    int v = 0;
    e = cudaMemcpyFromSymbol(&v, sqap::g_device_status, sizeof(int));
    if (e != cudaSuccess) {
        sqap::note_cuda_error(e);
        return SQAP_ERR_CUDA;
    }
    if (v != 0) {
        int zero = 0;
        cudaMemcpyToSymbol(sqap::g_device_status, &zero, sizeof(int));
        return SQAP_ERR_TIMEOUT;
    }
    return SQAP_OK;
}

int sqap_last_cuda_error(void) { return sqap::t_last_cuda_error; }

int64_t sqap_kernel_launch_count(void) { return sqap::g_launches.load(std::memory_order_relaxed); }

const char* sqap_status_string(sqap_status s) {
    switch (s) {
        case SQAP_OK: return "ok";
        case SQAP_ERR_INVALID: return "invalid argument";
        case SQAP_ERR_RANGE: return "value out of range";
        case SQAP_ERR_ALIGN: return "misaligned pointer, stride or size";
        case SQAP_ERR_UNSUPPORTED: return "unsupported shape or option";
        case SQAP_ERR_NOMEM: return "out of memory or workspace too small";
        case SQAP_ERR_CUDA: return "CUDA error";
        case SQAP_ERR_TIMEOUT: return "bounded device wait expired";
        case SQAP_ERR_TOO_LARGE: return "problem too large for the built-in scratch array";
    }
    return "unknown status";
}

// Eq. 2: lambda [u v 1]^T = K [R|t] [x y z 1]^T ; Eq. 3: t_u = floor(u / P_w), t_v = floor(v / P_h).
sqap_status sqap_project_center(const double Kmat[9], const double Rt[12], const double xyz[3], double patch_w,
                                double patch_h, int32_t out_tu_tv[2], int* in_front) {
    if (!Kmat || !Rt || !xyz || !out_tu_tv || !in_front) return SQAP_ERR_INVALID;
    if (!(patch_w > 0.0) || !(patch_h > 0.0)) return SQAP_ERR_INVALID;
    double c[3], p[3];
    for (int r = 0; r < 3; ++r) c[r] = Rt[4 * r] * xyz[0] + Rt[4 * r + 1] * xyz[1] + Rt[4 * r + 2] * xyz[2] + Rt[4 * r + 3];
    for (int r = 0; r < 3; ++r) p[r] = Kmat[3 * r] * c[0] + Kmat[3 * r + 1] * c[1] + Kmat[3 * r + 2] * c[2];
    out_tu_tv[0] = out_tu_tv[1] = 0;
    if (!(p[2] > 0.0)) {
        *in_front = 0;
        return SQAP_OK;
    }
    *in_front = 1;
    out_tu_tv[0] = static_cast<int32_t>(std::floor((p[0] / p[2]) / patch_w));
    out_tu_tv[1] = static_cast<int32_t>(std::floor((p[1] / p[2]) / patch_h));
    return SQAP_OK;
}

}  // extern "C"

// Shared host/device helpers of the sqap library (internal; not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <mutex>

#include "../../include/sqap.h"

namespace sqap {

// Host bookkeeping (api.cu).
void note_cuda_error(cudaError_t e);
void count_launch(int n = 1);
sqap_status check_launch();  // cudaGetLastError -> status

// Pointer to the device status word of the current device (set by kernels whose bounded waits expire).
int* device_status_word();

// What the launch code needs to know about a device, looked up once per device (api.cu; thread-safe).
constexpr int MAX_DEVICES = 64;
struct DeviceProps {
    int sms;           // multiprocessors
    int cc_major;      // compute capability, major
    int* status_word;  // device address of the status word
};
// Properties of the CURRENT device; nullptr if it cannot be queried (or its ordinal is >= MAX_DEVICES).
const DeviceProps* device_props();
// Multiprocessor count of the current device (148 if it cannot be queried).
int sm_count();

// Set-up that has to happen once per DEVICE rather than once per process (function attributes such as the
// dynamic shared-memory limit apply to the device that is current when they are set; occupancy figures differ
// between devices). run() calls fn(&value) the first time it is used with a given device current, under a lock,
// keeps the value it produced and from then on hands out a pointer to it (the value never changes again).
template <typename T>
class PerDevice {
public:
    template <typename F>
    sqap_status run(F fn, const T** out = nullptr) {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
            cudaGetLastError();
            return SQAP_ERR_CUDA;
        }
        std::lock_guard<std::mutex> lock(mutex_);
        if (!done_[dev]) {
            const sqap_status st = fn(&value_[dev]);
            if (st != SQAP_OK) return st;
            done_[dev] = true;
        }
        if (out) *out = &value_[dev];
        return SQAP_OK;
    }

private:
    std::mutex mutex_;
    bool done_[MAX_DEVICES] = {};
    T value_[MAX_DEVICES] = {};
};

// Raises a kernel's dynamic shared-memory limit on the current device (for PerDevice<int>::run).
template <typename K>
inline sqap_status set_max_dynamic_smem(K kernel, int bytes) {
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) {
        note_cuda_error(e);
        return SQAP_ERR_CUDA;
    }
    return SQAP_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Programmatic dependent launch, used along the short kernel chains of a decode step (quantizer -> weight
// streamer), where a kernel lasts a few microseconds and the gap between two kernels is of the same order.
// A kernel launched with launch_dependent() may start while the kernel before it in the stream still runs; it does
// whatever does not depend on that kernel (the streamers: fetch their first weights) and then calls pdl_wait(),
// which returns once the earlier kernel has completed and its writes are visible. The earlier kernel calls
// pdl_launch_dependents() as soon as it is running. Both calls do nothing in a kernel launched the plain way.
// THE RULE every kernel launched through launch_dependent() obeys: before its pdl_wait() it writes NO global
// memory and reads nothing that another kernel of the stream may write (in practice: packed weights and weight
// scales only, which are immutable after packing). Since these kernels release their dependents before their own
// wait, up to three kernels of a chain can be resident at once; the rule is what keeps the workspace (expanded
// codes, row sums, scales), which consecutive calls rewrite, and the activations free of races.
constexpr int PDL_MAX_ROWS = 32;   // the row counts of decode steps (the Hadamard quantizer treats them specially)
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Packed weight matrix in the library's private layout.
//
// Codes are stored two per byte, but not as neighbours: the K axis is cut into blocks of
// 2*half codes and byte j of a block holds code[j] (low nibble) and code[j + half] (high
// nibble), with half = 64 when K % 128 == 0 and 16 otherwise. The low nibble stores code + 8
// (0..15), the high nibble the two's-complement code. Masking a packed word then yields two
// valid int8 vectors without shifts or sign extension:
//     w & 0x0F0F0F0F = code_lo + 8          w & 0xF0F0F0F0 = 16 * code_hi
// The activation side compensates: codes that meet a low nibble are pre-multiplied by 16, so
// every product carries the factor 16, and the +8 bias adds 128 * (sum of those activation
// codes) per row, which the epilogue subtracts:  true = (acc - 128 * bias_sum[m]) >> 4.
struct Weights {
    uint8_t* packed;     // device [N][K/2]
    __half* scales;      // device [N]
    int N, K, half;      // half-block size of the nibble pairing (64 or 16)
    uint32_t flags;
    int device;
    // Tensor maps of the packed matrix for the tensor-core kernels' TMA loads (rows of K/2 bytes, 128B swizzle, a box
    // of 128 bytes x 128 rows, or x 64 rows where a gate / up pair shares a tile), encoded once at pack time: they
    // depend on nothing but the handle. Opaque 128-byte CUtensorMap objects; has_maps = 0 where the kernels that use
    // them cannot run the shape (K % 128 != 0) or the encoder is unavailable.
    alignas(64) unsigned char map_rows128[128];
    alignas(64) unsigned char map_rows64[128];
    int has_maps;
};

}  // namespace sqap

struct sqap_weights : sqap::Weights {};

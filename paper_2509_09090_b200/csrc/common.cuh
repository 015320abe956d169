// Shared host/device helpers of the sqap library (internal; not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/sqap.h"

namespace sqap {

// Host bookkeeping (api.cu).
void note_cuda_error(cudaError_t e);
void count_launch(int n = 1);
sqap_status check_launch();  // cudaGetLastError -> status

// Pointer to the device status word of the current device (set by kernels whose bounded waits expire).
int* device_status_word();

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Programmatic dependent launch, used along the short kernel chains of a decode step (quantizer -> weight
// streamer), where a kernel lasts a few microseconds and the gap between two kernels is of the same order.
// A kernel launched with launch_dependent() may start while the kernel before it in the stream still runs; it does
// whatever does not depend on that kernel (the streamers: fetch their first weights) and then calls pdl_wait(),
// which returns once the earlier kernel has completed and its writes are visible. The earlier kernel calls
// pdl_launch_dependents() as soon as it is running. Both calls do nothing in a kernel launched the plain way.
constexpr int PDL_MAX_ROWS = 32;   // the quantizers launch this way up to here (the row counts of decode steps)
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
};

}  // namespace sqap

struct sqap_weights : sqap::Weights {};

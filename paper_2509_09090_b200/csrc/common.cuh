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

// Internal interface of the activation quantizer (quantize.cu) for the fused quantize + linear call.
#pragma once

#include "common.cuh"

namespace sqap {

// Host-side validation shared by both entry points that quantize (x pointer, sizes, strides, flags).
sqap_status quantize_check_args(const void* x, int M, int K, int64_t ldx, uint32_t flags);

// Quantizes M rows exactly as sqap_quantize_act does, but writes the codes in the form the GEMM kernels
// multiply (linear.cuh): x8[m][k] = 16 * q[m][k] where k meets a low weight nibble, q[m][k] elsewhere,
// and bias_sum[m] = sum of q[m][k] over the former. half = the weight handle's nibble pairing (64 or 16).
sqap_status quantize_expanded(const __half* x, int M, int K, int64_t ldx, const int32_t* row_index, uint32_t flags,
                              int half, int8_t* x8, int32_t* bias_sum, float* scales, cudaStream_t s);

}  // namespace sqap

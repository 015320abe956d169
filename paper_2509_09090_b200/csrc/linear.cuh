// Internal interface between the W4A4 linear's dispatcher and its kernels.
#pragma once

#include "common.cuh"

namespace sqap {

// Everything a GEMM kernel needs. x8 / bias_sum live in the caller's workspace and are written by
// the expand pass: x8[m][k] = 16*q[m][k] where k meets a low weight nibble, q[m][k] elsewhere;
// bias_sum[m] = sum of q[m][k] over the former. A kernel accumulates raw = sum x8 * (masked weight
// byte) and finishes with  acc = (raw - 128 * bias_sum[m]) >> 4  (exact; see common.cuh).
struct LinearArgs {
    const int8_t* x8;
    const int32_t* bias_sum;
    const float* act_scales;
    int M, N, K, half;
    const uint8_t* w;       // gate (or the only) matrix
    const __half* w_scales;
    const uint8_t* w_up;    // nullptr unless SwiGLU
    const __half* w_up_scales;
    const Weights* w_handle;     // the handles themselves (for the tensor maps cached in them)
    const Weights* w_up_handle;
    void* out;
    int64_t ldo;
    int out_dtype;
    // Set only when the kernel itself is to quantize the (single) activation row: the fp16 source, as in
    // sqap_quantize_act; x8 / bias_sum / act_scales above are then OUTPUTS (written once, for later calls that
    // reuse the expanded form), not inputs.
    const __half* fuse_x;
    int64_t fuse_ldx;
    const int32_t* fuse_row_index;
};

__device__ __forceinline__ int finish_acc(int raw, int bias_sum) { return (raw - 128 * bias_sum) >> 4; }

__device__ __forceinline__ float dequant(int acc, float sx, float sw) { return __fmul_rn(__fmul_rn(static_cast<float>(acc), sx), sw); }

__device__ __forceinline__ float swiglu(float g, float u) { return g / (1.0f + expf(-g)) * u; }

__device__ __forceinline__ void store_out(void* out, int64_t idx, int out_dtype, float y, int acc) {
    if (out_dtype == SQAP_FP16) static_cast<__half*>(out)[idx] = __float2half_rn(y);
    else if (out_dtype == SQAP_BF16) static_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(y);
    else static_cast<int32_t*>(out)[idx] = acc;
}

// tcgen05 kernel (linear_tc.cu). Returns SQAP_ERR_UNSUPPORTED if the shape cannot run there.
sqap_status launch_linear_tcgen05(const LinearArgs& a, cudaStream_t s);
bool tcgen05_supports(const LinearArgs& a);

// tcgen05 kernel with the weight operand in tensor memory (linear_tc_ts.cu). Runs every shape the kernel
// above runs.
sqap_status launch_linear_tcgen05_ts(const LinearArgs& a, cudaStream_t s);

// The same on CTA pairs (linear_tc_pair.cu): the large-M kernel. Runs every shape the kernels above run.
sqap_status launch_linear_tcgen05_pair(const LinearArgs& a, cudaStream_t s);

// One cluster per tile with K split over its CTAs (linear_tc_splitk.cu): the kernel for a few dozen to a few
// hundred tokens. Runs every shape the kernels above run. forced_split: 0 = choose, 1..4 = that cluster size.
sqap_status launch_linear_tcgen05_splitk(const LinearArgs& a, int forced_split, cudaStream_t s);


// Register-MMA weight streamer for a handful of tokens (linear_mma.cu): K % 128 == 0 and M <= MMA_STREAM_MAX_M.
constexpr int MMA_STREAM_MAX_M = 32;
constexpr int MMA_FUSE_MAX_K = 16384;   // longest single row it will quantize itself (K bytes of shared memory)
bool mma_stream_supports(const LinearArgs& a);
sqap_status launch_linear_mma_stream(const LinearArgs& a, cudaStream_t s);

}  // namespace sqap

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

#ifdef __CUDACC__
// ------------------------------------------------------------------------------- device pieces of the quantizer,
// shared with the kernels that quantize a row themselves (the single-row weight streamer)
constexpr float MAGIC = 12582912.0f;   // 1.5 * 2^23: low byte of fl(y + MAGIC) = code as int8
constexpr float MAGIC8 = 12582920.0f;  // MAGIC + 8:  low nibble of fl(y + MAGIC8) = code + 8 (0..15)

__device__ __forceinline__ uint64_t pk(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void upk(uint64_t p, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p)); }
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ void scale_of(float amax, float& scale, float& inv) {
    scale = 1.0f;
    inv = 0.0f;
    if (amax != 0.0f) {
        scale = __fdiv_rn(amax, 7.0f);
        inv = __fdiv_rn(7.0f, amax);
    }
}

// Bits of fl(fl(v * inv) + magic) for a pair of values. The product must be rounded to fp32 before the sum
// (a fused multiply-add rounds once and lands on the other side of a tie): scalar __fmul_rn / __fadd_rn are
// never contracted, whereas a packed multiply followed by a packed add was seen to be.
__device__ __forceinline__ void round_pair(uint64_t v, float inv, float magic, uint32_t& lo, uint32_t& hi) {
    float a, b;
    upk(v, a, b);
    lo = __float_as_uint(__fadd_rn(__fmul_rn(a, inv), magic));
    hi = __float_as_uint(__fadd_rn(__fmul_rn(b, inv), magic));
}

// Low bytes of four words -> one word.
__device__ __forceinline__ uint32_t low_bytes(uint32_t t0, uint32_t t1, uint32_t t2, uint32_t t3) {
    return __byte_perm(__byte_perm(t0, t1, 0x0040), __byte_perm(t2, t3, 0x0040), 0x5410);
}
// A word of four int8 codes -> the same codes times 16 (each still fits a byte).
__device__ __forceinline__ uint32_t times16(uint32_t w) { return (w << 4) & 0xF0F0F0F0u; }

__device__ __forceinline__ void half8_to_pairs(const uint4& u, uint64_t* p) {
    const __half2* h = reinterpret_cast<const __half2*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h[i]);
        p[i] = pk(f.x, f.y);
    }
}

#endif

}  // namespace sqap

// Per-token symmetric INT4 activation quantizer with the optional Hadamard rotation of Eq. 6.
//
// HBM-bound: 2 bytes read and half a byte written per element. One CTA owns one row; the row
// stays in registers between the max-abs reduction and the rounding pass, so global memory is
// touched once. All fp32 steps use the explicitly rounded intrinsics, so no multiply-add is
// fused and the result is defined bit for bit by the order of operations stated in sqap.h.
#include "common.cuh"

namespace sqap {

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Block-wide max of non-negative values; every thread gets the result. red: >= 32 floats of smem.
__device__ __forceinline__ float block_max(float v, float* red) {
    v = warp_max(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = (blockDim.x + 31) >> 5;
    if (nwarps == 1) return v;
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float r = (lane < nwarps) ? red[lane] : 0.0f;
    r = warp_max(r);
    __syncthreads();
    return r;
}

__device__ __forceinline__ int quant_code(float v, float inv) {
    int q = __float2int_rn(__fmul_rn(v, inv));  // round half to even
    return max(-8, min(7, q));
}

// 8 fp32 values -> 8 two's-complement nibbles, value i in nibble i.
__device__ __forceinline__ uint32_t pack8(const float* v, float inv) {
    uint32_t w = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) w |= (static_cast<uint32_t>(quant_code(v[i], inv)) & 0xFu) << (4 * i);
    return w;
}

__device__ __forceinline__ void unpack_half8(const uint4& u, float* f) {
    const __half2* h = reinterpret_cast<const __half2*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 t = __half22float2(h[i]);
        f[2 * i] = t.x;
        f[2 * i + 1] = t.y;
    }
}

// ---------------------------------------------------------------------------------------------
// Plain (unrotated) rows. Thread t handles the 16-byte chunks t, t + T, t + 2T, ... of the row.
// Up to MAX_IT chunks per thread are kept in registers; longer rows are re-read (L2 hit).
constexpr int QUANT_MAX_IT = 8;

__global__ void __launch_bounds__(256) quantize_rows_kernel(const __half* __restrict__ x, int K, int64_t ldx,
                                                            const int32_t* __restrict__ row_index,
                                                            uint8_t* __restrict__ q, float* __restrict__ scales) {
    __shared__ float red[32];
    const int row = blockIdx.x;
    const int64_t src = row_index ? static_cast<int64_t>(row_index[row]) : static_cast<int64_t>(row);
    const uint4* xr = reinterpret_cast<const uint4*>(x + src * ldx);
    uint32_t* qr = reinterpret_cast<uint32_t*>(q + static_cast<int64_t>(row) * (K / 2));
    const int chunks = K / 8;
    const int T = blockDim.x;

    uint4 cache[QUANT_MAX_IT];
    float amax = 0.0f;
#pragma unroll
    for (int it = 0; it < QUANT_MAX_IT; ++it) {
        const int c = it * T + threadIdx.x;
        if (c < chunks) {
            cache[it] = __ldg(xr + c);
            float f[8];
            unpack_half8(cache[it], f);
#pragma unroll
            for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(f[i]));
        }
    }
    for (int c = QUANT_MAX_IT * T + threadIdx.x; c < chunks; c += T) {
        float f[8];
        unpack_half8(__ldg(xr + c), f);
#pragma unroll
        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(f[i]));
    }
    amax = block_max(amax, red);
    float scale = 1.0f, inv = 0.0f;
    if (amax != 0.0f) {
        scale = __fdiv_rn(amax, 7.0f);
        inv = __fdiv_rn(7.0f, amax);
    }
    if (threadIdx.x == 0) scales[row] = scale;
#pragma unroll
    for (int it = 0; it < QUANT_MAX_IT; ++it) {
        const int c = it * T + threadIdx.x;
        if (c < chunks) {
            float f[8];
            unpack_half8(cache[it], f);
            qr[c] = pack8(f, inv);
        }
    }
    for (int c = QUANT_MAX_IT * T + threadIdx.x; c < chunks; c += T) {
        float f[8];
        unpack_half8(__ldg(xr + c), f);
        qr[c] = pack8(f, inv);
    }
}

// ---------------------------------------------------------------------------------------------
// Rotated rows: fast Walsh-Hadamard transform, stages h = 1, 2, 4, ..., K/2 in that order, each
// pair (j, j+h) -> (a+b, a-b). Thread t holds the E contiguous elements E*t .. E*t+E-1, so the
// first log2(E) stages are register-local, the next (up to 5) are warp shuffles, and the rest
// go through shared memory. T = K / E threads.
template <int E>
__global__ void __launch_bounds__(1024) quantize_rows_rotate_kernel(const __half* __restrict__ x, int K, int64_t ldx,
                                                                    const int32_t* __restrict__ row_index,
                                                                    float norm, uint8_t* __restrict__ q,
                                                                    float* __restrict__ scales) {
    extern __shared__ float sm[];  // K floats when K/E > 32, plus 32 for the reduction
    float* red = sm;
    float* buf = sm + 32;
    const int row = blockIdx.x;
    const int t = threadIdx.x;
    const int T = blockDim.x;
    const int lane = t & 31;
    const int64_t src = row_index ? static_cast<int64_t>(row_index[row]) : static_cast<int64_t>(row);
    const __half* xr = x + src * ldx + static_cast<int64_t>(t) * E;

    float v[E];
    if constexpr (E >= 8) {
#pragma unroll
        for (int c = 0; c < E / 8; ++c) unpack_half8(__ldg(reinterpret_cast<const uint4*>(xr) + c), v + 8 * c);
    } else {
#pragma unroll
        for (int i = 0; i < E; i += 2) {
            float2 f = __half22float2(*reinterpret_cast<const __half2*>(xr + i));
            v[i] = f.x;
            v[i + 1] = f.y;
        }
    }
    // register-local stages
#pragma unroll
    for (int h = 1; h < E; h <<= 1) {
#pragma unroll
        for (int j = 0; j < E; ++j) {
            if ((j & h) == 0) {
                const float a = v[j], b = v[j + h];
                v[j] = __fadd_rn(a, b);
                v[j + h] = __fsub_rn(a, b);
            }
        }
    }
    // warp-shuffle stages: partner thread differs in one lane bit
    const int lane_stages = T >= 32 ? 32 : T;
    for (int m = 1; m < lane_stages; m <<= 1) {
        const bool upper = (lane & m) != 0;
#pragma unroll
        for (int j = 0; j < E; ++j) {
            const float p = __shfl_xor_sync(0xffffffffu, v[j], m);
            v[j] = upper ? __fsub_rn(p, v[j]) : __fadd_rn(v[j], p);
        }
    }
    // cross-warp stages through shared memory
    for (int m = 32; m < T; m <<= 1) {
#pragma unroll
        for (int j = 0; j < E; ++j) buf[j * T + t] = v[j];  // element-major: conflict-free
        __syncthreads();
        const bool upper = (t & m) != 0;
#pragma unroll
        for (int j = 0; j < E; ++j) {
            const float p = buf[j * T + (t ^ m)];
            v[j] = upper ? __fsub_rn(p, v[j]) : __fadd_rn(v[j], p);
        }
        __syncthreads();
    }
    float amax = 0.0f;
#pragma unroll
    for (int j = 0; j < E; ++j) {
        v[j] = __fmul_rn(v[j], norm);
        amax = fmaxf(amax, fabsf(v[j]));
    }
    amax = block_max(amax, red);
    float scale = 1.0f, inv = 0.0f;
    if (amax != 0.0f) {
        scale = __fdiv_rn(amax, 7.0f);
        inv = __fdiv_rn(7.0f, amax);
    }
    if (t == 0) scales[row] = scale;
    uint8_t* qr = q + static_cast<int64_t>(row) * (K / 2) + static_cast<int64_t>(t) * (E / 2);
    if constexpr (E >= 8) {
        uint32_t w[E / 8];
#pragma unroll
        for (int c = 0; c < E / 8; ++c) w[c] = pack8(v + 8 * c, inv);
        if constexpr (E == 16) {
            *reinterpret_cast<uint2*>(qr) = make_uint2(w[0], w[1]);
        } else {
            *reinterpret_cast<uint32_t*>(qr) = w[0];
        }
    } else {
#pragma unroll
        for (int i = 0; i < E; i += 2)
            qr[i / 2] = static_cast<uint8_t>((quant_code(v[i], inv) & 0xF) | ((quant_code(v[i + 1], inv) & 0xF) << 4));
    }
}

template <int E>
static void launch_rotate(const __half* x, int M, int K, int64_t ldx, const int32_t* row_index, uint8_t* q,
                          float* scales, cudaStream_t s) {
    const int T = K / E;
    const float norm = static_cast<float>(1.0 / sqrt(static_cast<double>(K)));
    const size_t smem = (32 + (T > 32 ? static_cast<size_t>(K) : 0)) * sizeof(float);
    if (smem > 48 * 1024)
        cudaFuncSetAttribute(quantize_rows_rotate_kernel<E>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(smem));
    quantize_rows_rotate_kernel<E><<<M, T, smem, s>>>(x, K, ldx, row_index, norm, q, scales);
}

}  // namespace sqap

extern "C" sqap_status sqap_quantize_act(const void* x, int M, int K, int64_t ldx, const int32_t* row_index,
                                         uint32_t flags, uint8_t* q_packed, float* scales, void* stream) {
    using namespace sqap;
    if (M < 0 || K <= 0 || ldx < K) return SQAP_ERR_INVALID;
    if (flags & ~SQAP_Q_ROTATE) return SQAP_ERR_INVALID;
    if (M == 0) return SQAP_OK;
    if (!x || !q_packed || !scales) return SQAP_ERR_INVALID;
    if (K % 32 != 0 || ldx % 8 != 0 || !aligned16(x) || !aligned16(q_packed)) return SQAP_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(scales) & 3u) return SQAP_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const __half* xh = static_cast<const __half*>(x);
    if (flags & SQAP_Q_ROTATE) {
        if ((K & (K - 1)) != 0 || K < 64 || K > 16384) return SQAP_ERR_UNSUPPORTED;
        // E elements per thread: 16 from K = 512 up (T = K/16 <= 1024), fewer for short rows so a full warp works
        if (K >= 512) launch_rotate<16>(xh, M, K, ldx, row_index, q_packed, scales, s);
        else if (K == 256) launch_rotate<8>(xh, M, K, ldx, row_index, q_packed, scales, s);
        else if (K == 128) launch_rotate<4>(xh, M, K, ldx, row_index, q_packed, scales, s);
        else launch_rotate<2>(xh, M, K, ldx, row_index, q_packed, scales, s);
    } else {
        int T = (K / 8 + 31) / 32 * 32;
        if (T > 256) T = 256;
        quantize_rows_kernel<<<M, T, 0, s>>>(xh, K, ldx, row_index, q_packed, scales);
    }
    count_launch();
    return check_launch();
}

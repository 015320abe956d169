// Offline weight side: INT4 codes + per-output-channel fp16 scales -> the private packed layout
// described in common.cuh, and its inverse for checking. Pure permutation / re-encoding.
#include <new>

#include "tc_common.cuh"

namespace sqap {

// One thread writes 4 packed bytes = 4 low codes + 4 high codes (both contiguous in the source).
__global__ void pack_weights_kernel(const int8_t* __restrict__ codes, int N, int K, int half,
                                    uint8_t* __restrict__ packed, int* __restrict__ bad) {
    const int64_t words_per_row = K / 8;
    const int64_t total = static_cast<int64_t>(N) * words_per_row;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t n = i / words_per_row;
        const int j = static_cast<int>(i % words_per_row) * 4;  // packed byte index within the row
        const int blk = j / half, r = j % half;
        const int8_t* row = codes + n * K;
        const char4 lo = *reinterpret_cast<const char4*>(row + blk * 2 * half + r);
        const char4 hi = *reinterpret_cast<const char4*>(row + blk * 2 * half + half + r);
        const int l[4] = {lo.x, lo.y, lo.z, lo.w}, h[4] = {hi.x, hi.y, hi.z, hi.w};
        uint32_t w = 0;
        bool oob = false;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            oob |= (l[b] < -8) | (l[b] > 7) | (h[b] < -8) | (h[b] > 7);
            w |= (static_cast<uint32_t>((l[b] + 8) & 0xF) | (static_cast<uint32_t>(h[b] & 0xF) << 4)) << (8 * b);
        }
        if (oob) atomicOr(bad, 1);
        reinterpret_cast<uint32_t*>(packed + n * (K / 2))[j / 4] = w;
    }
}

__global__ void check_scales_kernel(const __half* __restrict__ scales, int N, int* __restrict__ bad) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N) return;
    const float s = __half2float(scales[n]);
    if (!(s > 0.0f) || isinf(s)) atomicOr(bad, 2);
}

__global__ void unpack_weights_kernel(const uint8_t* __restrict__ packed, int N, int K, int half,
                                      int8_t* __restrict__ codes) {
    const int64_t total = static_cast<int64_t>(N) * (K / 2);
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t n = i / (K / 2);
        const int j = static_cast<int>(i % (K / 2));
        const int blk = j / half, r = j % half;
        const uint8_t b = packed[i];
        const int hi4 = b >> 4;
        codes[n * K + blk * 2 * half + r] = static_cast<int8_t>((b & 0xF) - 8);
        codes[n * K + blk * 2 * half + half + r] = static_cast<int8_t>(hi4 >= 8 ? hi4 - 16 : hi4);
    }
}

// ---------------------------------------------------------------------------------------------
// Offline weight quantizer: fp16 W [N][K] -> INT4 codes + fp16 per-channel scales, with the optional
// rotation of Eq. 6 (row n of W H^T = H applied to row n; H symmetric). Offline and run once per model,
// so it is written for clarity: one CTA per output channel, the row in shared memory as fp32, the
// Walsh-Hadamard stages h = 1, 2, 4, ... applied one after the other with a barrier between them
// (every stage output is one fp32 add of two fixed inputs, so the bits do not depend on the thread map).
__global__ void __launch_bounds__(256) quantize_weight_rows_kernel(const __half* __restrict__ w, int K, int64_t ldw,
                                                                   const float* __restrict__ ch_mul, int rotate,
                                                                   float norm, int8_t* __restrict__ codes,
                                                                   __half* __restrict__ scales) {
    extern __shared__ float row[];   // K floats
    __shared__ float red[8];
    const int n = blockIdx.x;
    const __half* wr = w + static_cast<int64_t>(n) * ldw;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        float v = __half2float(wr[k]);
        if (ch_mul) v = __fmul_rn(v, ch_mul[k]);
        row[k] = v;
    }
    __syncthreads();
    if (rotate) {
        for (int h = 1; h < K; h <<= 1) {
            for (int pr = threadIdx.x; pr < K / 2; pr += blockDim.x) {
                const int j = (pr / h) * 2 * h + (pr % h);
                const float a = row[j], b = row[j + h];
                row[j] = __fadd_rn(a, b);
                row[j + h] = __fsub_rn(a, b);
            }
            __syncthreads();
        }
        for (int k = threadIdx.x; k < K; k += blockDim.x) row[k] = __fmul_rn(row[k], norm);
        __syncthreads();
    }
    float amax = 0.0f;
    for (int k = threadIdx.x; k < K; k += blockDim.x) amax = fmaxf(amax, fabsf(row[k]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    amax = red[0];
    for (int i = 1; i < (blockDim.x >> 5); ++i) amax = fmaxf(amax, red[i]);
    __half s16 = __float2half_rn(1.0f);
    if (amax != 0.0f) {
        s16 = __float2half_rn(__fdiv_rn(amax, 7.0f));
        if ((__half_as_ushort(s16) & 0x7FFF) == 0) s16 = __ushort_as_half(0x0001);   // smallest positive fp16
    }
    if (threadIdx.x == 0) scales[n] = s16;
    const float sf = __half2float(s16);
    int8_t* cr = codes + static_cast<int64_t>(n) * K;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        const int q = __float2int_rn(__fdiv_rn(row[k], sf));
        cr[k] = static_cast<int8_t>(max(-8, min(7, q)));
    }
}

static bool is_device_pointer(const void* p) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return a.type == cudaMemoryTypeDevice || a.type == cudaMemoryTypeManaged;
}

#define SQAP_CUDA_TRY(expr)                  \
    do {                                     \
        cudaError_t e__ = (expr);            \
        if (e__ != cudaSuccess) {            \
            note_cuda_error(e__);            \
            st = (e__ == cudaErrorMemoryAllocation) ? SQAP_ERR_NOMEM : SQAP_ERR_CUDA; \
            goto fail;                       \
        }                                    \
    } while (0)

}  // namespace sqap

extern "C" {

sqap_status sqap_pack_weights(const int8_t* codes, const uint16_t* scales_fp16, int N, int K, uint32_t flags,
                              void* stream, sqap_weights** out) {
    using namespace sqap;
    if (!out) return SQAP_ERR_INVALID;
    *out = nullptr;
    if (!codes || !scales_fp16 || N <= 0 || K <= 0) return SQAP_ERR_INVALID;
    if (flags & ~SQAP_W_ROTATED) return SQAP_ERR_INVALID;
    if (K % 32 != 0) return SQAP_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    sqap_status st = SQAP_OK;
    sqap_weights* w = new (std::nothrow) sqap_weights();
    if (!w) return SQAP_ERR_NOMEM;
    w->packed = nullptr;
    w->scales = nullptr;
    w->N = N;
    w->K = K;
    w->half = (K % 128 == 0) ? 64 : 16;
    w->flags = flags;
    int8_t* staged = nullptr;
    int* bad = nullptr;
    int bad_host = 0;
    const size_t n_codes = static_cast<size_t>(N) * K;
    {
        SQAP_CUDA_TRY(cudaGetDevice(&w->device));
        SQAP_CUDA_TRY(cudaMalloc(&w->packed, n_codes / 2));
        SQAP_CUDA_TRY(cudaMalloc(&w->scales, sizeof(__half) * N));
        SQAP_CUDA_TRY(cudaMalloc(&bad, sizeof(int)));
        SQAP_CUDA_TRY(cudaMemsetAsync(bad, 0, sizeof(int), s));
        const int8_t* src = codes;
        if (!is_device_pointer(codes)) {
            SQAP_CUDA_TRY(cudaMalloc(&staged, n_codes));
            SQAP_CUDA_TRY(cudaMemcpyAsync(staged, codes, n_codes, cudaMemcpyHostToDevice, s));
            src = staged;
        } else if (reinterpret_cast<uintptr_t>(codes) & 3u) {
            st = SQAP_ERR_ALIGN;
            goto fail;
        }
        SQAP_CUDA_TRY(cudaMemcpyAsync(w->scales, scales_fp16, sizeof(__half) * N, cudaMemcpyDefault, s));
        const int64_t words = static_cast<int64_t>(n_codes / 8);
        const int blocks = static_cast<int>(words / 256 + 1 < 148 * 16 ? words / 256 + 1 : 148 * 16);
        pack_weights_kernel<<<blocks, 256, 0, s>>>(src, N, K, w->half, w->packed, bad);
        check_scales_kernel<<<(N + 255) / 256, 256, 0, s>>>(w->scales, N, bad);
        count_launch(2);
        st = check_launch();
        if (st != SQAP_OK) goto fail;
        SQAP_CUDA_TRY(cudaMemcpyAsync(&bad_host, bad, sizeof(int), cudaMemcpyDeviceToHost, s));
        SQAP_CUDA_TRY(cudaStreamSynchronize(s));
        if (bad_host) {
            st = SQAP_ERR_RANGE;
            goto fail;
        }
    }
    cudaFree(staged);
    cudaFree(bad);
    tc::encode_handle_maps(w);
    *out = w;
    return SQAP_OK;
fail:
    cudaFree(staged);
    cudaFree(bad);
    cudaFree(w->packed);
    cudaFree(w->scales);
    delete w;
    return st;
}

sqap_status sqap_quantize_weights(const void* w_fp16, int N, int K, int64_t ldw, uint32_t flags, const float* channel_mul,
                                  int8_t* codes_out, uint16_t* scales_out_fp16, void* stream) {
    using namespace sqap;
    if (N < 0 || K <= 0 || ldw < K) return SQAP_ERR_INVALID;
    if (flags & ~SQAP_Q_ROTATE) return SQAP_ERR_INVALID;
    if (N == 0) return SQAP_OK;
    if (!w_fp16 || !codes_out || !scales_out_fp16) return SQAP_ERR_INVALID;
    if (K % 32 != 0) return SQAP_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(w_fp16) & 1u) || (reinterpret_cast<uintptr_t>(scales_out_fp16) & 1u) ||
        (reinterpret_cast<uintptr_t>(channel_mul) & 3u))
        return SQAP_ERR_ALIGN;
    const bool rotate = (flags & SQAP_Q_ROTATE) != 0;
    if (rotate && ((K & (K - 1)) != 0 || K < 64)) return SQAP_ERR_UNSUPPORTED;
    if (K > 32768) return SQAP_ERR_UNSUPPORTED;   // the row is held in shared memory as fp32
    const size_t smem = sizeof(float) * static_cast<size_t>(K);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(quantize_weight_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem));
        if (e != cudaSuccess) {
            note_cuda_error(e);
            return SQAP_ERR_CUDA;
        }
    }
    const float norm = static_cast<float>(1.0 / sqrt(static_cast<double>(K)));
    quantize_weight_rows_kernel<<<N, 256, smem, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __half*>(w_fp16), K, ldw, channel_mul, rotate ? 1 : 0, norm, codes_out, reinterpret_cast<__half*>(scales_out_fp16));
    count_launch();
    return check_launch();
}

sqap_status sqap_free_weights(sqap_weights* w) {
    if (!w) return SQAP_OK;
    cudaDeviceSynchronize();
    cudaFree(w->packed);
    cudaFree(w->scales);
    delete w;
    return SQAP_OK;
}

sqap_status sqap_weights_info(const sqap_weights* w, int* N, int* K, uint32_t* flags) {
    if (!w) return SQAP_ERR_INVALID;
    if (N) *N = w->N;
    if (K) *K = w->K;
    if (flags) *flags = w->flags;
    return SQAP_OK;
}

sqap_status sqap_unpack_weights(const sqap_weights* w, int8_t* codes_out_host, uint16_t* scales_out_host) {
    using namespace sqap;
    if (!w || !codes_out_host || !scales_out_host) return SQAP_ERR_INVALID;
    sqap_status st = SQAP_OK;
    int8_t* tmp = nullptr;
    const size_t n_codes = static_cast<size_t>(w->N) * w->K;
    {
        SQAP_CUDA_TRY(cudaDeviceSynchronize());
        SQAP_CUDA_TRY(cudaMalloc(&tmp, n_codes));
        unpack_weights_kernel<<<148 * 8, 256>>>(w->packed, w->N, w->K, w->half, tmp);
        count_launch();
        st = check_launch();
        if (st != SQAP_OK) goto fail;
        SQAP_CUDA_TRY(cudaMemcpy(codes_out_host, tmp, n_codes, cudaMemcpyDeviceToHost));
        SQAP_CUDA_TRY(cudaMemcpy(scales_out_host, w->scales, sizeof(uint16_t) * w->N, cudaMemcpyDeviceToHost));
    }
fail:
    cudaFree(tmp);
    return st;
}

}  // extern "C"

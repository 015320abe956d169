// Offline weight side: INT4 codes + per-output-channel fp16 scales -> the private packed layout
// described in common.cuh, and its inverse for checking. Pure permutation / re-encoding.
#include <new>

#include "common.cuh"

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

// Per-token symmetric INT4 activation quantizer with the optional Hadamard rotation of Eq. 6.
//
// HBM-bound for plain rows (2 bytes read, half a byte written per element); with the rotation the
// 12 add/sub stages per element of K = 4096 put the fp32 pipes at about the same time as the memory
// system. Global memory is touched once: a row stays in registers (and, for the rotation, shared
// memory) between the max-abs reduction and the rounding pass. All fp32 steps use explicitly rounded,
// unfused operations, so the result is defined bit for bit by the order of operations stated in sqap.h.
//
// Rounding without a float-to-int conversion: for |y| < 2^22, fl(y + 1.5 * 2^23) has an ulp of 1, so the
// sum's low mantissa bits hold round_half_even(y) in two's complement. |v * inv| never exceeds 7 by more
// than rounding error for finite inputs (|v| <= amax, inv = fl(7 / amax)), so the clamp of the definition
// can never bind and is not evaluated; non-finite inputs give unspecified codes, as documented.
//
// Two output forms share every kernel (template parameter SINK):
//   SINK_NIBBLES   the public layout of sqap_quantize_act (two codes per byte)
//   SINK_EXPANDED  what the GEMM kernels multiply (linear.cuh): one int8 per code, codes that meet a low
//                  weight nibble pre-multiplied by 16, plus the per-row sum of those codes. This skips the
//                  expand pass when quantizer and linear run as one call (sqap_quantize_linear).
#include <atomic>

#include "quantize.cuh"

namespace sqap {

constexpr int SINK_NIBBLES = 0, SINK_EXPANDED = 1;
struct QuantOut {
    uint8_t* q;         // SINK_NIBBLES: [M][K/2]
    int8_t* x8;         // SINK_EXPANDED: [M][K]
    int32_t* bias_sum;  // SINK_EXPANDED: [M]
    float* scales;      // [M]
    int half;           // SINK_EXPANDED: half-block of the weight nibble pairing (64 or 16)
};

// ------------------------------------------------------------------------------- packed fp32 helpers
__device__ __forceinline__ void upk_bits(uint64_t p, uint32_t& lo, uint32_t& hi) { asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(p)); }
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}


// The other granularities of sqap_quantize_act_ex, as template parameters of the same kernels:
//   MUL   a static per-input-channel multiplier is applied to fp32(x) first ("channel-wise": smoothing)
//   MODE  QM_TOKEN  one scale per row (the default);
//         QM_AMAX   first pass of the tensor-wise form: only the max-abs, folded into one word with atomicMax
//                   (the bits of a non-negative float order like the float);
//         QM_GIVEN  second pass: every row is quantized with the max-abs found in that word.
constexpr int QM_TOKEN = 0, QM_AMAX = 1, QM_GIVEN = 2;
struct QuantEx {
    const float* ch_mul;      // [K] or nullptr
    unsigned* tensor_amax;    // the word of QM_AMAX / QM_GIVEN
};
__device__ __forceinline__ void fold_amax(unsigned* word, float amax) {
    const unsigned bits = __float_as_uint(amax);
    if (bits > *reinterpret_cast<volatile unsigned*>(word)) atomicMax(word, bits);   // most rows lose: skip their atomic
}
// Eight values k = 8c .. 8c+7 as packed pairs times their channel multipliers (each product rounded to fp32). Scalar
// __fmul_rn on purpose: it is never contracted with an add that follows (the first butterfly stage, when the row is
// rotated), whereas a packed multiply followed by a packed add was seen to become a fused multiply-add even with
// explicit rounding modes.
__device__ __forceinline__ void scale_channels(uint64_t* p, const float* __restrict__ ch_mul, int c) {
    const float4 m0 = __ldg(reinterpret_cast<const float4*>(ch_mul) + 2 * c), m1 = __ldg(reinterpret_cast<const float4*>(ch_mul) + 2 * c + 1);
    const float m[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float a, b;
        upk(p[i], a, b);
        p[i] = pk(__fmul_rn(a, m[2 * i]), __fmul_rn(b, m[2 * i + 1]));
    }
}
// A 16-byte load that does not take a line of L1 (the channel-wise form streams x once and wants the multipliers,
// which every row re-reads, to stay there).
__device__ __forceinline__ uint4 ld_once(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float absmax_pairs(const uint64_t* p, int n, float m) {
    for (int i = 0; i < n; ++i) {
        float a, b;
        upk(p[i], a, b);
        m = fmaxf(m, fmaxf(fabsf(a), fabsf(b)));
    }
    return m;
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
__device__ __forceinline__ int block_sum(int v, int* red) {
    v = warp_sum(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = (blockDim.x + 31) >> 5;
    if (nwarps == 1) return v;
    if (lane == 0) red[warp] = v;
    __syncthreads();
    int r = (lane < nwarps) ? red[lane] : 0;
    r = warp_sum(r);
    __syncthreads();
    return r;
}

// Two words of four bytes each holding code + 8 (0..15) -> eight two's-complement nibbles, value i in nibble i.
__device__ __forceinline__ uint32_t nibbles_of(uint32_t w0, uint32_t w1) {
    const uint32_t x0 = w0 | (w0 >> 4), x1 = w1 | (w1 >> 4);
    return __byte_perm(x0, x1, 0x6420) ^ 0x88888888u;
}
// Eight consecutive values (k = 8c .. 8c+7 of the row) -> output. v as four packed pairs.
template <int SINK>
__device__ __forceinline__ void emit_chunk(const uint64_t* v, float inv, int c, const QuantOut& o, int64_t row,
                                           int K, int& bias) {
    const float magic = SINK == SINK_NIBBLES ? MAGIC8 : MAGIC;
    uint32_t t[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) round_pair(v[i], inv, magic, t[2 * i], t[2 * i + 1]);
    const uint32_t w0 = low_bytes(t[0], t[1], t[2], t[3]), w1 = low_bytes(t[4], t[5], t[6], t[7]);
    if (SINK == SINK_NIBBLES) {
        reinterpret_cast<uint32_t*>(o.q + row * (K / 2))[c] = nibbles_of(w0, w1);
    } else {
        const bool low = ((8 * c) % (2 * o.half)) < o.half;
        uint2 out = make_uint2(w0, w1);
        if (low) {
            bias = __dp4a(static_cast<int>(w0), 0x01010101, bias);
            bias = __dp4a(static_cast<int>(w1), 0x01010101, bias);
            out = make_uint2(times16(w0), times16(w1));
        }
        reinterpret_cast<uint2*>(o.x8 + row * K)[c] = out;
    }
}

// ---------------------------------------------------------------------------------------------
// Plain (unrotated) rows. G threads own a row (256 / G rows per CTA); thread u of a row handles the 16-byte
// chunks u, u + G, ... of it, up to QUANT_NIT of them held in registers (128 bytes in flight per thread);
// longer rows are re-read in the second pass (L2 hit). The max-abs runs on the fp16 values themselves
// (a maximum needs no widening).
constexpr int QUANT_NIT = 8;
constexpr int QUANT_THREADS = 256;

template <int SINK, int G, int MODE = QM_TOKEN, bool MUL = false>
__global__ void __launch_bounds__(QUANT_THREADS) quantize_rows_kernel(const __half* __restrict__ x, int M, int K,
                                                                      int64_t ldx,
                                                                      const int32_t* __restrict__ row_index,
                                                                      QuantOut o, QuantEx ex) {
    constexpr int ROWS = QUANT_THREADS / G, WARPS = G / 32;
    __shared__ float red_f[ROWS][WARPS];
    __shared__ int red_i[ROWS][WARPS];
    pdl_launch_dependents();
    pdl_wait();   // x may be the output of the kernel before this one
    const int g = threadIdx.x / G, u = threadIdx.x % G;
    const int row = blockIdx.x * ROWS + g;
    const bool row_ok = row < M;
    const int64_t src = row_ok ? (row_index ? static_cast<int64_t>(row_index[row]) : static_cast<int64_t>(row)) : 0;
    const uint4* xr = reinterpret_cast<const uint4*>(x + src * ldx);
    const int chunks = row_ok ? K / 8 : 0;

    // the row's values as packed fp32 pairs, channel multipliers applied (the same products in both passes)
    auto pairs_of = [&](const uint4& raw, int c, uint64_t* p) {
        half8_to_pairs(raw, p);
        if constexpr (MUL) scale_channels(p, ex.ch_mul, c);
    };
    // held between the two passes: the raw fp16 chunks, or (channel-wise form) the fp32 products of half as many
    // chunks per thread (twice the threads per row), so that neither the products nor the multipliers are formed twice
    constexpr int NIT = MUL ? QUANT_NIT / 2 : QUANT_NIT;
    uint4 cache[MUL ? 1 : NIT];
    uint64_t prod[MUL ? NIT : 1][4];
    float amax = 0.0f;
    if constexpr (MODE == QM_GIVEN) {
        amax = __uint_as_float(*ex.tensor_amax);
    } else {
        __half2 m2 = __float2half2_rn(0.0f);
        auto absmax = [&](const uint4& v, int c) {
            if constexpr (MUL) {   // products are fp32
                uint64_t p[4];
                pairs_of(v, c, p);
                amax = absmax_pairs(p, 4, amax);
            } else {
                const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
                for (int i = 0; i < 4; ++i) m2 = __hmax2(m2, __habs2(h[i]));
            }
        };
        if constexpr (MUL) {
            uint4 raw[NIT];
#pragma unroll
            for (int it = 0; it < NIT; ++it)
                if (it * G + u < chunks) raw[it] = ld_once(xr + it * G + u);
#pragma unroll
            for (int it = 0; it < NIT; ++it)
                if (it * G + u < chunks) {
                    pairs_of(raw[it], it * G + u, prod[it]);
                    amax = absmax_pairs(prod[it], 4, amax);
                }
        } else {
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                const int c = it * G + u;
                if (c < chunks) cache[it] = __ldg(xr + c);
            }
#pragma unroll
            for (int it = 0; it < NIT; ++it)
                if (it * G + u < chunks) absmax(cache[it], it * G + u);
        }
        for (int c = NIT * G + u; c < chunks; c += G) absmax(__ldg(xr + c), c);
        if constexpr (!MUL) amax = fmaxf(__low2float(m2), __high2float(m2));
        amax = warp_max(amax);
        if (WARPS > 1) {
            if ((u & 31) == 0) red_f[g][u >> 5] = amax;
            __syncthreads();
#pragma unroll
            for (int w = 0; w < WARPS; ++w) amax = fmaxf(amax, red_f[g][w]);
        }
        if constexpr (MODE == QM_AMAX) {
            if (u == 0 && row_ok) fold_amax(ex.tensor_amax, amax);
            return;
        }
    }
    float scale, inv;
    scale_of(amax, scale, inv);
    if (u == 0 && row_ok) o.scales[row] = scale;
    int bias = 0;
#pragma unroll
    for (int it = 0; it < NIT; ++it) {
        const int c = it * G + u;
        if (c < chunks) {
            if constexpr (MUL && MODE != QM_GIVEN) {
                emit_chunk<SINK>(prod[it], inv, c, o, row, K, bias);
            } else {
                uint64_t p[4];
                pairs_of(MODE == QM_GIVEN ? __ldg(xr + c) : cache[MUL ? 0 : it], c, p);
                emit_chunk<SINK>(p, inv, c, o, row, K, bias);
            }
        }
    }
    for (int c = NIT * G + u; c < chunks; c += G) {
        uint64_t p[4];
        pairs_of(__ldg(xr + c), c, p);
        emit_chunk<SINK>(p, inv, c, o, row, K, bias);
    }
    if (SINK == SINK_EXPANDED) {
        bias = warp_sum(bias);
        if (WARPS > 1) {
            if ((u & 31) == 0) red_i[g][u >> 5] = bias;
            __syncthreads();
            bias = 0;
#pragma unroll
            for (int w = 0; w < WARPS; ++w) bias += red_i[g][w];
        }
        if (u == 0 && row_ok) o.bias_sum[row] = bias;
    }
}

template <int SINK, int G, int MODE = QM_TOKEN, bool MUL = false>
static void launch_plain(const __half* x, int M, int K, int64_t ldx, const int32_t* row_index, const QuantOut& o,
                         cudaStream_t s, QuantEx ex = QuantEx{nullptr, nullptr}) {
    constexpr int ROWS = QUANT_THREADS / G;
    const cudaError_t e = launch_dependent(quantize_rows_kernel<SINK, G, MODE, MUL>, dim3((M + ROWS - 1) / ROWS),
                                           dim3(QUANT_THREADS), 0, s, x, M, K, ldx, row_index, o, ex);
    if (e != cudaSuccess) note_cuda_error(e);
}

// ---------------------------------------------------------------------------------------------
// Rotated rows, any power-of-two K: fast Walsh-Hadamard transform, stages h = 1, 2, 4, ..., K/2 in that
// order, each pair (j, j+h) -> (a+b, a-b). Thread t holds the E contiguous elements E*t .. E*t+E-1, so
// the first log2(E) stages are register-local, the next (up to 5) are warp shuffles, and the rest go
// through shared memory. T = K / E threads.
template <int E, int SINK>
__global__ void __launch_bounds__(1024) quantize_rows_rotate_kernel(const __half* __restrict__ x, int K, int64_t ldx,
                                                                    const int32_t* __restrict__ row_index,
                                                                    float norm, QuantOut o, QuantEx ex, int mode) {
    extern __shared__ float sm[];  // K floats when K/E > 32, plus 32 for the reduction
    float* red = sm;
    float* buf = sm + 32;
    pdl_launch_dependents();
    pdl_wait();   // x may be the output of the kernel before this one
    const int row = blockIdx.x;
    const int t = threadIdx.x;
    const int T = blockDim.x;
    const int lane = t & 31;
    const int64_t src = row_index ? static_cast<int64_t>(row_index[row]) : static_cast<int64_t>(row);
    const __half* xr = x + src * ldx + static_cast<int64_t>(t) * E;

    float v[E];
    if constexpr (E >= 8) {
#pragma unroll
        for (int c = 0; c < E / 8; ++c) {
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(xr) + c);
            const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(h[i]);
                v[8 * c + 2 * i] = f.x;
                v[8 * c + 2 * i + 1] = f.y;
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < E; i += 2) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(xr + i));
            v[i] = f.x;
            v[i + 1] = f.y;
        }
    }
    if (ex.ch_mul) {   // channel-wise form: each product rounded to fp32 before the transform
#pragma unroll
        for (int i = 0; i < E; ++i) v[i] = __fmul_rn(v[i], __ldg(ex.ch_mul + t * E + i));
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
    if (mode == QM_GIVEN) {
        amax = __uint_as_float(*ex.tensor_amax);
    } else {
        amax = block_max(amax, red);
        if (mode == QM_AMAX) {
            if (t == 0) fold_amax(ex.tensor_amax, amax);
            return;
        }
    }
    float scale, inv;
    scale_of(amax, scale, inv);
    if (t == 0) o.scales[row] = scale;
    int bias = 0;
    if constexpr (E >= 8) {
#pragma unroll
        for (int c = 0; c < E / 8; ++c) {
            uint64_t p[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) p[i] = pk(v[8 * c + 2 * i], v[8 * c + 2 * i + 1]);
            emit_chunk<SINK>(p, inv, t * (E / 8) + c, o, row, K, bias);
        }
    } else {
        // short rows (K = 64, 128): E = 2 or 4 values per thread, written bytewise
        uint32_t code[E];
#pragma unroll
        for (int i = 0; i < E; ++i) code[i] = __float_as_uint(__fadd_rn(__fmul_rn(v[i], inv), MAGIC));
        if (SINK == SINK_NIBBLES) {
            uint8_t* qr = o.q + static_cast<int64_t>(row) * (K / 2) + static_cast<int64_t>(t) * (E / 2);
#pragma unroll
            for (int i = 0; i < E; i += 2) qr[i / 2] = static_cast<uint8_t>((code[i] & 0xFu) | ((code[i + 1] & 0xFu) << 4));
        } else {
            int8_t* xo = o.x8 + static_cast<int64_t>(row) * K + static_cast<int64_t>(t) * E;
            const bool low = ((t * E) % (2 * o.half)) < o.half;  // E divides the half-block: uniform per thread
#pragma unroll
            for (int i = 0; i < E; ++i) {
                const int qv = static_cast<int8_t>(code[i] & 0xFFu);
                xo[i] = static_cast<int8_t>(low ? qv * 16 : qv);
                if (low) bias += qv;
            }
        }
    }
    if (SINK == SINK_EXPANDED) {
        bias = block_sum(bias, reinterpret_cast<int*>(red));
        if (t == 0) o.bias_sum[row] = bias;
    }
}

// ---------------------------------------------------------------------------------------------
// Rotated rows of K = 4096, the hidden size of the backbone. 64 threads own a row (4 rows per CTA) and each
// holds 64 values as 32 packed pairs (2i, 2i+1): the stage inside a pair is scalar, the other five of a pass
// are packed add/sub on independent pairs. Pass A covers index bits 0-5 (h = 1..32) on 64 contiguous values;
// one transpose through shared memory (128-bit stores, swizzled so that neither side has a bank conflict)
// brings bits 6-11 into registers for pass B (h = 64..2048). The normalisation 1/sqrt(4096) = 2^-6 is exact,
// so it is folded into the scale instead of multiplying every element: fl(v * 2^-6) * fl(7 / (amax * 2^-6))
// and v * (fl(7 / (amax * 2^-6)) * 2^-6) are the same real product, rounded once.
// The codes return through shared memory as bytes, so that the row is written out in order.
constexpr int R4K = 4096, R4K_ROWS = 4, R4K_THREADS = 64 * R4K_ROWS;
constexpr int R4K_SMEM = R4K_ROWS * R4K * 4 + R4K_THREADS * 128;  // transpose buffers + staging

__device__ __forceinline__ void fwht64_pairs(uint64_t* P) {
    // stage on bit 0: inside each pair
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        float a, b;
        upk(P[i], a, b);
        P[i] = pk(__fadd_rn(a, b), __fsub_rn(a, b));
    }
    // stages on bits 1-5: pair i with pair i + h/2
#pragma unroll
    for (int hp = 1; hp < 32; hp <<= 1) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if ((i & hp) == 0) {
                const uint64_t a = P[i], b = P[i + hp];
                P[i] = add2(a, b);
                P[i + hp] = sub2(a, b);
            }
        }
    }
}

__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
// Barrier among the 64 threads of one row group (ids 1..4; id 0 is __syncthreads).
__device__ __forceinline__ void group_sync(int g) { asm volatile("bar.sync %0, 64;" ::"r"(g + 1) : "memory"); }

// Persistent: a CTA walks rows blockIdx.x*4 + g, + 4*gridDim.x, ... . Each thread stages its own 128 input bytes
// of the NEXT row with cp.async while the current row is transformed, so the HBM latency is off the critical path;
// the staging slots are private to a thread (it alone writes and reads them), so they need no barrier.
template <int SINK, int MODE = QM_TOKEN, bool MUL = false>
__global__ void __launch_bounds__(R4K_THREADS, 2) quantize_rotate4096_kernel(const __half* __restrict__ x, int M,
                                                                              int64_t ldx,
                                                                              const int32_t* __restrict__ row_index,
                                                                              QuantOut o, QuantEx ex) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    __shared__ float red_f[R4K_ROWS][2];
    __shared__ int red_i[R4K_ROWS][2];
    // With a handful of CTAs, letting the next kernel in early costs more than it saves: this kernel's CTAs are
    // large, so the SMs they sit on take the weight streamer's CTAs late, and those then finish last (measured at
    // 16 rows). One CTA, or a grid that fills the device (where the next kernel is a tensor-core linear whose
    // set-up then overlaps this kernel's tail), release their dependents at once.
    if (M <= R4K_ROWS || M > PDL_MAX_ROWS) pdl_launch_dependents();
    pdl_wait();   // x may be the output of the kernel before this one
    const int g = threadIdx.x >> 6, u = threadIdx.x & 63;  // row group, thread within the row
    float* buf = reinterpret_cast<float*>(smem_raw) + g * R4K;
    uint8_t* bytes = reinterpret_cast<uint8_t*>(buf);
    uint8_t* stage = smem_raw + R4K_ROWS * R4K * 4 + (g * 64 + u) * 128;  // this thread's 8 chunks, swizzled by u
    const uint32_t stage_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(stage));
    const int row_step = gridDim.x * R4K_ROWS;

    auto prefetch = [&](int row) {
        if (row < M) {
            const int64_t src = row_index ? static_cast<int64_t>(row_index[row]) : static_cast<int64_t>(row);
            const uint4* xr = reinterpret_cast<const uint4*>(x + src * ldx) + u * 8;
#pragma unroll
            for (int c = 0; c < 8; ++c) cp_async16(stage_u32 + ((c ^ (u & 7)) << 4), xr + c);
        }
        cp_async_commit();
    };

    int row = blockIdx.x * R4K_ROWS + g;
    prefetch(row);
    for (; row < M; row += row_step) {
        uint64_t P[32];
        cp_async_wait_all();
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            half8_to_pairs(*reinterpret_cast<const uint4*>(stage + ((c ^ (u & 7)) << 4)), P + 4 * c);
            if constexpr (MUL) scale_channels(P + 4 * c, ex.ch_mul, u * 8 + c);   // this thread's values are k = 64u ..
        }
        prefetch(row + row_step);  // the values above are in registers: the slots are free again
        fwht64_pairs(P);           // h = 1 .. 32

        // transpose: value r of thread u -> float u*64 + (r ^ ((u & 7) << 2)); 16 bytes = values 4g4 .. 4g4+3
#pragma unroll
        for (int g4 = 0; g4 < 16; ++g4) {
            uint32_t a0, a1, b0, b1;
            upk_bits(P[2 * g4], a0, a1);
            upk_bits(P[2 * g4 + 1], b0, b1);
            *reinterpret_cast<uint4*>(buf + u * 64 + ((g4 ^ (u & 7)) << 2)) = make_uint4(a0, a1, b0, b1);
        }
        group_sync(g);
        // thread u now takes value u of every thread r: element index r*64 + u
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int r0 = 2 * i, r1 = 2 * i + 1;
            const float lo = buf[r0 * 64 + (u ^ ((r0 & 7) << 2))];
            const float hi = buf[r1 * 64 + (u ^ ((r1 & 7) << 2))];
            P[i] = pk(lo, hi);
        }
        fwht64_pairs(P);  // h = 64 .. 2048

        float amax = 0.0f;
        if constexpr (MODE != QM_GIVEN) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                float a, b;
                upk(P[i], a, b);
                amax = fmaxf(amax, fmaxf(fabsf(a), fabsf(b)));
            }
            amax = warp_max(amax);
            if ((u & 31) == 0) red_f[g][u >> 5] = amax;
        }
        group_sync(g);  // also: every read of buf above is done before the bytes below overwrite it
        if constexpr (MODE == QM_GIVEN) amax = __uint_as_float(*ex.tensor_amax);
        else amax = fmaxf(red_f[g][0], red_f[g][1]) * 0.015625f;  // exact
        if constexpr (MODE == QM_AMAX) {
            if (u == 0) fold_amax(ex.tensor_amax, amax);
            group_sync(g);   // red_f is read: the next row may overwrite it
            continue;
        }
        float scale, inv;
        scale_of(amax, scale, inv);
        if (u == 0) o.scales[row] = scale;
        inv *= 0.015625f;  // exact
        const float magic = SINK == SINK_NIBBLES ? MAGIC8 : MAGIC;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            uint32_t t0, t1;
            round_pair(P[i], inv, magic, t0, t1);
            bytes[(2 * i) * 64 + u] = static_cast<uint8_t>(t0);
            bytes[(2 * i + 1) * 64 + u] = static_cast<uint8_t>(t1);
        }
        group_sync(g);
        // write-out: thread u takes the 16-code chunks u, u + 64, u + 128, u + 192 of the row
        int bias = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int c = u + 64 * i;
            const uint4 w = *reinterpret_cast<const uint4*>(bytes + 16 * c);
            if (SINK == SINK_NIBBLES) {
                reinterpret_cast<uint2*>(o.q + static_cast<int64_t>(row) * (R4K / 2))[c] =
                    make_uint2(nibbles_of(w.x, w.y), nibbles_of(w.z, w.w));
            } else {
                uint4 out = w;
                if ((c & 4) == 0) {  // codes 16c .. 16c+15 lie in the first 64 of their block of 128
                    bias = __dp4a(static_cast<int>(w.x), 0x01010101, bias);
                    bias = __dp4a(static_cast<int>(w.y), 0x01010101, bias);
                    bias = __dp4a(static_cast<int>(w.z), 0x01010101, bias);
                    bias = __dp4a(static_cast<int>(w.w), 0x01010101, bias);
                    out = make_uint4(times16(w.x), times16(w.y), times16(w.z), times16(w.w));
                }
                reinterpret_cast<uint4*>(o.x8 + static_cast<int64_t>(row) * R4K)[c] = out;
            }
        }
        if (SINK == SINK_EXPANDED) {
            bias = warp_sum(bias);
            if ((u & 31) == 0) red_i[g][u >> 5] = bias;
        }
        group_sync(g);  // bytes (and red_f / red_i) are read: the next row may overwrite them
        if (SINK == SINK_EXPANDED && u == 0) o.bias_sum[row] = red_i[g][0] + red_i[g][1];
    }
    cp_async_wait_all();
}

template <int E, int SINK>
static void launch_rotate(const __half* x, int M, int K, int64_t ldx, const int32_t* row_index, const QuantOut& o,
                          cudaStream_t s, QuantEx ex = QuantEx{nullptr, nullptr}, int mode = QM_TOKEN) {
    const int T = K / E;
    const float norm = static_cast<float>(1.0 / sqrt(static_cast<double>(K)));
    const size_t smem = (32 + (T > 32 ? static_cast<size_t>(K) : 0)) * sizeof(float);
    if (smem > 48 * 1024) {
        static PerDevice<int> setup;   // one per kernel instantiation; the limit covers the longest supported row
        if (setup.run([](int*) { return set_max_dynamic_smem(quantize_rows_rotate_kernel<E, SINK>, (32 + 16384) * 4); }) != SQAP_OK)
            return;
    }
    const cudaError_t e = launch_dependent(quantize_rows_rotate_kernel<E, SINK>, dim3(M), dim3(T), smem, s, x, K, ldx, row_index, norm, o,
                                           ex, mode);
    if (e != cudaSuccess) note_cuda_error(e);
}

template <int SINK, int MODE, bool MUL>
static sqap_status launch_rotate4096(const __half* x, int M, int64_t ldx, const int32_t* row_index, const QuantOut& o,
                                     const QuantEx& ex, cudaStream_t s) {
    static PerDevice<int> setup;   // one per kernel instantiation
    const sqap_status st = setup.run([](int*) { return set_max_dynamic_smem(quantize_rotate4096_kernel<SINK, MODE, MUL>, R4K_SMEM); });
    if (st != SQAP_OK) return st;
    int ctas = (M + R4K_ROWS - 1) / R4K_ROWS;
    const int resident = 2 * sm_count();
    if (ctas > resident) ctas = resident;
    const cudaError_t e = launch_dependent(quantize_rotate4096_kernel<SINK, MODE, MUL>, dim3(ctas), dim3(R4K_THREADS), R4K_SMEM, s,
                                           x, M, ldx, row_index, o, ex);
    if (e != cudaSuccess) note_cuda_error(e);
    return SQAP_OK;
}

template <int SINK>
static sqap_status launch_quantize(const __half* x, int M, int K, int64_t ldx, const int32_t* row_index, bool rotate,
                                   const QuantOut& o, cudaStream_t s) {
    if (rotate) {
        if (K == R4K) {
            const sqap_status st = launch_rotate4096<SINK, QM_TOKEN, false>(x, M, ldx, row_index, o, QuantEx{nullptr, nullptr}, s);
            if (st != SQAP_OK) return st;
        }
        // E elements per thread: 16 from K = 512 up (T = K/16 <= 1024), fewer for short rows so a full warp works
        else if (K >= 512) launch_rotate<16, SINK>(x, M, K, ldx, row_index, o, s);
        else if (K == 256) launch_rotate<8, SINK>(x, M, K, ldx, row_index, o, s);
        else if (K == 128) launch_rotate<4, SINK>(x, M, K, ldx, row_index, o, s);
        else launch_rotate<2, SINK>(x, M, K, ldx, row_index, o, s);
    } else {
        // the fewest threads per row that keep the whole row in registers (8 chunks of 8 values per thread)
        const int chunks = K / 8;
        if (chunks <= 32 * QUANT_NIT) launch_plain<SINK, 32>(x, M, K, ldx, row_index, o, s);
        else if (chunks <= 64 * QUANT_NIT) launch_plain<SINK, 64>(x, M, K, ldx, row_index, o, s);
        else if (chunks <= 128 * QUANT_NIT) launch_plain<SINK, 128>(x, M, K, ldx, row_index, o, s);
        else launch_plain<SINK, 256>(x, M, K, ldx, row_index, o, s);
    }
    count_launch();
    return check_launch();
}

sqap_status quantize_check_args(const void* x, int M, int K, int64_t ldx, uint32_t flags) {
    if (M < 0 || K <= 0 || ldx < K) return SQAP_ERR_INVALID;
    if (flags & ~SQAP_Q_ROTATE) return SQAP_ERR_INVALID;
    if (M == 0) return SQAP_OK;
    if (!x) return SQAP_ERR_INVALID;
    if (K % 32 != 0 || ldx % 8 != 0 || !aligned16(x)) return SQAP_ERR_ALIGN;
    if ((flags & SQAP_Q_ROTATE) && ((K & (K - 1)) != 0 || K < 64 || K > 16384)) return SQAP_ERR_UNSUPPORTED;
    return SQAP_OK;
}

sqap_status quantize_expanded(const __half* x, int M, int K, int64_t ldx, const int32_t* row_index, uint32_t flags,
                              int half, int8_t* x8, int32_t* bias_sum, float* scales, cudaStream_t s) {
    QuantOut o{nullptr, x8, bias_sum, scales, half};
    return launch_quantize<SINK_EXPANDED>(x, M, K, ldx, row_index, (flags & SQAP_Q_ROTATE) != 0, o, s);
}

// ---------------------------------------------------------------------------------------------
// The other activation granularities the paper names (one scale per TENSOR; a per-CHANNEL multiplier applied
// first) run in the same kernels as the per-token form (template parameters MODE / MUL above). The tensor-wise form
// takes two launches: the first folds every row's max-abs into one word, the second quantizes with it (its reads
// of x mostly hit L2). The word comes from a small pool in device memory, one slot per call in turn, cleared by a
// 4-byte memset on the call's stream: calls in flight on different streams use different slots unless more than
// TENSOR_SLOTS of them overlap; a captured CUDA graph keeps the slot it was captured with.
constexpr int TENSOR_SLOTS = 64;
__device__ unsigned g_tensor_amax[TENSOR_SLOTS];

static unsigned* tensor_amax_slot() {
    static PerDevice<unsigned*> base;
    unsigned* const* p = nullptr;
    if (base.run([](unsigned** out) {
            void* addr = nullptr;
            const cudaError_t e = cudaGetSymbolAddress(&addr, g_tensor_amax);
            if (e != cudaSuccess) {
                note_cuda_error(e);
                return SQAP_ERR_CUDA;
            }
            *out = static_cast<unsigned*>(addr);
            return SQAP_OK;
        }, &p) != SQAP_OK)
        return nullptr;
    static std::atomic<unsigned> next{0};
    return *p + next.fetch_add(1) % TENSOR_SLOTS;
}

template <int MODE, bool MUL>
static sqap_status launch_ex(const __half* x, int M, int K, int64_t ldx, const int32_t* row_index, bool rotate, const QuantOut& o,
                             const QuantEx& ex, cudaStream_t s) {
    constexpr int SINK = SINK_NIBBLES;
    if (rotate) {
        if (K == R4K) {
            const sqap_status st = launch_rotate4096<SINK, MODE, MUL>(x, M, ldx, row_index, o, ex, s);
            if (st != SQAP_OK) return st;
        } else if (K >= 512) launch_rotate<16, SINK>(x, M, K, ldx, row_index, o, s, ex, MODE);
        else if (K == 256) launch_rotate<8, SINK>(x, M, K, ldx, row_index, o, s, ex, MODE);
        else if (K == 128) launch_rotate<4, SINK>(x, M, K, ldx, row_index, o, s, ex, MODE);
        else launch_rotate<2, SINK>(x, M, K, ldx, row_index, o, s, ex, MODE);
    } else {
        const int chunks = K / 8;
        constexpr int nit = MUL ? QUANT_NIT / 2 : QUANT_NIT;   // chunks a thread holds between the passes
        if (chunks <= 32 * nit) launch_plain<SINK, 32, MODE, MUL>(x, M, K, ldx, row_index, o, s, ex);
        else if (chunks <= 64 * nit) launch_plain<SINK, 64, MODE, MUL>(x, M, K, ldx, row_index, o, s, ex);
        else if (chunks <= 128 * nit) launch_plain<SINK, 128, MODE, MUL>(x, M, K, ldx, row_index, o, s, ex);
        else launch_plain<SINK, 256, MODE, MUL>(x, M, K, ldx, row_index, o, s, ex);
    }
    count_launch();
    return check_launch();
}

template <int MODE>
static sqap_status launch_ex_mul(const __half* x, int M, int K, int64_t ldx, const int32_t* row_index, bool rotate,
                                 const QuantOut& o, const QuantEx& ex, cudaStream_t s) {
    return ex.ch_mul ? launch_ex<MODE, true>(x, M, K, ldx, row_index, rotate, o, ex, s)
                     : launch_ex<MODE, false>(x, M, K, ldx, row_index, rotate, o, ex, s);
}

}  // namespace sqap

extern "C" sqap_status sqap_quantize_act_ex(const void* x, int M, int K, int64_t ldx, const int32_t* row_index,
                                            uint32_t flags, const float* channel_mul, uint8_t* q_packed, float* scales,
                                            void* stream) {
    using namespace sqap;
    if (flags & ~(SQAP_Q_ROTATE | SQAP_Q_PER_TENSOR)) return SQAP_ERR_INVALID;
    if (!(flags & SQAP_Q_PER_TENSOR) && !channel_mul)   // nothing extended asked for
        return sqap_quantize_act(x, M, K, ldx, row_index, flags, q_packed, scales, stream);
    const sqap_status st = quantize_check_args(x, M, K, ldx, flags & SQAP_Q_ROTATE);
    if (st != SQAP_OK || M == 0) return st;
    if (!q_packed || !scales) return SQAP_ERR_INVALID;
    if (!aligned16(q_packed)) return SQAP_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(scales) & 3u) return SQAP_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(channel_mul) & 15u) return SQAP_ERR_ALIGN;   // read 16 bytes at a time
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool rotate = (flags & SQAP_Q_ROTATE) != 0;
    const __half* xh = static_cast<const __half*>(x);
    QuantOut o{q_packed, nullptr, nullptr, scales, 64};
    QuantEx ex{channel_mul, nullptr};
    if (!(flags & SQAP_Q_PER_TENSOR)) return launch_ex_mul<QM_TOKEN>(xh, M, K, ldx, row_index, rotate, o, ex, s);
    ex.tensor_amax = tensor_amax_slot();
    if (!ex.tensor_amax) return SQAP_ERR_CUDA;
    const cudaError_t e = cudaMemsetAsync(ex.tensor_amax, 0, sizeof(unsigned), s);
    if (e != cudaSuccess) {
        note_cuda_error(e);
        return SQAP_ERR_CUDA;
    }
    const sqap_status s1 = launch_ex_mul<QM_AMAX>(xh, M, K, ldx, row_index, rotate, o, ex, s);
    if (s1 != SQAP_OK) return s1;
    return launch_ex_mul<QM_GIVEN>(xh, M, K, ldx, row_index, rotate, o, ex, s);
}

extern "C" sqap_status sqap_quantize_act(const void* x, int M, int K, int64_t ldx, const int32_t* row_index,
                                         uint32_t flags, uint8_t* q_packed, float* scales, void* stream) {
    using namespace sqap;
    const sqap_status st = quantize_check_args(x, M, K, ldx, flags);
    if (st != SQAP_OK || M == 0) return st;
    if (!q_packed || !scales) return SQAP_ERR_INVALID;
    if (!aligned16(q_packed)) return SQAP_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(scales) & 3u) return SQAP_ERR_ALIGN;
    QuantOut o{q_packed, nullptr, nullptr, scales, 64};
    return launch_quantize<SINK_NIBBLES>(static_cast<const __half*>(x), M, K, ldx, row_index,
                                         (flags & SQAP_Q_ROTATE) != 0, o, static_cast<cudaStream_t>(stream));
}

// W4A4 linear: dispatcher, the activation expand pass, the CUDA-core GEMM (any shape) and the
// weight-streaming kernel for very few rows. The tensor-core kernel lives in linear_tc.cu.
#include "linear.cuh"
#include "quantize.cuh"

namespace sqap {

// ---------------------------------------------------------------------------------------------
// Expand pass: public nibble-packed activations -> int8 in the form the GEMM kernels multiply.
// One CTA per row. A 16-byte packed chunk (32 codes) becomes 32 int8.
__device__ __forceinline__ void expand_word(uint32_t w, bool times16, uint32_t& out0, uint32_t& out1) {
    uint32_t e, o;  // byte b of e = code 2b, of o = code 2b+1
    if (times16) {
        e = (w << 4) & 0xF0F0F0F0u;
        o = w & 0xF0F0F0F0u;
    } else {
        e = w & 0x0F0F0F0Fu;
        o = (w >> 4) & 0x0F0F0F0Fu;
        e |= (e & 0x08080808u) * 0x1Eu;  // sign-extend each nibble to a byte
        o |= (o & 0x08080808u) * 0x1Eu;
    }
    out0 = __byte_perm(e, o, 0x5140);
    out1 = __byte_perm(e, o, 0x7362);
}

__global__ void __launch_bounds__(128) expand_act_kernel(const uint8_t* __restrict__ q, int K, int half,
                                                         int8_t* __restrict__ x8, int32_t* __restrict__ bias_sum) {
    __shared__ int red[4];
    const int row = blockIdx.x;
    const uint4* src = reinterpret_cast<const uint4*>(q + static_cast<int64_t>(row) * (K / 2));
    uint4* dst = reinterpret_cast<uint4*>(x8 + static_cast<int64_t>(row) * K);
    int s16 = 0;
    for (int c = threadIdx.x; c < K / 32; c += blockDim.x) {
        const uint4 p = __ldg(src + c);
        const uint32_t w[4] = {p.x, p.y, p.z, p.w};
        uint32_t o[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int k = c * 32 + i * 8;
            const bool t16 = (k % (2 * half)) < half;
            expand_word(w[i], t16, o[2 * i], o[2 * i + 1]);
            if (t16) {
                s16 = __dp4a(static_cast<int>(o[2 * i]), 0x01010101, s16);
                s16 = __dp4a(static_cast<int>(o[2 * i + 1]), 0x01010101, s16);
            }
        }
        dst[2 * c] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[2 * c + 1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s16 += __shfl_xor_sync(0xffffffffu, s16, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s16;
    __syncthreads();
    if (threadIdx.x == 0) bias_sum[row] = (red[0] + red[1] + red[2] + red[3]) >> 4;
}

// Offsets (in codes, relative to the start of the row) that the low / high nibbles of packed 16-byte
// chunk c of a weight row cover.
__device__ __forceinline__ void chunk_k(int c, int half, int& lo_k, int& hi_k) {
    if (half == 64) {
        lo_k = (c >> 2) * 128 + (c & 3) * 16;
        hi_k = lo_k + 64;
    } else {
        lo_k = c * 32;
        hi_k = lo_k + 16;
    }
}

// ---------------------------------------------------------------------------------------------
// CUDA-core GEMM: 64x64 output tile per CTA, 128 codes of K per step, dp4a on int8 words held in
// shared memory. Runs every shape the API accepts; the reference point for the other kernels.
constexpr int ST_M = 64, ST_N = 64, ST_KW = 32;  // KW = 32-bit words of K per step

template <bool SWIGLU>
__global__ void __launch_bounds__(128) w4a4_simt_kernel(LinearArgs a) {
    __shared__ uint32_t Xs[ST_M][ST_KW + 1];
    __shared__ uint32_t Ws[ST_N][ST_KW + 1];
    __shared__ uint32_t Us[SWIGLU ? ST_N : 1][ST_KW + 1];
    const int tid = threadIdx.x;
    const int tn = tid & 7, tm = tid >> 3;
    const int m0 = blockIdx.y * ST_M, n0 = blockIdx.x * ST_N;
    int acc[4][8], accu[SWIGLU ? 4 : 1][8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            acc[i][j] = 0;
            if (SWIGLU) accu[i][j] = 0;
        }
    const int chunks_per_row = a.K / 32;  // packed 16-byte chunks in a weight row
    for (int k0 = 0; k0 < a.K; k0 += 128) {
        // activations: 64 rows x 8 chunks of 16 int8
        for (int i = tid; i < ST_M * 8; i += 128) {
            const int r = i >> 3, c = i & 7;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (m0 + r < a.M && k0 + c * 16 < a.K)
                v = __ldg(reinterpret_cast<const uint4*>(a.x8 + static_cast<int64_t>(m0 + r) * a.K + k0) + c);
            Xs[r][c * 4 + 0] = v.x;
            Xs[r][c * 4 + 1] = v.y;
            Xs[r][c * 4 + 2] = v.z;
            Xs[r][c * 4 + 3] = v.w;
        }
        // weights: 64 rows x 4 packed chunks, masked into two int8 chunks each
        for (int i = tid; i < ST_N * 4; i += 128) {
            const int r = i >> 2, cl = i & 3;
            const int c = k0 / 32 + cl;
            int lo_k, hi_k;
            chunk_k(c, a.half, lo_k, hi_k);
            lo_k -= k0;
            hi_k -= k0;
            uint4 v = make_uint4(0, 0, 0, 0), u = make_uint4(0, 0, 0, 0);
            const bool ok = (n0 + r < a.N) && (c < chunks_per_row);
            if (ok) {
                v = __ldg(reinterpret_cast<const uint4*>(a.w + static_cast<int64_t>(n0 + r) * (a.K / 2)) + c);
                if (SWIGLU) u = __ldg(reinterpret_cast<const uint4*>(a.w_up + static_cast<int64_t>(n0 + r) * (a.K / 2)) + c);
            }
            if (lo_k >= 0 && hi_k + 16 <= 128) {  // always true for valid chunks; keeps indices provably in range
                const uint32_t wv[4] = {v.x, v.y, v.z, v.w}, wu[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    Ws[r][lo_k / 4 + q] = wv[q] & 0x0F0F0F0Fu;
                    Ws[r][hi_k / 4 + q] = wv[q] & 0xF0F0F0F0u;
                    if (SWIGLU) {
                        Us[r][lo_k / 4 + q] = wu[q] & 0x0F0F0F0Fu;
                        Us[r][hi_k / 4 + q] = wu[q] & 0xF0F0F0F0u;
                    }
                }
            }
        }
        __syncthreads();
#pragma unroll 8
        for (int kk = 0; kk < ST_KW; ++kk) {
            int xa[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) xa[i] = static_cast<int>(Xs[tm * 4 + i][kk]);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int wb = static_cast<int>(Ws[tn + 8 * j][kk]);
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[i][j] = __dp4a(xa[i], wb, acc[i][j]);
                if (SWIGLU) {
                    const int ub = static_cast<int>(Us[tn + 8 * j][kk]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) accu[i][j] = __dp4a(xa[i], ub, accu[i][j]);
                }
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + tm * 4 + i;
        if (m >= a.M) continue;
        const int bs = a.bias_sum[m];
        const float sx = a.act_scales[m];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int n = n0 + tn + 8 * j;
            if (n >= a.N) continue;
            const int t = finish_acc(acc[i][j], bs);
            float y = dequant(t, sx, __half2float(a.w_scales[n]));
            if (SWIGLU) y = swiglu(y, dequant(finish_acc(accu[i][j], bs), sx, __half2float(a.w_up_scales[n])));
            store_out(a.out, static_cast<int64_t>(m) * a.ldo + n, a.out_dtype, y, t);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Weight-streaming kernel for M <= 8 (the single-token decode steps): HBM-bound on the packed
// weights, N*K/2 bytes per call. One warp owns one output channel and streams its row with
// 128-bit loads; the few activation rows are re-read through L1.
template <int MM, bool SWIGLU>
__global__ void __launch_bounds__(256) w4a4_gemv_kernel(LinearArgs a) {
    const int lane = threadIdx.x & 31;
    const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (n >= a.N) return;
    const uint4* wrow = reinterpret_cast<const uint4*>(a.w + static_cast<int64_t>(n) * (a.K / 2));
    const uint4* urow = SWIGLU ? reinterpret_cast<const uint4*>(a.w_up + static_cast<int64_t>(n) * (a.K / 2)) : nullptr;
    int acc[MM], accu[SWIGLU ? MM : 1];
#pragma unroll
    for (int m = 0; m < MM; ++m) {
        acc[m] = 0;
        if (SWIGLU) accu[m] = 0;
    }
    const int chunks = a.K / 32;
#pragma unroll 4
    for (int c = lane; c < chunks; c += 32) {
        const uint4 wv = __ldg(wrow + c);
        uint4 uv = make_uint4(0, 0, 0, 0);
        if (SWIGLU) uv = __ldg(urow + c);
        int lo_k, hi_k;
        chunk_k(c, a.half, lo_k, hi_k);
        const uint32_t w4[4] = {wv.x, wv.y, wv.z, wv.w}, u4[4] = {uv.x, uv.y, uv.z, uv.w};
#pragma unroll
        for (int m = 0; m < MM; ++m) {
            if (m < a.M) {
                const int8_t* xr = a.x8 + static_cast<int64_t>(m) * a.K;
                const uint4 xl = __ldg(reinterpret_cast<const uint4*>(xr + lo_k));
                const uint4 xh = __ldg(reinterpret_cast<const uint4*>(xr + hi_k));
                const int l4[4] = {(int)xl.x, (int)xl.y, (int)xl.z, (int)xl.w};
                const int h4[4] = {(int)xh.x, (int)xh.y, (int)xh.z, (int)xh.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[m] = __dp4a(l4[i], static_cast<int>(w4[i] & 0x0F0F0F0Fu), acc[m]);
                    acc[m] = __dp4a(h4[i], static_cast<int>(w4[i] & 0xF0F0F0F0u), acc[m]);
                    if (SWIGLU) {
                        accu[m] = __dp4a(l4[i], static_cast<int>(u4[i] & 0x0F0F0F0Fu), accu[m]);
                        accu[m] = __dp4a(h4[i], static_cast<int>(u4[i] & 0xF0F0F0F0u), accu[m]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int m = 0; m < MM; ++m) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            acc[m] += __shfl_xor_sync(0xffffffffu, acc[m], off);
            if (SWIGLU) accu[m] += __shfl_xor_sync(0xffffffffu, accu[m], off);
        }
    }
    if (lane == 0) {
        const float sw = __half2float(a.w_scales[n]);
#pragma unroll
        for (int m = 0; m < MM; ++m) {
            if (m < a.M) {
                const int bs = a.bias_sum[m];
                const float sx = a.act_scales[m];
                const int t = finish_acc(acc[m], bs);
                float y = dequant(t, sx, sw);
                if (SWIGLU) y = swiglu(y, dequant(finish_acc(accu[m], bs), sx, __half2float(a.w_up_scales[n])));
                store_out(a.out, static_cast<int64_t>(m) * a.ldo + n, a.out_dtype, y, t);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Single-row decode step (M = 1): the one activation row lives in registers. A lane always meets the same
// 16-byte weight chunks (lane, lane + 32, ...) of whatever row its warp streams, so it loads the 2 x 16
// activation bytes that go with each of them once and then only streams weights. An item is two weight rows (for a
// gate / up pair: the same row of both matrices), all their loads issued before the first dp4a; for the gated pair a
// warp keeps TWO items in flight in two register buffers and refills a buffer as soon as it has used it, so its
// loads never stop while it computes. The first item(s) are fetched before the dependency wait. Persistent warps
// stride over the output channels.
// FUSEQ: the kernel also quantizes the row (plain per-token quantizer, no rotation): every CTA repeats the small
// job (one 16-byte chunk or two per thread, two block-wide reductions) into shared memory while its first weight
// rows are in flight, which takes a whole kernel out of a decode step's chain; CTA 0 also leaves the expanded codes,
// their sum and the scale in the workspace, as the separate quantizer would have.
template <bool SWIGLU, int CPL, bool FUSEQ>
__global__ void __launch_bounds__(256, SWIGLU ? 2 : 3) w4a4_gemv1_kernel(LinearArgs a) {
    __shared__ __align__(16) int8_t xs[FUSEQ ? 32 * 32 * CPL : 16];
    __shared__ float red_f[8];
    __shared__ int red_i[8];
    const int lane = threadIdx.x & 31;
    const int gw = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), W = gridDim.x * (blockDim.x >> 5);
    const int chunks = a.K / 32;
    auto load_row = [&](const uint8_t* wbase, int n, uint4* wv) {
        const uint4* row = reinterpret_cast<const uint4*>(wbase + static_cast<int64_t>(n) * (a.K / 2));
#pragma unroll
        for (int i = 0; i < CPL; ++i) {
            const int c = lane + 32 * i;
            wv[i] = c < chunks ? __ldg(row + c) : make_uint4(0, 0, 0, 0);   // zero weights meet zero activations
        }
    };
    // item n: rows n and n + W of the matrix, or row n of the gate and of the up matrix
    auto load_item = [&](int n, uint4* p, uint4* q) {
        load_row(a.w, n, p);
        if (SWIGLU) load_row(a.w_up, n, q);
        else if (n + W < a.N) load_row(a.w, n + W, q);
    };
    const int step = (SWIGLU ? 1 : 2) * W;
    // The first items' weights do not depend on the kernel before this one (the quantizer): fetch them, then wait.
    // The gate / up pair (three to four items per warp at 11008 channels) runs two items deep: measured 11.5 -> 9.4 us.
    // The plain matrices (one or two items per warp) gain nothing from the second buffer and lose the third resident
    // CTA to its registers (QKV: 6.8 -> 7.1 us), so they keep one.
    constexpr bool DEEP = SWIGLU;
    uint4 A0[CPL], A1[CPL], B0[DEEP ? CPL : 1], B1[DEEP ? CPL : 1];
    if (gw < a.N) load_item(gw, A0, A1);
    if (DEEP && gw + step < a.N) load_item(gw + step, B0, B1);
    pdl_launch_dependents();
    pdl_wait();
    int bs;
    float sx;
    if (FUSEQ) {
        // the quantizer of quantize.cu for one row: max-abs, scale = amax / 7, inv = 7 / amax, codes by the magic add
        const int tid = threadIdx.x, wid = tid >> 5, n8 = a.K / 8;   // n8 <= 2 * 256 chunks of eight values
        const int64_t src = a.fuse_row_index ? static_cast<int64_t>(a.fuse_row_index[0]) : 0;
        const uint4* xr = reinterpret_cast<const uint4*>(a.fuse_x + src * a.fuse_ldx);
        uint4 c8[2];
        float amax = 0.0f;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int c = tid + 256 * i;
            c8[i] = make_uint4(0, 0, 0, 0);
            if (c < n8) {
                c8[i] = __ldg(xr + c);
                const __half2* h = reinterpret_cast<const __half2*>(&c8[i]);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float2 f = __half22float2(__habs2(h[q]));
                    amax = fmaxf(amax, fmaxf(f.x, f.y));
                }
            }
        }
        amax = warp_max(amax);
        if (lane == 0) red_f[wid] = amax;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < 8; ++w) amax = fmaxf(amax, red_f[w]);
        float inv;
        scale_of(amax, sx, inv);
        int bias = 0;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int c = tid + 256 * i;
            if (c < n8) {
                uint64_t p[4];
                uint32_t t[8];
                half8_to_pairs(c8[i], p);
#pragma unroll
                for (int q = 0; q < 4; ++q) round_pair(p[q], inv, MAGIC, t[2 * q], t[2 * q + 1]);
                uint32_t w0 = low_bytes(t[0], t[1], t[2], t[3]), w1 = low_bytes(t[4], t[5], t[6], t[7]);
                if (((8 * c) % (2 * a.half)) < a.half) {   // these codes meet low weight nibbles
                    bias = __dp4a(static_cast<int>(w0), 0x01010101, bias);
                    bias = __dp4a(static_cast<int>(w1), 0x01010101, bias);
                    w0 = times16(w0);
                    w1 = times16(w1);
                }
                reinterpret_cast<uint2*>(xs)[c] = make_uint2(w0, w1);
                if (blockIdx.x == 0) reinterpret_cast<uint2*>(const_cast<int8_t*>(a.x8))[c] = make_uint2(w0, w1);
            }
        }
        bias = warp_sum(bias);
        if (lane == 0) red_i[wid] = bias;
        __syncthreads();   // also: xs is complete
        bs = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) bs += red_i[w];
        if (blockIdx.x == 0 && tid == 0) {
            const_cast<int32_t*>(a.bias_sum)[0] = bs;
            const_cast<float*>(a.act_scales)[0] = sx;
        }
    } else {
        bs = a.bias_sum[0];
        sx = a.act_scales[0];
    }
    uint4 xl[CPL], xh[CPL];
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
        const int c = lane + 32 * i;
        xl[i] = xh[i] = make_uint4(0, 0, 0, 0);
        if (c < chunks) {
            int lo_k, hi_k;
            chunk_k(c, a.half, lo_k, hi_k);
            if (FUSEQ) {
                xl[i] = *reinterpret_cast<const uint4*>(xs + lo_k);
                xh[i] = *reinterpret_cast<const uint4*>(xs + hi_k);
            } else {
                xl[i] = __ldg(reinterpret_cast<const uint4*>(a.x8 + lo_k));
                xh[i] = __ldg(reinterpret_cast<const uint4*>(a.x8 + hi_k));
            }
        }
    }
    auto dot = [&](const uint4* wv) {
        int acc = 0;
#pragma unroll
        for (int i = 0; i < CPL; ++i) {
            const uint32_t w4[4] = {wv[i].x, wv[i].y, wv[i].z, wv[i].w};
            const int l4[4] = {(int)xl[i].x, (int)xl[i].y, (int)xl[i].z, (int)xl[i].w};
            const int h4[4] = {(int)xh[i].x, (int)xh[i].y, (int)xh[i].z, (int)xh[i].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                acc = __dp4a(l4[q], static_cast<int>(w4[q] & 0x0F0F0F0Fu), acc);
                acc = __dp4a(h4[q], static_cast<int>(w4[q] & 0xF0F0F0F0u), acc);
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        return acc;
    };
    auto finish = [&](int n, int raw_g, int raw_u) {
        if (lane != 0) return;
        const int t = finish_acc(raw_g, bs);
        float y = dequant(t, sx, __half2float(a.w_scales[n]));
        if (SWIGLU) y = swiglu(y, dequant(finish_acc(raw_u, bs), sx, __half2float(a.w_up_scales[n])));
        store_out(a.out, n, a.out_dtype, y, t);
    };
    auto do_item = [&](int n, const uint4* p, const uint4* q) {
        if (SWIGLU) {
            finish(n, dot(p), dot(q));
        } else {
            finish(n, dot(p), 0);
            if (n + W < a.N) finish(n + W, dot(q), 0);
        }
    };
    if (DEEP) {
        for (int n = gw; n < a.N; n += 2 * step) {
            do_item(n, A0, A1);
            if (n + 2 * step < a.N) load_item(n + 2 * step, A0, A1);
            if (n + step < a.N) {
                do_item(n + step, B0, B1);
                if (n + 3 * step < a.N) load_item(n + 3 * step, B0, B1);
            }
        }
    } else {
        // plain matrix: the two halves of an item are single rows n, n + W, ...; each half is refilled with the row two
        // places further as soon as it has been used, so a load is always in flight while the other half is multiplied
        for (int n = gw; n < a.N; n += 2 * W) {
            finish(n, dot(A0), 0);
            if (n + 2 * W < a.N) load_row(a.w, n + 2 * W, A0);
            if (n + W < a.N) {
                finish(n + W, dot(A1), 0);
                if (n + 3 * W < a.N) load_row(a.w, n + 3 * W, A1);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Single-row decode step with a row longer than 4096 codes (the down projection: 11008): the activation codes do
// not fit a lane's registers, so they live in shared memory, ordered the way the packed weight chunks meet them
// (lo[c] / hi[c]: the 16 codes that meet the low / high nibbles of packed chunk c, so a warp's reads are contiguous).
// A CTA owns a contiguous block of output channels (N / gridDim of them); its warps take the block's items (4096
// codes = 2 KB of one weight row) round-robin, so that rows of two or three items spread over several warps and every
// warp gets the same number of items to within one; two items are in flight per warp (two register buffers, used in
// turn), both fetched before the dependency wait. The items' sums meet in shared memory, and the CTA finishes its
// channels together at the end. FUSEQ as above (rows of up to
// MMA_FUSE_MAX_K codes); otherwise the expanded codes come from the workspace.
constexpr int GL_CPI = 4;   // 16-byte chunks per lane and item

template <bool FUSEQ>
__global__ void __launch_bounds__(256, 3) w4a4_gemv1_long_kernel(LinearArgs a) {
    extern __shared__ __align__(16) uint8_t xs_long[];   // K bytes: lo array, then hi array
    __shared__ float red_f[8];
    __shared__ int red_i[8];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int chunks = a.K / 32, nseg = (chunks + 32 * GL_CPI - 1) / (32 * GL_CPI);
    uint4* lo = reinterpret_cast<uint4*>(xs_long);
    uint4* hi = reinterpret_cast<uint4*>(xs_long + a.K / 2);
    auto load_item = [&](int n, int seg, uint4* wv) {
        const uint4* row = reinterpret_cast<const uint4*>(a.w + static_cast<int64_t>(n) * (a.K / 2));
#pragma unroll
        for (int i = 0; i < GL_CPI; ++i) {
            const int c = seg * 32 * GL_CPI + lane + 32 * i;
            wv[i] = c < chunks ? __ldg(row + c) : make_uint4(0, 0, 0, 0);
        }
    };
    // this CTA's channels [r0, r1) and this warp's items wid, wid + 8, ... of their (r1 - r0) * nseg items
    const int r0 = static_cast<int>(static_cast<int64_t>(blockIdx.x) * a.N / gridDim.x);
    const int r1 = static_cast<int>(static_cast<int64_t>(blockIdx.x + 1) * a.N / gridDim.x);
    const int n_items = (r1 - r0) * nseg;
    int* partial = reinterpret_cast<int*>(xs_long + a.K);   // one sum per item
    uint4 bufA[GL_CPI], bufB[GL_CPI];   // two items in flight, both fetched before the dependency wait
    auto item_row = [&](int j) { return r0 + (wid + 8 * j) / nseg; };
    auto item_seg = [&](int j) { return (wid + 8 * j) % nseg; };
    const int n_mine = (n_items - wid + 7) / 8;
    if (0 < n_mine) load_item(item_row(0), item_seg(0), bufA);
    if (1 < n_mine) load_item(item_row(1), item_seg(1), bufB);
    pdl_launch_dependents();
    pdl_wait();
    int bs;
    float sx;
    // place of the 16 codes k = 16j .. 16j+15 of the row: block b = k / 128; offsets below 64 meet low nibbles
    auto place = [&](int j) -> uint4* {
        const int k = 16 * j, b = k >> 7, o = k & 127;
        return (o < 64 ? lo : hi) + b * 4 + ((o & 63) >> 4);
    };
    if (FUSEQ) {
        // the quantizer of quantize.cu for one row: max-abs, scale = amax / 7, inv = 7 / amax, codes by the magic add
        const int n16 = a.K / 16;
        const int64_t src = a.fuse_row_index ? static_cast<int64_t>(a.fuse_row_index[0]) : 0;
        const uint4* xr = reinterpret_cast<const uint4*>(a.fuse_x + src * a.fuse_ldx);
        float amax = 0.0f;
        for (int c = tid; c < 2 * n16; c += 256) {
            const uint4 v = __ldg(xr + c);
            const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 f = __half22float2(__habs2(h[q]));
                amax = fmaxf(amax, fmaxf(f.x, f.y));
            }
        }
        amax = warp_max(amax);
        if (lane == 0) red_f[wid] = amax;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < 8; ++w) amax = fmaxf(amax, red_f[w]);
        float inv;
        scale_of(amax, sx, inv);
        int bias = 0;
        for (int j = tid; j < n16; j += 256) {
            uint32_t wd[4];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                uint64_t p[4];
                uint32_t t[8];
                half8_to_pairs(__ldg(xr + 2 * j + e), p);
#pragma unroll
                for (int q = 0; q < 4; ++q) round_pair(p[q], inv, MAGIC, t[2 * q], t[2 * q + 1]);
                wd[2 * e] = low_bytes(t[0], t[1], t[2], t[3]);
                wd[2 * e + 1] = low_bytes(t[4], t[5], t[6], t[7]);
            }
            if (((16 * j) & 127) < 64) {   // these codes meet low weight nibbles
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    bias = __dp4a(static_cast<int>(wd[e]), 0x01010101, bias);
                    wd[e] = times16(wd[e]);
                }
            }
            const uint4 out = make_uint4(wd[0], wd[1], wd[2], wd[3]);
            *place(j) = out;
            if (blockIdx.x == 0) reinterpret_cast<uint4*>(const_cast<int8_t*>(a.x8))[j] = out;
        }
        bias = warp_sum(bias);
        if (lane == 0) red_i[wid] = bias;
        __syncthreads();   // also: the codes are complete
        bs = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) bs += red_i[w];
        if (blockIdx.x == 0 && tid == 0) {
            const_cast<int32_t*>(a.bias_sum)[0] = bs;
            const_cast<float*>(a.act_scales)[0] = sx;
        }
    } else {
        for (int j = tid; j < a.K / 16; j += 256) *place(j) = __ldg(reinterpret_cast<const uint4*>(a.x8) + j);
        bs = a.bias_sum[0];
        sx = a.act_scales[0];
        __syncthreads();
    }
    auto do_item = [&](int it, uint4* wv) {
        const int seg = item_seg(it);
        int acc = 0;
#pragma unroll
        for (int i = 0; i < GL_CPI; ++i) {
            const int c = seg * 32 * GL_CPI + lane + 32 * i;
            if (c < chunks) {
                const uint4 xl = lo[c], xh = hi[c];
                const uint32_t w4[4] = {wv[i].x, wv[i].y, wv[i].z, wv[i].w};
                const int l4[4] = {(int)xl.x, (int)xl.y, (int)xl.z, (int)xl.w};
                const int h4[4] = {(int)xh.x, (int)xh.y, (int)xh.z, (int)xh.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    acc = __dp4a(l4[q], static_cast<int>(w4[q] & 0x0F0F0F0Fu), acc);
                    acc = __dp4a(h4[q], static_cast<int>(w4[q] & 0xF0F0F0F0u), acc);
                }
            }
        }
        acc = warp_sum(acc);
        if (lane == 0) partial[wid + 8 * it] = acc;
        if (it + 2 < n_mine) load_item(item_row(it + 2), item_seg(it + 2), wv);
    };
    for (int it = 0; it < n_mine; it += 2) {
        do_item(it, bufA);
        if (it + 1 < n_mine) do_item(it + 1, bufB);
    }
    __syncthreads();
    for (int r = tid; r < r1 - r0; r += 256) {
        int acc = 0;
        for (int sg = 0; sg < nseg; ++sg) acc += partial[r * nseg + sg];
        const int n = r0 + r;
        const int t = finish_acc(acc, bs);
        store_out(a.out, n, a.out_dtype, dequant(t, sx, __half2float(a.w_scales[n])), t);
    }
}

static void launch_gemv1_long(const LinearArgs& a, cudaStream_t s) {
    const int blocks = sm_count() * 3;
    const int need = (a.N + 7) / 8;
    int grid = need < blocks ? need : blocks;
    const int nseg = (a.K / 32 + 32 * GL_CPI - 1) / (32 * GL_CPI);
    // shared memory: the codes (K <= MMA_FUSE_MAX_K bytes) and one partial sum per item of a CTA, within the default
    // dynamic limit; a matrix with more channels than that allows per CTA gets more CTAs than are resident at once
    const int rows_cap = (48 * 1024 - a.K) / (4 * nseg) - 1;
    if ((a.N + grid - 1) / grid > rows_cap) grid = (a.N + rows_cap - 1) / rows_cap;
    const size_t smem = static_cast<size_t>(a.K) + sizeof(int) * static_cast<size_t>((a.N + grid - 1) / grid + 1) * nseg;
    cudaError_t e;
    if (a.fuse_x) e = launch_dependent(w4a4_gemv1_long_kernel<true>, dim3(grid), dim3(256), smem, s, a);
    else e = launch_dependent(w4a4_gemv1_long_kernel<false>, dim3(grid), dim3(256), smem, s, a);
    if (e != cudaSuccess) note_cuda_error(e);
}

template <int CPL>
static void launch_gemv1(const LinearArgs& a, cudaStream_t s) {
    const int blocks = sm_count() * (a.w_up ? 2 : 3);   // resident CTAs per SM: the gated pair holds two register buffers
    const int need = (a.N + 7) / 8;
    const int grid = need < blocks ? need : blocks;
    cudaError_t e;
    if (a.fuse_x) {
        if (a.w_up) e = launch_dependent(w4a4_gemv1_kernel<true, CPL, true>, dim3(grid), dim3(256), 0, s, a);
        else e = launch_dependent(w4a4_gemv1_kernel<false, CPL, true>, dim3(grid), dim3(256), 0, s, a);
    } else {
        if (a.w_up) e = launch_dependent(w4a4_gemv1_kernel<true, CPL, false>, dim3(grid), dim3(256), 0, s, a);
        else e = launch_dependent(w4a4_gemv1_kernel<false, CPL, false>, dim3(grid), dim3(256), 0, s, a);
    }
    if (e != cudaSuccess) note_cuda_error(e);
}

template <int MM>
static void launch_gemv(const LinearArgs& a, cudaStream_t s) {
    const int warps = 8;
    const int blocks = (a.N + warps - 1) / warps;
    if (a.w_up) w4a4_gemv_kernel<MM, true><<<blocks, warps * 32, 0, s>>>(a);
    else w4a4_gemv_kernel<MM, false><<<blocks, warps * 32, 0, s>>>(a);
}

static size_t round256(size_t v) { return (v + 255) / 256 * 256; }

}  // namespace sqap

namespace sqap {

enum LinearPath { PATH_SIMT, PATH_TC, PATH_TC_TS, PATH_TC_PAIR, PATH_TC_SPLITK, PATH_GEMV, PATH_MMA };

// Argument rules shared by the entry points that run a linear (everything except the activation side).
static sqap_status check_linear_args(int M, const sqap_weights* w, const sqap_weights* w_up, const void* out,
                                     int64_t ldo, int out_dtype, uint32_t flags, uint32_t allowed_flags) {
    if (M < 0 || !w) return SQAP_ERR_INVALID;
    if (out_dtype != SQAP_FP16 && out_dtype != SQAP_BF16 && out_dtype != SQAP_I32) return SQAP_ERR_INVALID;
    if (flags & ~(allowed_flags | SQAP_L_KSPLIT_MASK)) return SQAP_ERR_INVALID;
    if ((flags & SQAP_L_KSPLIT_MASK) && !(flags & SQAP_L_FORCE_TCGEN05_SPLITK)) return SQAP_ERR_INVALID;
    const uint32_t force = flags & SQAP_L_FORCE_MASK;
    if ((force & (force - 1)) != 0) return SQAP_ERR_INVALID;  // at most one forced kernel
    if (w_up && (w_up->N != w->N || w_up->K != w->K || w_up->half != w->half || w_up->device != w->device))
        return SQAP_ERR_INVALID;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return SQAP_ERR_CUDA;
    }
    if (dev != w->device) return SQAP_ERR_INVALID;   // the packed weights live on another device than the current one
    if (w_up && out_dtype == SQAP_I32) return SQAP_ERR_INVALID;
    if (ldo < w->N) return SQAP_ERR_INVALID;
    if (M == 0) return SQAP_OK;
    if (!out) return SQAP_ERR_INVALID;
    const int esz = out_dtype == SQAP_I32 ? 4 : 2;
    if (!aligned16(out) || (ldo * esz) % 16 != 0) return SQAP_ERR_ALIGN;
    return SQAP_OK;
}

static LinearArgs make_args(void* workspace, const float* act_scales, int M, const sqap_weights* w,
                            const sqap_weights* w_up, void* out, int64_t ldo, int out_dtype) {
    LinearArgs a;
    a.x8 = static_cast<int8_t*>(workspace);
    a.bias_sum = reinterpret_cast<int32_t*>(static_cast<uint8_t*>(workspace) + round256(static_cast<size_t>(M) * w->K));
    a.act_scales = act_scales;
    a.M = M;
    a.N = w->N;
    a.K = w->K;
    a.half = w->half;
    a.w = w->packed;
    a.w_scales = w->scales;
    a.w_up = w_up ? w_up->packed : nullptr;
    a.w_up_scales = w_up ? w_up->scales : nullptr;
    a.w_handle = w;
    a.w_up_handle = w_up;
    a.out = out;
    a.ldo = ldo;
    a.out_dtype = out_dtype;
    a.fuse_x = nullptr;
    a.fuse_ldx = 0;
    a.fuse_row_index = nullptr;
    return a;
}

static sqap_status pick_path(const LinearArgs& a, uint32_t flags, LinearPath* path) {
    if (flags & SQAP_L_FORCE_SIMT) *path = PATH_SIMT;
    else if (flags & SQAP_L_FORCE_GEMV) {
        if (a.M > 8) return SQAP_ERR_UNSUPPORTED;
        *path = PATH_GEMV;
    } else if (flags & SQAP_L_FORCE_TCGEN05) {
        if (!tcgen05_supports(a)) return SQAP_ERR_UNSUPPORTED;
        *path = PATH_TC;
    } else if (flags & SQAP_L_FORCE_TCGEN05_TS) {
        if (!tcgen05_supports(a)) return SQAP_ERR_UNSUPPORTED;
        *path = PATH_TC_TS;
    } else if (flags & SQAP_L_FORCE_TCGEN05_PAIR) {
        if (!tcgen05_supports(a)) return SQAP_ERR_UNSUPPORTED;
        *path = PATH_TC_PAIR;
    } else if (flags & SQAP_L_FORCE_TCGEN05_SPLITK) {
        if (!tcgen05_supports(a)) return SQAP_ERR_UNSUPPORTED;
        *path = PATH_TC_SPLITK;
    } else if (flags & SQAP_L_FORCE_MMA) {
        if (!mma_stream_supports(a)) return SQAP_ERR_UNSUPPORTED;
        *path = PATH_MMA;
    } else {
        // tensor-memory kernels: CTA pairs once there are enough token tiles to fill them, one CTA per tile below
        // the weight-streaming kernel re-reads the activations per row of M, so beyond two rows it only wins where
        // the tensor-memory kernel has too few weight tiles to fill the SMs
        const bool tc_ok = tcgen05_supports(a);
        const int w_tiles = (a.w_up ? 2 * a.N : a.N) / 128;
        // A handful of rows: the register-MMA streamer (its MMA rate holds up to ~16 rows; where the tensor-memory
        // kernel has too few weight tiles to fill the SMs it stays ahead up to 32). One row: the dp4a streamers
        // (codes in registers up to 4096 of them; in shared memory up to 16384 for plain matrices).
        const bool one_row_in_registers = a.M == 1 && (a.K / 32 <= 32 * 4 || (a.half == 64 && a.K <= MMA_FUSE_MAX_K && !a.w_up));
        const bool stream = mma_stream_supports(a) && !one_row_in_registers && (a.M <= 16 || w_tiles < 64);
        const bool gemv = !stream && a.M <= 8 && (!tc_ok || a.M <= 2 || (a.M <= 4 && w_tiles < 64));
        // CTA pairs fetch each token once per 256 weight rows: ahead from ~144 tokens on when there are enough pairs
        const bool pairs = a.M >= 512 || (a.M >= 144 && w_tiles >= 64) || (a.M > 320 && a.K >= 8192);
        // Few weight tiles and a long K (the down projection of one observation: 32 tiles x 43 stages): one cluster
        // per tile with K split over its CTAs; measured ahead of both other kernels there, behind them elsewhere
        // (its two cluster barriers and the exchange of partial sums cost about as much as 8 stages).
        const bool split_k = !pairs && a.M >= 64 && a.M <= 320 && w_tiles < 64 && a.K >= 8192;   // beyond ~320 rows the pairs win
        *path = stream ? PATH_MMA : gemv ? PATH_GEMV
                : (tc_ok ? (pairs ? PATH_TC_PAIR : split_k ? PATH_TC_SPLITK : PATH_TC_TS) : PATH_SIMT);
    }
    return SQAP_OK;
}

static sqap_status run_gemm(const LinearArgs& a, LinearPath path, uint32_t flags, cudaStream_t s) {
    if (path == PATH_TC) return launch_linear_tcgen05(a, s);
    if (path == PATH_TC_SPLITK)
        return launch_linear_tcgen05_splitk(a, static_cast<int>((flags & SQAP_L_KSPLIT_MASK) >> 8), s);
    if (path == PATH_TC_TS) return launch_linear_tcgen05_ts(a, s);
    if (path == PATH_TC_PAIR) return launch_linear_tcgen05_pair(a, s);
    if (path == PATH_MMA) return launch_linear_mma_stream(a, s);
    if (path == PATH_GEMV) {
        const int chunks = a.K / 32;
        // rows up to 4096 codes: activation row in registers; longer rows would not amortise loading it
        if (a.M == 1 && chunks <= 32 * 4) launch_gemv1<4>(a, s);
        else if (a.M == 1 && a.half == 64 && a.K <= MMA_FUSE_MAX_K && !a.w_up) launch_gemv1_long(a, s);
        else if (a.M == 1) launch_gemv<1>(a, s);
        else if (a.M == 2) launch_gemv<2>(a, s);
        else if (a.M <= 4) launch_gemv<4>(a, s);
        else launch_gemv<8>(a, s);
    } else {
        dim3 grid((a.N + ST_N - 1) / ST_N, (a.M + ST_M - 1) / ST_M);
        if (a.w_up) w4a4_simt_kernel<true><<<grid, 128, 0, s>>>(a);
        else w4a4_simt_kernel<false><<<grid, 128, 0, s>>>(a);
    }
    count_launch();
    return check_launch();
}

}  // namespace sqap

extern "C" {

size_t sqap_workspace_bytes(int M, int N, int K, uint32_t flags) {
    (void)N;
    (void)flags;
    if (M <= 0 || K <= 0) return 256;
    return sqap::round256(static_cast<size_t>(M) * K) + sqap::round256(sizeof(int32_t) * static_cast<size_t>(M));
}

sqap_status sqap_w4a4_linear(const uint8_t* q_packed, const float* act_scales, int M, const sqap_weights* w,
                             const sqap_weights* w_up, void* out, int64_t ldo, int out_dtype, uint32_t flags,
                             void* workspace, size_t workspace_bytes, void* stream) {
    using namespace sqap;
    sqap_status st = check_linear_args(M, w, w_up, out, ldo, out_dtype, flags,
                                       SQAP_L_FORCE_MASK | SQAP_L_REUSE_EXPANDED);
    if (st != SQAP_OK || M == 0) return st;
    if (!q_packed || !act_scales || !workspace) return SQAP_ERR_INVALID;
    if (!aligned16(q_packed)) return SQAP_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SQAP_ERR_ALIGN;
    if (workspace_bytes < sqap_workspace_bytes(M, w->N, w->K, flags)) return SQAP_ERR_NOMEM;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    const LinearArgs a = make_args(workspace, act_scales, M, w, w_up, out, ldo, out_dtype);
    LinearPath path;
    st = pick_path(a, flags, &path);
    if (st != SQAP_OK) return st;

    if (!(flags & SQAP_L_REUSE_EXPANDED)) {
        expand_act_kernel<<<M, 128, 0, s>>>(q_packed, a.K, a.half, const_cast<int8_t*>(a.x8),
                                            const_cast<int32_t*>(a.bias_sum));
        count_launch();
        st = check_launch();
        if (st != SQAP_OK) return st;
    }
    return run_gemm(a, path, flags, s);
}

size_t sqap_quantize_linear_workspace_bytes(int M, int N, int K) {
    if (M <= 0 || K <= 0) return 256;
    return sqap_workspace_bytes(M, N, K, 0) + sqap::round256(sizeof(float) * static_cast<size_t>(M));
}

sqap_status sqap_quantize_linear(const void* x, int M, int64_t ldx, const int32_t* row_index, uint32_t qflags,
                                 const sqap_weights* w, const sqap_weights* w_up, void* out, int64_t ldo,
                                 int out_dtype, uint32_t lflags, void* workspace, size_t workspace_bytes,
                                 void* stream) {
    using namespace sqap;
    sqap_status st = check_linear_args(M, w, w_up, out, ldo, out_dtype, lflags, SQAP_L_FORCE_MASK);
    if (st != SQAP_OK) return st;
    st = quantize_check_args(x, M, w->K, ldx, qflags);
    if (st != SQAP_OK || M == 0) return st;
    if (!workspace) return SQAP_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SQAP_ERR_ALIGN;
    if (workspace_bytes < sqap_quantize_linear_workspace_bytes(M, w->N, w->K)) return SQAP_ERR_NOMEM;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    float* scales = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + sqap_workspace_bytes(M, w->N, w->K, 0));
    LinearArgs a = make_args(workspace, scales, M, w, w_up, out, ldo, out_dtype);
    LinearPath path;
    st = pick_path(a, lflags, &path);
    if (st != SQAP_OK) return st;
    const bool one_plain_row = M == 1 && !(qflags & SQAP_Q_ROTATE);
    if (one_plain_row && ((path == PATH_GEMV && (a.K / 32 <= 32 * 4 || (a.half == 64 && a.K <= MMA_FUSE_MAX_K && !w_up))) ||
                          (path == PATH_MMA && a.K <= MMA_FUSE_MAX_K))) {
        // one row, no rotation: the streamer quantizes the row itself (one kernel instead of two)
        a.fuse_x = static_cast<const __half*>(x);
        a.fuse_ldx = ldx;
        a.fuse_row_index = row_index;
        return run_gemm(a, path, lflags, s);
    }
    st = quantize_expanded(static_cast<const __half*>(x), M, a.K, ldx, row_index, qflags, a.half,
                           const_cast<int8_t*>(a.x8), const_cast<int32_t*>(a.bias_sum), scales, s);
    if (st != SQAP_OK) return st;
    return run_gemm(a, path, lflags, s);
}

}  // extern "C"

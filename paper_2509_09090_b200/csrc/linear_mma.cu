// W4A4 linear for a handful of tokens (3 <= M <= 32): the call is bound by the HBM stream of the packed
// weights (N*K/2 bytes), so the kernel is a weight streamer. Nothing is staged: every lane pulls 16-byte pieces
// of weight rows straight from global memory into registers, masks the two nibble planes apart (two ANDs per
// word) and feeds them to register-level int8 MMAs (m16n8k32) against the expanded int8 activations, which stay
// in L1. The register MMA is here only because dp4a cannot keep 16-32 tokens' worth of arithmetic under the
// HBM time; the tensor-memory kernels need shared-memory and TMEM pipelines whose fill and drain cost more
// than this whole call.
//
// Work split: a row block is 16 weight rows (with SwiGLU: the same 16 rows of the gate and of the up matrix); the
// eight warps of a CTA take its 128-code blocks of K round-robin and add their partial sums through shared memory
// (integer sums: the order cannot change the result). CTAs are persistent, two per SM, and walk the row blocks.
//
// Fragment bookkeeping (g = lane / 4, t = lane % 4). The MMA multiplies A (16 rows x 32 k) by B (32 k x 8
// columns); a lane supplies A words for rows g and g + 8 at k-slots 4t..4t+3 and 16+4t..16+4t+3 and B words for
// column g at the same k-slots. Which codes sit in which k-slot is free as long as A and B agree, so lane t takes
// the 16-byte chunk t of the block's 64 packed bytes: word i of that chunk carries codes 16t+4i..16t+4i+3 in its
// low nibbles and codes 64+16t+4i.. in its high nibbles, and meets words i of the activation row at byte offsets
// 16t and 64+16t of the block. Four MMAs per block and token group: (words 0,1 low), (2,3 low), (0,1 high),
// (2,3 high).
#include "linear.cuh"
#include "quantize.cuh"

namespace sqap {

namespace mmas {

constexpr int MMA_WARPS = 8;

__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Weights are read once: keep them out of L1, which holds the activations.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// One block of 128 codes: rows (wa: g, wb: g + 8) against NG token groups.
template <int NG>
__device__ __forceinline__ void block_mma(int (&acc)[NG][4], const uint4& wa, const uint4& wb, const uint4 (&xl)[NG],
                                          const uint4 (&xh)[NG]) {
    constexpr uint32_t L = 0x0F0F0F0Fu, H = 0xF0F0F0F0u;
#pragma unroll
    for (int j = 0; j < NG; ++j) {
        mma_s8(acc[j], wa.x & L, wb.x & L, wa.y & L, wb.y & L, xl[j].x, xl[j].y);
        mma_s8(acc[j], wa.z & L, wb.z & L, wa.w & L, wb.w & L, xl[j].z, xl[j].w);
        mma_s8(acc[j], wa.x & H, wb.x & H, wa.y & H, wb.y & H, xh[j].x, xh[j].y);
        mma_s8(acc[j], wa.z & H, wb.z & H, wa.w & H, wb.w & H, xh[j].z, xh[j].w);
    }
}

// A warp's share of one row block is cut into items of KU blocks of 128 codes; the weights of an item are loaded
// one item ahead of the MMAs that use them (two register buffers), also across row blocks, so that the stream
// from HBM does not stop while a row block is reduced and written out.
template <int KU, bool SWIGLU>
struct ItemWeights {
    uint4 a[KU], b[KU];                                   // rows g and g + 8
    uint4 ua[SWIGLU ? KU : 1], ub[SWIGLU ? KU : 1];       // the same rows of the up matrix
};

// NG = token groups of 8 (M <= 8 * NG). Persistent: CTA c takes row blocks c, c + gridDim.x, ...
// FUSEQ (one row only): the kernel quantizes the activation row itself, as the single-row streamer of linear.cu
// does: every CTA repeats the plain per-token quantizer into (dynamic) shared memory, K bytes, while its first
// weights are in flight; CTA 0 also writes the expanded form to the workspace.
template <int NG, bool SWIGLU, bool FUSEQ = false>
__global__ void __launch_bounds__(MMA_WARPS * 32, 2) w4a4_mma_kernel(LinearArgs a) {
    extern __shared__ __align__(16) int8_t xs[];   // FUSEQ: the expanded codes of the row
    __shared__ float q_red_f[MMA_WARPS];
    __shared__ int q_red_i[MMA_WARPS];
    __shared__ int q_bias;
    __shared__ float q_scale;
    constexpr int SETS = SWIGLU ? 2 : 1;
    constexpr int KU = SWIGLU ? (NG <= 2 ? 2 : 1) : (NG <= 2 ? 4 : 2);
    __shared__ int red[MMA_WARPS][SETS * NG * 4][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int64_t row_bytes = a.K / 2;
    const int blocks = a.K / 128;
    const int items_per_rb = ((blocks + MMA_WARPS - 1) / MMA_WARPS + KU - 1) / KU;
    const int n_rb = (a.N + 15) / 16;
    const int my_rbs = static_cast<int>(blockIdx.x) < n_rb ? (n_rb - 1 - static_cast<int>(blockIdx.x)) / static_cast<int>(gridDim.x) + 1 : 0;
    const int total_items = my_rbs * items_per_rb;

    const uint4* xp[NG];
    bool xok[NG];
#pragma unroll
    for (int j = 0; j < NG; ++j) {
        const int m = 8 * j + g;
        xok[j] = m < a.M;
        xp[j] = reinterpret_cast<const uint4*>(a.x8 + static_cast<int64_t>(xok[j] ? m : 0) * a.K) + t;
    }
    int acc[NG][4], accu[SWIGLU ? NG : 1][4];
    auto clear_acc = [&]() {
#pragma unroll
        for (int j = 0; j < NG; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                acc[j][c] = 0;
                if (SWIGLU) accu[j][c] = 0;
            }
    };
    clear_acc();

    // block b of item (ci, u): the warps take the blocks of a row round-robin
    auto block_of = [&](int ci, int u) { return warp + MMA_WARPS * (ci * KU + u); };

    int l_rb = blockIdx.x, l_ci = 0;     // load cursor: row block and item within it
    auto load_item = [&](ItemWeights<KU, SWIGLU>& w) {
        const int n0 = l_rb * 16;
        // rows past N are clamped for the loads and never stored
        const int64_t o0 = static_cast<int64_t>(min(n0 + g, a.N - 1)) * row_bytes, o1 = static_cast<int64_t>(min(n0 + g + 8, a.N - 1)) * row_bytes;
#pragma unroll
        for (int u = 0; u < KU; ++u) {
            const int b = block_of(l_ci, u);
            w.a[u] = w.b[u] = make_uint4(0, 0, 0, 0);
            if (SWIGLU) w.ua[u] = w.ub[u] = make_uint4(0, 0, 0, 0);
            if (b < blocks) {
                w.a[u] = ld_stream(reinterpret_cast<const uint4*>(a.w + o0) + 4 * b + t);
                w.b[u] = ld_stream(reinterpret_cast<const uint4*>(a.w + o1) + 4 * b + t);
                if (SWIGLU) {
                    w.ua[u] = ld_stream(reinterpret_cast<const uint4*>(a.w_up + o0) + 4 * b + t);
                    w.ub[u] = ld_stream(reinterpret_cast<const uint4*>(a.w_up + o1) + 4 * b + t);
                }
            }
        }
        if (++l_ci == items_per_rb) { l_ci = 0; l_rb += gridDim.x; }
    };

    int c_rb = blockIdx.x, c_ci = 0;     // compute cursor
    auto compute_item = [&](const ItemWeights<KU, SWIGLU>& w) {
#pragma unroll
        for (int u = 0; u < KU; ++u) {
            const int b = block_of(c_ci, u);
            if (b < blocks) {            // uniform over the warp
                uint4 xl[NG], xh[NG];
#pragma unroll
                for (int j = 0; j < NG; ++j) {
                    xl[j] = xh[j] = make_uint4(0, 0, 0, 0);   // tokens past M contribute zeros
                    if (xok[j]) {
                        if (FUSEQ) {   // one row: token 0 only
                            xl[j] = *reinterpret_cast<const uint4*>(xs + 128 * b + 16 * t);
                            xh[j] = *reinterpret_cast<const uint4*>(xs + 128 * b + 64 + 16 * t);
                        } else {
                            xl[j] = __ldg(xp[j] + 8 * b);
                            xh[j] = __ldg(xp[j] + 8 * b + 4);
                        }
                    }
                }
                block_mma<NG>(acc, w.a[u], w.b[u], xl, xh);
                if constexpr (SWIGLU) block_mma<NG>(accu, w.ua[u], w.ub[u], xl, xh);
            }
        }
        if (++c_ci < items_per_rb) return;
        // the row block is complete: add the warps' partial sums (integers: any order) and write it out
        const int n0 = c_rb * 16;
#pragma unroll
        for (int j = 0; j < NG; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                red[warp][j * 4 + c][lane] = acc[j][c];
                if (SWIGLU) red[warp][NG * 4 + j * 4 + c][lane] = accu[j][c];
            }
        clear_acc();
        __syncthreads();
        // accumulator word c of lane (g, t), group j = row g + 8 * (c / 2), token 8 j + 2 t + (c % 2)
        for (int q = threadIdx.x; q < NG * 4 * 32; q += MMA_WARPS * 32) {
            const int idx = q >> 5, ln = q & 31;
            const int j = idx >> 2, c = idx & 3;
            const int n = n0 + (ln >> 2) + ((c & 2) ? 8 : 0);
            const int m = 8 * j + 2 * (ln & 3) + (c & 1);
            int raw = 0, raw_u = 0;
#pragma unroll
            for (int w8 = 0; w8 < MMA_WARPS; ++w8) {
                raw += red[w8][idx][ln];
                if (SWIGLU) raw_u += red[w8][NG * 4 + idx][ln];
            }
            if (n < a.N && m < a.M) {
                const int bs = FUSEQ ? q_bias : a.bias_sum[m];
                const float sx = FUSEQ ? q_scale : a.act_scales[m];
                const int tq = finish_acc(raw, bs);
                float y = dequant(tq, sx, __half2float(a.w_scales[n]));
                if (SWIGLU) y = swiglu(y, dequant(finish_acc(raw_u, bs), sx, __half2float(a.w_up_scales[n])));
                store_out(a.out, static_cast<int64_t>(m) * a.ldo + n, a.out_dtype, y, tq);
            }
        }
        __syncthreads();   // red is free again
        c_ci = 0;
        c_rb += gridDim.x;
    };

    ItemWeights<KU, SWIGLU> w0, w1;
    if (total_items > 0) load_item(w0);
    pdl_launch_dependents();
    pdl_wait();   // the activations come from the kernel before this one; the weights above do not
    if (FUSEQ) {
        // the quantizer of quantize.cu for one row (two passes over it, the second from cache): max-abs,
        // scale = amax / 7, inv = 7 / amax, codes by the magic add; half = 64 here (K % 128 == 0)
        const int tid = threadIdx.x, n8 = a.K / 8;
        const int64_t src = a.fuse_row_index ? static_cast<int64_t>(a.fuse_row_index[0]) : 0;
        const uint4* xr = reinterpret_cast<const uint4*>(a.fuse_x + src * a.fuse_ldx);
        float amax = 0.0f;
        for (int c = tid; c < n8; c += MMA_WARPS * 32) {
            const uint4 v = __ldg(xr + c);
            const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 f = __half22float2(__habs2(h[q]));
                amax = fmaxf(amax, fmaxf(f.x, f.y));
            }
        }
        amax = warp_max(amax);
        if (lane == 0) q_red_f[warp] = amax;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < MMA_WARPS; ++w) amax = fmaxf(amax, q_red_f[w]);
        float scale, inv;
        scale_of(amax, scale, inv);
        int bias = 0;
        for (int c = tid; c < n8; c += MMA_WARPS * 32) {
            const uint4 v = __ldg(xr + c);
            uint64_t p[4];
            uint32_t tt[8];
            half8_to_pairs(v, p);
#pragma unroll
            for (int q = 0; q < 4; ++q) round_pair(p[q], inv, MAGIC, tt[2 * q], tt[2 * q + 1]);
            uint32_t w0 = low_bytes(tt[0], tt[1], tt[2], tt[3]), w1 = low_bytes(tt[4], tt[5], tt[6], tt[7]);
            if (((8 * c) & 127) < 64) {   // these codes meet low weight nibbles
                bias = __dp4a(static_cast<int>(w0), 0x01010101, bias);
                bias = __dp4a(static_cast<int>(w1), 0x01010101, bias);
                w0 = times16(w0);
                w1 = times16(w1);
            }
            reinterpret_cast<uint2*>(xs)[c] = make_uint2(w0, w1);
            if (blockIdx.x == 0) reinterpret_cast<uint2*>(const_cast<int8_t*>(a.x8))[c] = make_uint2(w0, w1);
        }
        bias = warp_sum(bias);
        if (lane == 0) q_red_i[warp] = bias;
        __syncthreads();   // also: xs is complete
        if (tid == 0) {
            int total = 0;
#pragma unroll
            for (int w = 0; w < MMA_WARPS; ++w) total += q_red_i[w];
            q_bias = total;
            q_scale = scale;
            if (blockIdx.x == 0) {
                const_cast<int32_t*>(a.bias_sum)[0] = total;
                const_cast<float*>(a.act_scales)[0] = scale;
            }
        }
        // q_bias / q_scale are read only after the __syncthreads of a row block's reduction
    }
    for (int i = 0; i < total_items; i += 2) {
        if (i + 1 < total_items) load_item(w1);
        compute_item(w0);
        if (i + 1 >= total_items) break;
        if (i + 2 < total_items) load_item(w0);
        compute_item(w1);
    }
}

template <int NG>
void launch_ng(const LinearArgs& a, cudaStream_t s) {
    const int resident = 2 * sm_count();    // CTAs that fit the device at two per SM
    const int n_rb = (a.N + 15) / 16;
    const int grid = n_rb < resident ? n_rb : resident;
    cudaError_t e;
    if (NG == 1 && a.fuse_x) {
        const size_t smem = static_cast<size_t>(a.K);   // <= MMA_FUSE_MAX_K: within the default dynamic limit
        if (a.w_up) e = launch_dependent(w4a4_mma_kernel<1, true, true>, dim3(grid), dim3(MMA_WARPS * 32), smem, s, a);
        else e = launch_dependent(w4a4_mma_kernel<1, false, true>, dim3(grid), dim3(MMA_WARPS * 32), smem, s, a);
    } else if (a.w_up) e = launch_dependent(w4a4_mma_kernel<NG, true>, dim3(grid), dim3(MMA_WARPS * 32), 0, s, a);
    else e = launch_dependent(w4a4_mma_kernel<NG, false>, dim3(grid), dim3(MMA_WARPS * 32), 0, s, a);
    if (e != cudaSuccess) note_cuda_error(e);
}

}  // namespace mmas
using namespace mmas;

bool mma_stream_supports(const LinearArgs& a) {
    return a.half == 64 && a.K % 128 == 0 && a.K >= 128 && a.M >= 1 && a.M <= MMA_STREAM_MAX_M;
}

sqap_status launch_linear_mma_stream(const LinearArgs& a, cudaStream_t s) {
    if (!mma_stream_supports(a)) return SQAP_ERR_UNSUPPORTED;
    if (a.M <= 8) launch_ng<1>(a, s);
    else if (a.M <= 16) launch_ng<2>(a, s);
    else if (a.M <= 24) launch_ng<3>(a, s);
    else launch_ng<4>(a, s);
    count_launch();
    return check_launch();
}

}  // namespace sqap

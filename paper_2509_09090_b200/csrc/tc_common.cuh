// Pieces shared by the tcgen05 kernels of the W4A4 linear: PTX wrappers, the epilogue of one accumulator
// tile, tensor-map creation.
#pragma once

#include <cuda.h>

#include <cstring>

#include "linear.cuh"

namespace sqap {
namespace tc {

constexpr long long WAIT_LIMIT_CLOCKS = 4000000000LL;  // ~2 s

struct Args {
    const int32_t* bias_sum;
    const float* act_scales;
    const __half* w_scales;
    const __half* w_up_scales;
    void* out;
    int64_t ldo;
    int M, N, K;
    int BN;        // tokens per tile
    int m_tiles, n_tiles;
    int out_dtype;
    int swiglu;    // 1: tile rows 2i / 2i+1 hold gate / up of output channel n0/2 + i
    int stages;    // depth of the TMA ring (kernels that size it at run time)
    int a_tiles;   // depth of the ring of unpacked weight tiles in tensor memory (the same)
    int* status;
};

// ------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Non-blocking probe of the same condition.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within `limit` clocks or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          long long limit = WAIT_LIMIT_CLOCKS) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3FFu) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit) return false;
        }
    }
    return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
// The same two, issued by the lane(s) with issue != 0 of a converged warp (see tc_commit_if).
__device__ __forceinline__ void mbar_expect_tx_if(uint32_t bar, uint32_t bytes, uint32_t issue) {
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.b32 q, %2, 0;\n\t"
        "@q mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t}"
        ::"r"(bar), "r"(bytes), "r"(issue)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d_if(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar, uint32_t issue) {
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n\t}"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar), "r"(issue)
        : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 1 in exactly one (elected) lane of a converged warp, 0 in the others.
__device__ __forceinline__ uint32_t elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred;
}
// tcgen05.commit issued by the lane(s) with issue != 0; the warp stays converged around it, so that the operands
// of the tensor-core instructions can stay in uniform registers (a branch on the lane id costs a transfer from
// the vector to the uniform register file per operand and instruction: some 60 cycles per MMA).
__device__ __forceinline__ void tc_commit_if(uint32_t bar, uint32_t issue) {
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(bar), "r"(issue)
        : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major, 128-byte-swizzled operand tile: rows 128 B apart, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    return static_cast<uint64_t>((addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ float silu_mul_fast(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

// Part of one finished accumulator tile -> global memory. The thread owns one TMEM lane (output channel n;
// with SwiGLU the even lane of a pair holds the gate and the odd lane the up projection of channel n) and
// walks the tokens [c_begin, c_end) of the tile 16 at a time; the per-token bias sums and scales of a chunk
// are fetched by lanes 0-15 with one coalesced load each (one chunk ahead) and broadcast by shuffle.
template <int OUT, bool SWIGLU, int XCHG = 1>
__device__ __forceinline__ void epilogue_tile(const Args& a, uint32_t taddr, int m0, int c_begin, int c_end, int n,
                                              bool n_ok, float sw, int lane) {
    constexpr int ESZ = OUT == SQAP_I32 ? 4 : 2;
    const int ml = lane & 15;
    const bool odd = (lane & XCHG) != 0;   // SwiGLU: this lane holds the up projection, its partner (lane ^ XCHG) the gate
    const int64_t row_bytes = a.ldo * ESZ;
    int mm = m0 + c_begin + ml;
    int bs_next = mm < a.M ? (__ldg(a.bias_sum + mm) << 7) : 0;
    float sx_next = mm < a.M ? __ldg(a.act_scales + mm) : 0.0f;
    for (int c = c_begin; c < c_end; c += 16) {
        uint32_t v[16];
        tc_ld16(taddr + c, v);
        const int bs_cur = bs_next;
        const float sx_cur = sx_next;
        mm = m0 + c + 16 + ml;
        if (c + 16 < c_end) {
            bs_next = mm < a.M ? (__ldg(a.bias_sum + mm) << 7) : 0;
            sx_next = mm < a.M ? __ldg(a.act_scales + mm) : 0.0f;
        }
        tc_wait_ld();
        const int valid = a.M - (m0 + c);  // tokens of this chunk that exist
        uint8_t* optr = static_cast<uint8_t*>(a.out) + static_cast<int64_t>(m0 + c) * row_bytes + static_cast<int64_t>(n) * ESZ;
        if (SWIGLU) {
            // Columns are handled in pairs: the even lane finishes column j (needs the up value of its
            // partner), the odd lane column j+1 (needs the gate value of its partner): one exchange per pair.
#pragma unroll
            for (int j = 0; j < 16; j += 2) {
                const float y0 = __fmul_rn(__fmul_rn(static_cast<float>((static_cast<int>(v[j]) - __shfl_sync(0xffffffffu, bs_cur, j)) >> 4),
                                                     __shfl_sync(0xffffffffu, sx_cur, j)), sw);
                const float y1 = __fmul_rn(__fmul_rn(static_cast<float>((static_cast<int>(v[j + 1]) - __shfl_sync(0xffffffffu, bs_cur, j + 1)) >> 4),
                                                     __shfl_sync(0xffffffffu, sx_cur, j + 1)), sw);
                const float got = __shfl_xor_sync(0xffffffffu, odd ? y0 : y1, XCHG);
                const float h = odd ? silu_mul_fast(got, y1) : silu_mul_fast(y0, got);
                const int jj = odd ? j + 1 : j;
                if (n_ok && jj < valid) {
                    uint8_t* o = optr + jj * row_bytes;
                    if (OUT == SQAP_FP16) *reinterpret_cast<__half*>(o) = __float2half_rn(h);
                    else *reinterpret_cast<__nv_bfloat16*>(o) = __float2bfloat16_rn(h);
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int bs = __shfl_sync(0xffffffffu, bs_cur, j);
                const float sx = __shfl_sync(0xffffffffu, sx_cur, j);
                const int t = (static_cast<int>(v[j]) - bs) >> 4;
                const float y = __fmul_rn(__fmul_rn(static_cast<float>(t), sx), sw);
                if (n_ok && j < valid) {
                    if (OUT == SQAP_FP16) *reinterpret_cast<__half*>(optr) = __float2half_rn(y);
                    else if (OUT == SQAP_BF16) *reinterpret_cast<__nv_bfloat16*>(optr) = __float2bfloat16_rn(y);
                    else *reinterpret_cast<int32_t*>(optr) = t;
                }
                optr += row_bytes;
            }
        }
    }
}

// Barrier among `nthreads` threads (named barrier `id`) that also ORs a predicate over them: every thread gets
// true if any thread passed true.
__device__ __forceinline__ bool bar_or(int id, int nthreads, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %3, 0;\n\t"
        "bar.red.or.pred p, %1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(nthreads), "r"(static_cast<uint32_t>(pred))
        : "memory");
    return r != 0;
}

// One 16-token chunk of an accumulator tile, raw sums in registers -> global memory. The thread owns one output
// channel n (one tensor-memory lane; with SwiGLU the gate and up projections of a channel sit in lanes XCHG apart)
// and 16 consecutive tokens, the first of which is token `m_first` of the matrix. t4 points at the staged
// per-token constants of those tokens: {128 * bias_sum, bits of the activation scale} per token ({0, 0} past M),
// two tokens per 16-byte shared-memory load (a broadcast: every lane of a warp needs the same pair).
template <int OUT, bool SWIGLU, int XCHG>
__device__ __forceinline__ void epilogue_chunk(const Args& a, const uint32_t* v, int m_first, int n, bool n_ok, float sw,
                                               int lane, const int4* t4) {
    constexpr int ESZ = OUT == SQAP_I32 ? 4 : 2;
    const bool odd = (lane & XCHG) != 0;   // SwiGLU: this lane holds the up projection, its partner (lane ^ XCHG) the gate
    const int64_t row_bytes = a.ldo * ESZ;
    const int valid = a.M - m_first;  // tokens of this chunk that exist
    uint8_t* optr = static_cast<uint8_t*>(a.out) + static_cast<int64_t>(m_first) * row_bytes + static_cast<int64_t>(n) * ESZ;
#pragma unroll
    for (int j = 0; j < 16; j += 2) {
        const int4 t = t4[j >> 1];
        const int t0 = (static_cast<int>(v[j]) - t.x) >> 4, t1 = (static_cast<int>(v[j + 1]) - t.z) >> 4;
        const float y0 = __fmul_rn(__fmul_rn(static_cast<float>(t0), __int_as_float(t.y)), sw);
        const float y1 = __fmul_rn(__fmul_rn(static_cast<float>(t1), __int_as_float(t.w)), sw);
        if (SWIGLU) {
            // the gate lane finishes token j (needs the up value of its partner), the up lane token j+1
            const float got = __shfl_xor_sync(0xffffffffu, odd ? y0 : y1, XCHG);
            const float h = odd ? silu_mul_fast(got, y1) : silu_mul_fast(y0, got);
            const int jj = odd ? j + 1 : j;
            if (n_ok && jj < valid) {
                uint8_t* o = optr + jj * row_bytes;
                if (OUT == SQAP_FP16) *reinterpret_cast<__half*>(o) = __float2half_rn(h);
                else *reinterpret_cast<__nv_bfloat16*>(o) = __float2bfloat16_rn(h);
            }
        } else {
            if (n_ok && j < valid) {
                uint8_t* o = optr + j * row_bytes;
                if (OUT == SQAP_FP16) *reinterpret_cast<__half*>(o) = __float2half_rn(y0);
                else if (OUT == SQAP_BF16) *reinterpret_cast<__nv_bfloat16*>(o) = __float2bfloat16_rn(y0);
                else *reinterpret_cast<int32_t*>(o) = t0;
            }
            if (n_ok && j + 1 < valid) {
                uint8_t* o = optr + (j + 1) * row_bytes;
                if (OUT == SQAP_FP16) *reinterpret_cast<__half*>(o) = __float2half_rn(y1);
                else if (OUT == SQAP_BF16) *reinterpret_cast<__nv_bfloat16*>(o) = __float2bfloat16_rn(y1);
                else *reinterpret_cast<int32_t*>(o) = t1;
            }
        }
    }
}

// Part of one finished accumulator tile -> global memory, with the per-token constants staged in shared memory:
// tok[c] = {128 * bias_sum, bits of the activation scale} of token m0 + c ({0, 0} past M). One broadcast
// shared-memory load per two tokens; fetching them by warp shuffles instead (the routine above) was measured to
// slow the main loop, because shuffles share a pipe with the unpack warps' shared-memory loads.
template <int OUT, bool SWIGLU, int XCHG>
__device__ __forceinline__ void epilogue_tile_staged(const Args& a, uint32_t taddr, int m0, int c_begin, int c_end, int n,
                                                     bool n_ok, float sw, int lane, const int2* tok) {
    for (int c = c_begin; c < c_end; c += 16) {
        uint32_t v[16];
        tc_ld16(taddr + c, v);
        const int4* t4 = reinterpret_cast<const int4*>(tok + c);   // two tokens per 16-byte load
        tc_wait_ld();
        epilogue_chunk<OUT, SWIGLU, XCHG>(a, v, m0 + c, n, n_ok, sw, lane, t4);
    }
}

// ---- epilogue with coalesced global stores (fp16 / bf16 outputs)
// In tensor memory a thread owns one output channel and a row of tokens, while in the output matrix the channels of
// one token are contiguous: stored straight from registers, a warp writes 64 bytes per instruction (32 channels x
// 2 bytes of one token), and those narrow stores were measured to take about 100 cycles each per warp. Here the 128
// threads that share a half of the tile's tokens (one warp per lane quadrant) first put each 16-token chunk into
// shared memory as [token][channel], meet at a named barrier, and copy it out 16 bytes per thread, 512 contiguous
// bytes per warp instruction. Two buffers per half take turns, so one barrier per chunk is enough: a thread can
// only be two chunks ahead of the slowest after passing the barrier in between, which every thread reaches after
// its own copy-out of the chunk before.
constexpr int EPI_STAGE_BYTES = 16 * 128 * 2;                // one chunk: 16 tokens x up to 128 channels x 2 bytes
constexpr int EPI_STAGE_TOTAL = 2 * 2 * EPI_STAGE_BYTES;     // two halves x two buffers

__device__ __forceinline__ void bar_sync_named(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

template <int OUT>
__device__ __forceinline__ uint16_t bits16(float y) {
    static_assert(OUT == SQAP_FP16 || OUT == SQAP_BF16, "16-bit outputs only");
    return OUT == SQAP_FP16 ? __half_as_ushort(__float2half_rn(y)) : __bfloat16_as_ushort(__float2bfloat16_rn(y));
}

// Four consecutive tokens of this thread's channel: raw sums v0..v3 -> 16-bit outputs in the staging buffer.
// tq: the four tokens' constants (two int4, see epilogue_chunk); mine: the buffer position of the first of the four
// tokens for this thread's channel; ROWB apart per token. SwiGLU: gate and up of a channel sit 16 lanes apart; the
// gate lane finishes tokens 0 and 2 (it needs the up value of its partner), the up lane tokens 1 and 3.
template <int OUT, bool SWIGLU>
__device__ __forceinline__ void epilogue_quad_to_stage(uint32_t v0, uint32_t v1, uint32_t v2, uint32_t v3, const int4* tq,
                                                       float sw, bool odd, uint8_t* mine) {
    constexpr int ROWB = SWIGLU ? 128 : 256;
    const int4 ta = tq[0], tb = tq[1];
    const float y0 = __fmul_rn(__fmul_rn(static_cast<float>((static_cast<int>(v0) - ta.x) >> 4), __int_as_float(ta.y)), sw);
    const float y1 = __fmul_rn(__fmul_rn(static_cast<float>((static_cast<int>(v1) - ta.z) >> 4), __int_as_float(ta.w)), sw);
    const float y2 = __fmul_rn(__fmul_rn(static_cast<float>((static_cast<int>(v2) - tb.x) >> 4), __int_as_float(tb.y)), sw);
    const float y3 = __fmul_rn(__fmul_rn(static_cast<float>((static_cast<int>(v3) - tb.z) >> 4), __int_as_float(tb.w)), sw);
    if (SWIGLU) {
        const float g0 = __shfl_xor_sync(0xffffffffu, odd ? y0 : y1, 16);
        const float g1 = __shfl_xor_sync(0xffffffffu, odd ? y2 : y3, 16);
        const float h0 = odd ? silu_mul_fast(g0, y1) : silu_mul_fast(y0, g0);
        const float h1 = odd ? silu_mul_fast(g1, y3) : silu_mul_fast(y2, g1);
        *reinterpret_cast<uint16_t*>(mine + (odd ? 1 : 0) * ROWB) = bits16<OUT>(h0);
        *reinterpret_cast<uint16_t*>(mine + (odd ? 3 : 2) * ROWB) = bits16<OUT>(h1);
    } else {
        *reinterpret_cast<uint16_t*>(mine) = bits16<OUT>(y0);
        *reinterpret_cast<uint16_t*>(mine + ROWB) = bits16<OUT>(y1);
        *reinterpret_cast<uint16_t*>(mine + 2 * ROWB) = bits16<OUT>(y2);
        *reinterpret_cast<uint16_t*>(mine + 3 * ROWB) = bits16<OUT>(y3);
    }
}

// A staged chunk ([16 tokens][64 or 128 channels] of 16-bit outputs) -> global memory, 16 bytes per thread.
template <bool SWIGLU>
__device__ __forceinline__ void epilogue_stage_copy_out(const Args& a, int m_first, int n_tile0, const uint8_t* stage,
                                                        int tid_half) {
    constexpr int ROWB = SWIGLU ? 128 : 256;
    constexpr int PPR = ROWB / 16;             // 16-byte pieces (8 channels) per token
#pragma unroll
    for (int p = tid_half; p < 16 * PPR; p += 128) {
        const int token = p / PPR, piece = p % PPR;
        const int m = m_first + token, n = n_tile0 + piece * 8;
        if (m < a.M && n < a.N) {
            const uint8_t* src = stage + token * ROWB + piece * 16;
            uint8_t* dst = static_cast<uint8_t*>(a.out) + (static_cast<int64_t>(m) * a.ldo + n) * 2;
            if (n + 8 <= a.N) {
                *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
            } else {
                for (int e = 0; e < a.N - n; ++e)
                    reinterpret_cast<uint16_t*>(dst)[e] = reinterpret_cast<const uint16_t*>(src)[e];
            }
        }
    }
}

// v: the raw sums of this thread's channel for 16 consecutive tokens starting at token m_first of the matrix.
// ch: the thread's channel within the tile (plain: 0..127 = tensor-memory lane; SwiGLU: 0..63, gate and up of a
// channel sit 16 lanes apart); n_tile0: first output channel of the tile; sw: this lane's weight scale.
// stage: the buffer for this chunk; tid_half: 0..127 among the threads sharing it; bar_id: their named barrier.
template <int OUT, bool SWIGLU>
__device__ __forceinline__ void epilogue_chunk_coalesced(const Args& a, const uint32_t* v, int m_first, int n_tile0, int ch,
                                                         float sw, int lane, const int4* t4, uint8_t* stage, int tid_half,
                                                         int bar_id) {
    constexpr int ROWB = SWIGLU ? 128 : 256;   // bytes of one token's channels in the buffer
    const bool odd = (lane & 16) != 0;         // SwiGLU: this lane holds the up projection, lane ^ 16 the gate
    uint8_t* mine = stage + ch * 2;
#pragma unroll
    for (int q = 0; q < 4; ++q)
        epilogue_quad_to_stage<OUT, SWIGLU>(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3], t4 + 2 * q, sw, odd,
                                            mine + 4 * q * ROWB);
    bar_sync_named(bar_id, 128);
    epilogue_stage_copy_out<SWIGLU>(a, m_first, n_tile0, stage, tid_half);
}

// Tokens [c_begin, c_end) of a finished accumulator tile through the routine above. stage_half: this half's two
// buffers (2 * EPI_STAGE_BYTES); tok as in epilogue_tile_staged.
template <int OUT, bool SWIGLU>
__device__ __forceinline__ void epilogue_tile_coalesced(const Args& a, uint32_t taddr, int m0, int c_begin, int c_end,
                                                        int n_tile0, int ch, float sw, int lane, const int2* tok,
                                                        uint8_t* stage_half, int tid_half, int bar_id) {
    int flip = 0;
    for (int c = c_begin; c < c_end; c += 16, flip ^= 1) {
        uint32_t v[16];
        tc_ld16(taddr + c, v);
        const int4* t4 = reinterpret_cast<const int4*>(tok + c);   // two tokens per 16-byte load
        tc_wait_ld();
        epilogue_chunk_coalesced<OUT, SWIGLU>(a, v, m0 + c, n_tile0, ch, sw, lane, t4, stage_half + flip * EPI_STAGE_BYTES,
                                              tid_half, bar_id);
    }
}

// ------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    // the driver entry point is the same for every device; the function-local static is initialised once,
    // thread-safely
    static const EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(p);
        cudaGetLastError();
        return static_cast<EncodeTiledFn>(nullptr);
    }();
    return fn;
}

// 2-D uint8 tensor [rows][row_bytes], box [box_rows][box_bytes].
inline bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t row_bytes, uint32_t box_rows,
                     uint32_t box_bytes, CUtensorMapSwizzle swz) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {row_bytes, rows};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {box_bytes, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The two weight tensor maps of a launch (w and, for a gate / up pair, w_up; else w twice): taken from the handles
// where they were encoded at pack time, encoded here otherwise. BKB = bytes of K per box row (128).
inline bool weight_maps(const LinearArgs& a, bool swiglu, uint32_t rows_per_tile, uint32_t bkb, CUtensorMap* tm_w, CUtensorMap* tm_u) {
    const uint32_t box_rows = swiglu ? rows_per_tile / 2 : rows_per_tile;
    auto from_handle = [&](const Weights* h, CUtensorMap* out) {
        if (!h || !h->has_maps || bkb != 128 || (box_rows != 128 && box_rows != 64)) return false;
        memcpy(out, box_rows == 128 ? h->map_rows128 : h->map_rows64, sizeof(CUtensorMap));
        return true;
    };
    if (!from_handle(a.w_handle, tm_w) && !make_map(tm_w, a.w, a.N, a.K / 2, box_rows, bkb, CU_TENSOR_MAP_SWIZZLE_128B)) return false;
    if (!swiglu) {
        *tm_u = *tm_w;
        return true;
    }
    return from_handle(a.w_up_handle, tm_u) || make_map(tm_u, a.w_up, a.N, a.K / 2, box_rows, bkb, CU_TENSOR_MAP_SWIZZLE_128B);
}

// Encodes a handle's maps (weights.cu, at pack time).
inline void encode_handle_maps(Weights* w) {
    w->has_maps = 0;
    if (w->half != 64) return;   // K % 128 != 0: the tensor-core kernels do not run the shape
    static_assert(sizeof(CUtensorMap) == 128, "tensor map storage in the handle");
    CUtensorMap a, b;
    if (!make_map(&a, w->packed, w->N, w->K / 2, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B)) return;
    if (!make_map(&b, w->packed, w->N, w->K / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B)) return;
    memcpy(w->map_rows128, &a, 128);
    memcpy(w->map_rows64, &b, 128);
    w->has_maps = 1;
}

// Splits M tokens into m_tiles tiles of BN tokens (multiple of 16, <= bn_max) for a persistent kernel whose
// `units` workers (CTAs or CTA pairs) each take whole tiles: the split that minimises waves x time per tile, so
// that e.g. 224 tiles on 74 workers (4 waves, the last almost empty) become 288 narrower tiles (4 full waves).
// Time per 256-code stage of a tile, in cycles: the MMAs take 4 per token, the stage's TMA traffic (16 KB of
// packed weights + x_bytes_per_token per token: 256, or 128 where a CTA pair shares the token tile) moves at
// about 58 bytes per cycle, and each tile costs about 96 more per stage for its fill and hand-over.
inline void choose_token_tiles(int M, int n_tiles, int units, int bn_max, int x_bytes_per_token, int* m_tiles, int* BN) {
    const int mt_min = (M + bn_max - 1) / bn_max;
    *m_tiles = mt_min;
    *BN = ((M + mt_min - 1) / mt_min + 15) / 16 * 16;
    double best_cost = -1.0;
    for (int mt = mt_min; mt <= mt_min + 12 && mt <= (M + 15) / 16; ++mt) {
        const int per = (M + mt - 1) / mt;
        const int bn = (per + 15) / 16 * 16;
        if (bn > bn_max) continue;
        const long tiles = static_cast<long>(mt) * n_tiles;
        const long waves = (tiles + units - 1) / units;
        const double mma = 4.0 * bn, fetch = (16384.0 + static_cast<double>(x_bytes_per_token) * bn) / 58.0;
        const double cost = static_cast<double>(waves) * ((mma > fetch ? mma : fetch) + 96.0);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            *m_tiles = mt;
            *BN = bn;
        }
    }
}

inline bool device_is_sm100() {
    const DeviceProps* p = device_props();
    return p && p->cc_major == 10;
}

}  // namespace tc
}  // namespace sqap

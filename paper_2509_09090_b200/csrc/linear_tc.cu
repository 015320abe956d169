// tcgen05 tensor-core kernel of the W4A4 linear for sm_100a.
//
// D[n][m] = sum_k W[n][k] * X[m][k] with the WEIGHTS as the 128-row MMA-M operand and the tokens as
// the MMA-N operand (up to 256 per tile), int8 x int8 -> int32 in tensor memory (kind::i8).
//
// Per CTA (persistent, one per SM), warp roles:
//   warp 0      TMA producer: per K-step of 128 codes, one box of packed weights (128 rows x 64 B,
//               4-bit) and one box of expanded int8 activations (BN rows x 128 B, 128B-swizzled)
//   warps 2-5   unpack: packed nibbles -> two int8 vectors by masking alone (see common.cuh), written
//               in the 128B-swizzled K-major layout the MMA reads; 2 logic ops per 8 weights
//   warp 1      MMA issuer: 4 x tcgen05.mma (K = 32 each) per K-step into one of two TMEM accumulators
//   warps 6-13  epilogue: tcgen05.ld the finished accumulator, remove the nibble bias, apply both
//               scales (or SwiGLU), store; overlaps the next tile's main loop
// Every wait on an mbarrier is bounded; on expiry the kernel records SQAP_ERR_TIMEOUT in the device
// status word, drains and frees its tensor memory, and returns.
#include "tc_common.cuh"

namespace sqap {
namespace tc {

constexpr int BM = 128;             // weight rows per tile (MMA M)
constexpr int BK = 128;             // codes of K per pipeline stage
constexpr int BN_MAX = 256;         // tokens per tile (MMA N), runtime BN <= BN_MAX, multiple of 16
constexpr int STAGES = 4;
constexpr int X_BYTES = BN_MAX * BK;      // 32 KB, int8
constexpr int WU_BYTES = BM * BK;         // 16 KB, unpacked int8
constexpr int WP_BYTES = BM * BK / 2;     // 8 KB, packed
constexpr int OFF_X = 0;
constexpr int OFF_WU = OFF_X + STAGES * X_BYTES;
constexpr int OFF_WP = OFF_WU + STAGES * WU_BYTES;
constexpr int OFF_BAR = OFF_WP + STAGES * WP_BYTES;
constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;  // barriers + slack for 1024-byte alignment
constexpr int EPI_WARPS = 8;                 // two per TMEM lane quadrant, each takes half of the tile's tokens
constexpr int THREADS = 32 * (6 + EPI_WARPS);
// ------------------------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(THREADS, 1)
w4a4_tc_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_w_up,
               const __grid_constant__ CUtensorMap tm_x, Args a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar0 = base + OFF_BAR;
    // barrier slots (8 bytes each)
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto ufull = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto empty = [&](int s) { return bar0 + 8u * (2 * STAGES + s); };
    auto acc_full = [&](int b) { return bar0 + 8u * (3 * STAGES + b); };
    auto acc_empty = [&](int b) { return bar0 + 8u * (3 * STAGES + 2 + b); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + OFF_BAR + 8 * (3 * STAGES + 4));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + OFF_BAR + 8 * (3 * STAGES + 4) + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_steps = a.K / BK;
    const int total_tiles = a.m_tiles * a.n_tiles;
    const uint32_t stage_tx = static_cast<uint32_t>(WP_BYTES + a.BN * BK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full(s), 1);
            mbar_init(ufull(s), 128);
            mbar_init(empty(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full(b), 1);
            mbar_init(acc_empty(b), 32 * EPI_WARPS);
        }
        abort_flag[0] = 0;
        abort_flag[1] = 0;  // always-zero word for waits that must ignore the abort request
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool failed = false;

    if (warp == 0) {
        // ---------------- TMA producer (one lane)
        if (lane == 0) {
            uint32_t it = 0;
            for (int tile = blockIdx.x; tile < total_tiles && !failed; tile += gridDim.x) {
                const int n0 = (tile % a.n_tiles) * BM, m0 = (tile / a.n_tiles) * a.BN;
                for (int ks = 0; ks < k_steps; ++ks, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(empty(s), ph ^ 1u, abort_flag)) { failed = true; break; }
                    mbar_expect_tx(full(s), stage_tx);
                    if (a.swiglu) {
                        tma_load_2d(base + OFF_WP + s * WP_BYTES, &tm_w, ks * (BK / 2), n0 / 2, full(s));
                        tma_load_2d(base + OFF_WP + s * WP_BYTES + WP_BYTES / 2, &tm_w_up, ks * (BK / 2), n0 / 2, full(s));
                    } else {
                        tma_load_2d(base + OFF_WP + s * WP_BYTES, &tm_w, ks * (BK / 2), n0, full(s));
                    }
                    tma_load_2d(base + OFF_X + s * X_BYTES, &tm_x, ks * BK, m0, full(s));
                }
            }
            if (failed) {
                // drain: give every armed stage a bounded chance to land before shared memory is released
                for (int s = 0; s < STAGES; ++s) {
                    const uint32_t last = it > static_cast<uint32_t>(s) ? (it - 1 - s) : 0xFFFFFFFFu;
                    if (last != 0xFFFFFFFFu) mbar_wait(full(last % STAGES), (last / STAGES) & 1u, abort_flag + 1);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (one lane)
        if (lane == 0) {
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a.BN >> 3) << 17) |
                                   (static_cast<uint32_t>(BM >> 4) << 24);
            uint32_t it = 0, lt = 0;
            for (int tile = blockIdx.x; tile < total_tiles && !failed; tile += gridDim.x, ++lt) {
                const int b = lt & 1;
                if (!mbar_wait(acc_empty(b), ((lt >> 1) & 1u) ^ 1u, abort_flag)) { failed = true; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(b * BN_MAX);
                for (int ks = 0; ks < k_steps; ++ks, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(full(s), ph, abort_flag) || !mbar_wait(ufull(s), ph, abort_flag)) { failed = true; break; }
                    tc_fence_after();
                    const uint64_t adesc = smem_desc_sw128(base + OFF_WU + s * WU_BYTES);
                    const uint64_t bdesc = smem_desc_sw128(base + OFF_X + s * X_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k)
                        tc_mma_i8(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (ks | k) != 0 ? 1u : 0u);
                    tc_commit(empty(s));
                }
                if (failed) break;
                tc_commit(acc_full(b));
            }
        }
    } else if (warp < 6) {
        // ---------------- unpack warps: thread = one weight row of the tile
        const int r = threadIdx.x - 64;
        // SwiGLU: packed rows 0-63 are gate rows, 64-127 up rows; interleave them so that a lane pair
        // of the accumulator holds (gate, up) of one output channel.
        const int dr = a.swiglu ? ((r & 63) * 2 + (r >> 6)) : r;
        uint32_t it = 0;
        for (int tile = blockIdx.x; tile < total_tiles && !failed; tile += gridDim.x) {
            for (int ks = 0; ks < k_steps; ++ks, ++it) {
                const int s = it % STAGES;
                if (!__all_sync(0xffffffffu, mbar_wait(full(s), (it / STAGES) & 1u, abort_flag))) { failed = true; break; }
                const uint8_t* src = sm + OFF_WP + s * WP_BYTES + r * 64;
                uint8_t* dst = sm + OFF_WU + s * WU_BYTES + dr * 128;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int c = ((r >> 1) + j) & 3;  // order that keeps both the read and the write conflict-free
                    const uint4 v = *reinterpret_cast<const uint4*>(src + c * 16);
                    uint4 lo, hi;
                    lo.x = v.x & 0x0F0F0F0Fu; lo.y = v.y & 0x0F0F0F0Fu; lo.z = v.z & 0x0F0F0F0Fu; lo.w = v.w & 0x0F0F0F0Fu;
                    hi.x = v.x & 0xF0F0F0F0u; hi.y = v.y & 0xF0F0F0F0u; hi.z = v.z & 0xF0F0F0F0u; hi.w = v.w & 0xF0F0F0F0u;
                    *reinterpret_cast<uint4*>(dst + ((c ^ (dr & 7)) << 4)) = lo;        // codes k = 16c .. 16c+15
                    *reinterpret_cast<uint4*>(dst + (((c + 4) ^ (dr & 7)) << 4)) = hi;  // codes k = 64+16c ..
                }
                fence_proxy_async();
                mbar_arrive(ufull(s));
            }
        }
    } else {
        // ---------------- epilogue warps: warp % 4 selects the 32-lane quadrant of tensor memory
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const int split = ((a.BN / 16 + 1) / 2) * 16;  // first token of the second half of the tile
        const int c_begin = (warp - 6) < 4 ? 0 : (EPI_WARPS == 8 ? split : 0);
        const int c_end = (EPI_WARPS == 8 && (warp - 6) < 4) ? split : a.BN;
        uint32_t lt = 0;
        for (int tile = blockIdx.x; tile < total_tiles && !failed; tile += gridDim.x, ++lt) {
            const int b = lt & 1;
            const int n0 = (tile % a.n_tiles) * BM, m0 = (tile / a.n_tiles) * a.BN;
            if (!__all_sync(0xffffffffu, mbar_wait(acc_full(b), (lt >> 1) & 1u, abort_flag))) { failed = true; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(b * BN_MAX);
            int n;
            float sw;
            bool n_ok;
            if (a.swiglu) {
                n = n0 / 2 + (row >> 1);
                n_ok = n < a.N;
                sw = n_ok ? __half2float((row & 1) ? a.w_up_scales[n] : a.w_scales[n]) : 0.0f;
            } else {
                n = n0 + row;
                n_ok = n < a.N;
                sw = n_ok ? __half2float(a.w_scales[n]) : 0.0f;
            }
            if (a.swiglu) {
                if (a.out_dtype == SQAP_FP16) epilogue_tile<SQAP_FP16, true>(a, taddr, m0, c_begin, c_end, n, n_ok, sw, lane);
                else epilogue_tile<SQAP_BF16, true>(a, taddr, m0, c_begin, c_end, n, n_ok, sw, lane);
            } else {
                if (a.out_dtype == SQAP_FP16) epilogue_tile<SQAP_FP16, false>(a, taddr, m0, c_begin, c_end, n, n_ok, sw, lane);
                else if (a.out_dtype == SQAP_BF16) epilogue_tile<SQAP_BF16, false>(a, taddr, m0, c_begin, c_end, n, n_ok, sw, lane);
                else epilogue_tile<SQAP_I32, false>(a, taddr, m0, c_begin, c_end, n, n_ok, sw, lane);
            }
            tc_fence_before();
            mbar_arrive(acc_empty(b));
        }
    }

    if (failed) {
        *abort_flag = 1;
        atomicOr(a.status, SQAP_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

}  // namespace tc

bool tcgen05_supports(const LinearArgs& a) {
    if (a.half != 64 || a.K % tc::BK != 0 || a.K < tc::BK) return false;
    if (a.M < 1) return false;
    if ((a.N * (a.K / 2)) % 16 != 0) return false;
    if (a.w_up && (a.N % 64 != 0)) return false;  // gate/up half-tiles must not straddle the matrix end
    return tc::device_is_sm100() && tc::encode_fn() != nullptr;
}

sqap_status launch_linear_tcgen05(const LinearArgs& a, cudaStream_t s) {
    using namespace tc;
    Args k;
    k.bias_sum = a.bias_sum;
    k.act_scales = a.act_scales;
    k.w_scales = a.w_scales;
    k.w_up_scales = a.w_up_scales;
    k.out = a.out;
    k.ldo = a.ldo;
    k.M = a.M;
    k.N = a.N;
    k.K = a.K;
    k.m_tiles = (a.M + BN_MAX - 1) / BN_MAX;
    const int per = (a.M + k.m_tiles - 1) / k.m_tiles;
    k.BN = (per + 15) / 16 * 16;
    k.swiglu = a.w_up ? 1 : 0;
    k.n_tiles = k.swiglu ? (2 * a.N + BM - 1) / BM : (a.N + BM - 1) / BM;
    k.out_dtype = a.out_dtype;
    k.status = device_status_word();
    if (!k.status) return SQAP_ERR_CUDA;

    CUtensorMap tm_w, tm_u, tm_x;
    const uint32_t w_box_rows = k.swiglu ? BM / 2 : BM;
    if (!make_map(&tm_w, a.w, a.N, a.K / 2, w_box_rows, BK / 2, CU_TENSOR_MAP_SWIZZLE_NONE)) return SQAP_ERR_CUDA;
    if (!make_map(&tm_u, k.swiglu ? a.w_up : a.w, a.N, a.K / 2, w_box_rows, BK / 2, CU_TENSOR_MAP_SWIZZLE_NONE))
        return SQAP_ERR_CUDA;
    if (!make_map(&tm_x, a.x8, a.M, a.K, k.BN, BK, CU_TENSOR_MAP_SWIZZLE_128B)) return SQAP_ERR_CUDA;

    static PerDevice<int> setup;
    const sqap_status st = setup.run([](int*) { return set_max_dynamic_smem(w4a4_tc_kernel, SMEM_BYTES); });
    if (st != SQAP_OK) return st;
    const int tiles = k.m_tiles * k.n_tiles;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    w4a4_tc_kernel<<<grid, THREADS, SMEM_BYTES, s>>>(tm_w, tm_u, tm_x, k);
    count_launch();
    return check_launch();
}

}  // namespace sqap

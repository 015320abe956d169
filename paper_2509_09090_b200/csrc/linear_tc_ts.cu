// tcgen05 kernel of the W4A4 linear with the weight operand in TENSOR MEMORY, for large token counts.
//
// D[n][m] = sum_k W[n][k] * X[m][k], weights as the 128-row MMA-M operand, tokens as the MMA-N operand
// (BN <= 192 per tile), int8 x int8 -> int32 (kind::i8). What bounds the kernel in linear_tc.cu is shared-memory
// bandwidth: besides the tensor core's own operand reads and the TMA writes, its unpack warps read the packed
// weights from shared memory and write them back as int8 for the MMA to read again. Here the unpacked weights
// never touch shared memory: the unpack warps go from the packed TMA tile through registers (two ANDs per 8
// weights, see common.cuh) into tensor memory (tcgen05.st), and the MMA takes its A operand from there.
// Tensor memory (512 columns): two accumulators (the epilogue overlaps the next tile's main loop) + a ring of
// 64-column weight tiles (256 int8 per lane): 2 x 192 + 2 tiles, or 2 x 128 + 4 tiles where the token tile is
// narrow enough.
// Both rings are sized at launch from the token-tile width: as many TMA stages as fit in shared memory (3 at 192
// tokens, 8 at 16), four weight tiles in tensor memory when the accumulators leave room. For narrow tiles this
// takes TMA latency out of the loop; what remains there is the chain unpack -> MMA -> commit -> unpack, measured
// at ~750 cycles per stage and CTA however few tokens the tile has (the eight MMAs themselves finish within ~100
// cycles of their commit), which caps one CTA at 16 KB of weights per ~0.4 us.
// One thread issues every MMA, and a tcgen05.mma, a tcgen05.commit or an mbarrier wait each cost it some 60
// cycles: a pipeline stage therefore covers 256 codes of K (8 MMAs of 96 cycles) per wait and per commit, and
// a single barrier per stage ("done") releases both the shared-memory slot and the tensor-memory weight tile.
//
// Per CTA (persistent, one per SM), warp roles:
//   warp 0      TMA producer (converged warp, one elected lane issues): per stage one box of packed weights
//               (128 rows x 128 B) and two boxes of int8 activations (BN rows x 128 B), all 128B-swizzled
//   warps 2-5   unpack: thread = one tensor-memory lane = one weight row of the tile
//   warp 1      MMA issuer: 8 x tcgen05.mma (K = 32 each, A in tensor memory) per stage
//   warps 6-13  epilogue (as in linear_tc.cu)
// Every wait on an mbarrier is bounded; on expiry the kernel records SQAP_ERR_TIMEOUT in the device status
// word, drains and frees its tensor memory, and returns.
#include "tc_common.cuh"

namespace sqap {
namespace tcts {

using namespace tc;

constexpr int BM = 128;                   // weight rows per tile (MMA M)
constexpr int BKH = 128;                  // codes of K per TMA box / per block of the packed weight layout
constexpr int BK = 2 * BKH;               // codes of K per pipeline stage
constexpr int BN_MAX = 192;               // tokens per tile (MMA N), runtime BN <= BN_MAX, multiple of 16
constexpr int S_MAX = 8;                  // TMA ring (packed weights + activation tile): depth chosen at launch
constexpr int U_MAX = 4;                  // ring of unpacked weight tiles in tensor memory: 2 or 4
constexpr int W_BYTES = BM * BK / 2;      // 16 KB: a stage's packed weights, 128 rows of 128 bytes
constexpr int RING_BYTES = 206 * 1024;    // stage s: [weights][tokens half 0][tokens half 1]
constexpr int OFF_BAR = RING_BYTES;
constexpr int OFF_TOK = OFF_BAR + 512;    // per-token epilogue constants, two tiles x BN_MAX x 8 bytes
constexpr int OFF_STAGE = OFF_TOK + 2 * BN_MAX * 8;   // staging of the coalesced epilogue (tc_common.cuh)
constexpr int SMEM_BYTES = OFF_STAGE + EPI_STAGE_TOTAL + 1024;  // + slack for 1024-byte alignment
constexpr int A_COLS = BK / 4;            // 64 columns hold 256 int8 per lane
constexpr int ACC_NARROW = 128;           // accumulator stride (columns) with four weight tiles, else BN_MAX
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 32 * (6 + EPI_WARPS);
static_assert(2 * BN_MAX + 2 * A_COLS <= 512 && 2 * ACC_NARROW + U_MAX * A_COLS <= 512, "tensor memory budget");
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
static_assert(8 * (3 * S_MAX + U_MAX + 4) + 16 <= 512, "barrier block");

// Bytes of one stage for a token tile of BN rows (BN a multiple of 16: every operand tile stays 1024-byte aligned).
inline __host__ __device__ int stage_bytes_for(int BN) { return W_BYTES + 2 * BN * BKH; }

// D (tensor memory) += A (tensor memory: lane = row, 4 int8 per 32-bit column) * B (shared memory descriptor).
// Issued by the lane(s) with issue != 0 of a converged warp.
__device__ __forceinline__ void tc_mma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate,
                                             uint32_t issue) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(issue)
        : "memory");
}
// 32 consecutive columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__global__ void __launch_bounds__(THREADS, 1)
w4a4_tc_ts_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_w_up,
                  const __grid_constant__ CUtensorMap tm_x, Args a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar0 = base + OFF_BAR;
    auto full = [&](int s) { return bar0 + 8u * s; };                      // TMA landed (weights + activations)
    auto done = [&](int s) { return bar0 + 8u * (S_MAX + s); };            // the MMAs of the stage in slot s are done
    auto wp_empty = [&](int s) { return bar0 + 8u * (2 * S_MAX + s); };    // unpack warps have read the packed weights
    auto a_full = [&](int j) { return bar0 + 8u * (3 * S_MAX + j); };      // weight tile j is in tensor memory
    auto acc_full = [&](int b) { return bar0 + 8u * (3 * S_MAX + U_MAX + b); };
    auto acc_empty = [&](int b) { return bar0 + 8u * (3 * S_MAX + U_MAX + 2 + b); };
    constexpr int NBAR = 3 * S_MAX + U_MAX + 4;
    const int S = a.stages, U = a.a_tiles;     // S > U: a stage's done barrier must not wrap before the unpack warps saw it
    const uint32_t xh_bytes = static_cast<uint32_t>(a.BN * BKH);
    const uint32_t stage_bytes = static_cast<uint32_t>(stage_bytes_for(a.BN));
    auto w_addr = [&](int s) { return base + s * stage_bytes; };
    auto x_addr = [&](int s, int h) { return base + s * stage_bytes + W_BYTES + h * xh_bytes; };
    const int acc_stride = U == U_MAX ? ACC_NARROW : BN_MAX;               // accumulator b: columns from b * acc_stride
    const int tmem_a_col = 2 * acc_stride;                                 // weight tiles from here
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + OFF_BAR + 8 * NBAR);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + OFF_BAR + 8 * NBAR + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_steps = (a.K + BK - 1) / BK;   // a last half-stage past K is zero-filled by TMA and adds nothing
    const int total_tiles = a.m_tiles * a.n_tiles;
    const uint32_t stage_tx = stage_bytes;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full(s), 1);
            mbar_init(done(s), 1);
            mbar_init(wp_empty(s), 4);
        }
        for (int j = 0; j < U; ++j) {
            mbar_init(a_full(j), 4);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full(b), 1);
            mbar_init(acc_empty(b), EPI_WARPS);
        }
        abort_flag[0] = 0;
        abort_flag[1] = 0;  // always-zero word for waits that must ignore the abort request
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pdl_launch_dependents();   // the next kernel of the stream may start its own set-up (it waits before it touches data)
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool failed = false;
    // Everything above is independent of the kernel before this one in the stream; its output (the activations,
    // their sums and scales) is read, and this kernel's output written, only after pdl_wait() below. The packed
    // weights are immutable, so the producer fetches the first stages' weights BEFORE that wait: they travel while
    // the quantizer before this kernel is still running.
    if (warp == 0) {
        // ---------------- TMA producer: the whole warp walks the loop, one elected lane issues
        const uint32_t issue = elect_one();
        // packed weights of stage ks of the tile at weight row n0: rows of 128 bytes (both 128-code blocks) in one box
        auto load_weights = [&](int st, int ks, int n0) {
            const uint32_t wp = w_addr(st);
            if (a.swiglu) {
                tma_load_2d_if(wp, &tm_w, ks * (BK / 2), n0 / 2, full(st), issue);
                tma_load_2d_if(wp + W_BYTES / 2, &tm_w_up, ks * (BK / 2), n0 / 2, full(st), issue);
            } else {
                tma_load_2d_if(wp, &tm_w, ks * (BK / 2), n0, full(st), issue);
            }
        };
        uint32_t early = 0;   // stages of the first tile whose weights are already on their way
        if (static_cast<int>(blockIdx.x) < total_tiles) {
            early = static_cast<uint32_t>(k_steps < S ? k_steps : S);
            for (uint32_t ks = 0; ks < early; ++ks) {
                mbar_expect_tx_if(full(ks), stage_tx, issue);   // the whole stage: the activations follow after the wait
                load_weights(static_cast<int>(ks), static_cast<int>(ks), (static_cast<int>(blockIdx.x) % a.n_tiles) * BM);
            }
        }
        pdl_wait();
        uint32_t it = 0;
        int s = 0;
        uint32_t ph = 0;
        for (int tile = blockIdx.x; tile < total_tiles && !failed; tile += gridDim.x) {
            const int n0 = (tile % a.n_tiles) * BM, m0 = (tile / a.n_tiles) * a.BN;
            for (int ks = 0; ks < k_steps; ++ks, ++it) {
                if (it >= early) {
                    const bool ok = mbar_wait(done(s), ph ^ 1u, abort_flag) && mbar_wait(wp_empty(s), ph ^ 1u, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                    mbar_expect_tx_if(full(s), stage_tx, issue);
                    load_weights(s, ks, n0);
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) tma_load_2d_if(x_addr(s, h), &tm_x, ks * BK + h * BKH, m0, full(s), issue);
                if (++s == S) { s = 0; ph ^= 1u; }
            }
        }
        if (failed && issue) {
            // drain: give every armed stage a bounded chance to land before shared memory is released
            for (int back = 0; back < S; ++back) {
                const uint32_t last = it > static_cast<uint32_t>(back) ? (it - 1 - back) : 0xFFFFFFFFu;
                if (last != 0xFFFFFFFFu) mbar_wait(full(last % S), (last / S) & 1u, abort_flag + 1);
            }
        }
    } else if (warp == 1) {
        pdl_wait();
        // ---------------- MMA issuer: the whole warp walks the loop, one elected lane issues
        {
            const uint32_t issue = elect_one();
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a.BN >> 3) << 17) |
                                   (static_cast<uint32_t>(BM >> 4) << 24);
            uint32_t lt = 0;
            int s = 0, j = 0;
            uint32_t jph = 0;
            for (int tile = blockIdx.x; tile < total_tiles && !failed; tile += gridDim.x, ++lt) {
                const int b = lt & 1;
                if (!__all_sync(0xffffffffu, mbar_wait(acc_empty(b), ((lt >> 1) & 1u) ^ 1u, abort_flag))) { failed = true; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(b * acc_stride);
                for (int ks = 0; ks < k_steps; ++ks) {
                    // the unpack warps arrive on a_full(j) only after they saw full(s): this wait covers both operands
                    if (!__all_sync(0xffffffffu, mbar_wait(a_full(j), jph, abort_flag))) { failed = true; break; }
                    tc_fence_after();
                    const uint32_t a_tmem = tmem_base + static_cast<uint32_t>(tmem_a_col + j * A_COLS);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint64_t bdesc = smem_desc_sw128(x_addr(s, h));
#pragma unroll
                        for (int k = 0; k < BKH / 32; ++k)
                            tc_mma_i8_ts(d_tmem, a_tmem + 32u * h + 8u * k, bdesc + 2u * k, idesc, (ks | h | k) != 0 ? 1u : 0u, issue);
                    }
                    tc_commit_if(done(s), issue);
                    if (++s == S) s = 0;
                    if (++j == U) { j = 0; jph ^= 1u; }
                }
                if (failed) break;
                tc_commit_if(acc_full(b), issue);
            }
        }
    } else if (warp < 6) {
        // (no dependency wait here: these warps touch shared and tensor memory only, and may unpack the weights that
        // were fetched early while the kernel before this one still runs)
        // ---------------- unpack warps: thread = one tensor-memory lane = one weight row of the tile
        const int quad = warp & 3;                 // the lane quadrant this warp may write
        const int L = quad * 32 + lane;            // tensor-memory lane
        // Source row of the packed stage. Plain: row L. SwiGLU: the stage holds 64 gate rows then 64 up rows;
        // within each quadrant lanes 0-15 take gate rows and lanes 16-31 the up rows of the same 16 channels.
        const int src_row = a.swiglu ? (quad * 16 + (lane & 15) + ((lane >> 4) << 6)) : L;
        // 128-byte rows under the 128B TMA swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7).
        // Consecutive rows then hit different banks for the same c, so the register a chunk lands in is fixed.
        const int sw = src_row & 7;
        const int my_tiles = static_cast<int>(blockIdx.x) < total_tiles
                                 ? (total_tiles - 1 - static_cast<int>(blockIdx.x)) / static_cast<int>(gridDim.x) + 1 : 0;
        const uint32_t total_its = static_cast<uint32_t>(my_tiles) * static_cast<uint32_t>(k_steps);
        // One stage: packed row (shared memory) -> two ANDs per word -> tensor-memory weight tile j_.
        auto unpack_stage = [&](int s_, int j_) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint8_t* src = sm + s_ * stage_bytes + src_row * 128;
                uint32_t r[32];   // column q holds codes k = 4q .. 4q+3 of this half of the row
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint4 v = *reinterpret_cast<const uint4*>(src + (((4 * h + c) ^ sw) << 4));
                    r[4 * c + 0] = v.x & 0x0F0F0F0Fu; r[4 * c + 1] = v.y & 0x0F0F0F0Fu;      // codes 16c .. 16c+15 (+8)
                    r[4 * c + 2] = v.z & 0x0F0F0F0Fu; r[4 * c + 3] = v.w & 0x0F0F0F0Fu;
                    r[16 + 4 * c + 0] = v.x & 0xF0F0F0F0u; r[16 + 4 * c + 1] = v.y & 0xF0F0F0F0u;  // codes 64+16c .. (x16)
                    r[16 + 4 * c + 2] = v.z & 0xF0F0F0F0u; r[16 + 4 * c + 3] = v.w & 0xF0F0F0F0u;
                }
                tc_st32(tmem_base + (static_cast<uint32_t>(quad * 32) << 16) +
                            static_cast<uint32_t>(tmem_a_col + j_ * A_COLS + 32 * h), r);
            }
        };
        // With deep rings (narrow token tiles) two stages per round: every barrier operation costs this warp its
        // latency (100-200 cycles even on a completed phase), so the four probes of a round are issued together and
        // the two stages share one wait::st and one round of arrivals; with shallow rings that would hold two of three
        // slots at once, so there a round is one stage. Stage it lives in slot it % S and weight tile it % U; weight
        // tile j was last read by the MMAs of stage it - U, whose completion is that stage's done barrier (slot sd).
        const bool pairwise = S >= 6 && U == U_MAX;
        int s = 0, j = 0, sd = 0;
        uint32_t ph = 0, phd = 0;
        for (uint32_t it = 0; it < total_its && !failed; it += pairwise ? 2u : 1u) {
            const bool two = pairwise && it + 1 < total_its;
            const int s1 = s + 1 == S ? 0 : s + 1, j1 = j + 1;          // pairwise: U is even and j stays even
            const uint32_t ph1 = s + 1 == S ? ph ^ 1u : ph;
            const bool need_done = it >= static_cast<uint32_t>(U);      // then also for stage it + 1
            const int sd1 = sd + 1 == S ? 0 : sd + 1;
            const uint32_t phd1 = sd + 1 == S ? phd ^ 1u : phd;
            const bool f0 = mbar_test_wait(full(s), ph);
            const bool f1 = !two || mbar_test_wait(full(s1), ph1);
            const bool d0 = !need_done || mbar_test_wait(done(sd), phd);
            const bool d1 = !need_done || !two || mbar_test_wait(done(sd1), phd1);
            bool ok = f0 || mbar_wait(full(s), ph, abort_flag);
            ok = ok && (f1 || mbar_wait(full(s1), ph1, abort_flag));
            ok = ok && (d0 || mbar_wait(done(sd), phd, abort_flag));
            ok = ok && (d1 || mbar_wait(done(sd1), phd1, abort_flag));
            if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
            tc_fence_after();
            unpack_stage(s, j);
            if (two) unpack_stage(s1, j1);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(wp_empty(s));
                mbar_arrive(a_full(j));
                if (two) {
                    mbar_arrive(wp_empty(s1));
                    mbar_arrive(a_full(j1));
                }
            }
            const int adv = pairwise ? 2 : 1;
            if (need_done) {
                sd += adv;
                if (sd >= S) { sd -= S; phd ^= 1u; }
            }
            s += adv;
            if (s >= S) { s -= S; ph ^= 1u; }
            j += adv;
            if (j >= U) j = 0;
        }
    } else {
        pdl_wait();
        // ---------------- epilogue warps: warp % 4 selects the 32-lane quadrant of tensor memory
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const int split = ((a.BN / 16 + 1) / 2) * 16;  // first token of the second half of the tile
        const int c_begin = (warp - 6) < 4 ? 0 : split;
        const int c_end = (warp - 6) < 4 ? split : a.BN;
        uint32_t lt = 0;
        for (int tile = blockIdx.x; tile < total_tiles && !failed; tile += gridDim.x, ++lt) {
            const int b = lt & 1;
            const int n0 = (tile % a.n_tiles) * BM, m0 = (tile / a.n_tiles) * a.BN;
            // stage the tile's per-token constants (the other buffer may still be read by slower warps)
            int2* tok = reinterpret_cast<int2*>(sm + OFF_TOK) + b * BN_MAX;
            const int et = static_cast<int>(threadIdx.x) - 6 * 32;
            if (et < a.BN) {
                const int m = m0 + et;
                tok[et] = m < a.M ? make_int2(__ldg(a.bias_sum + m) << 7, __float_as_int(__ldg(a.act_scales + m))) : make_int2(0, 0);
            }
            // all epilogue warps leave the loop together if any wait ran out, so the barrier below never hangs
            if (bar_or(1, 32 * EPI_WARPS, !mbar_wait(acc_full(b), (lt >> 1) & 1u, abort_flag))) { failed = true; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(b * acc_stride);
            int n;
            float sw;
            bool n_ok;
            if (a.swiglu) {
                n = n0 / 2 + quad * 16 + (lane & 15);      // lanes 0-15 of a quadrant: gate, 16-31: up, same channels
                n_ok = n < a.N;
                sw = n_ok ? __half2float((lane & 16) ? a.w_up_scales[n] : a.w_scales[n]) : 0.0f;
            } else {
                n = n0 + row;
                n_ok = n < a.N;
                sw = n_ok ? __half2float(a.w_scales[n]) : 0.0f;
            }
            // fp16 / bf16: through shared memory, 16 bytes per thread to global memory; raw int32 (checking): directly
            const int hf = (warp - 6) >> 2, tid_half = static_cast<int>(threadIdx.x) - (6 + 4 * hf) * 32;
            uint8_t* stage_half = sm + OFF_STAGE + hf * 2 * EPI_STAGE_BYTES;
            if (a.swiglu) {
                const int ch = quad * 16 + (lane & 15);
                if (a.out_dtype == SQAP_FP16) epilogue_tile_coalesced<SQAP_FP16, true>(a, taddr, m0, c_begin, c_end, n0 / 2, ch, sw, lane, tok, stage_half, tid_half, 2 + hf);
                else epilogue_tile_coalesced<SQAP_BF16, true>(a, taddr, m0, c_begin, c_end, n0 / 2, ch, sw, lane, tok, stage_half, tid_half, 2 + hf);
            } else {
                if (a.out_dtype == SQAP_FP16) epilogue_tile_coalesced<SQAP_FP16, false>(a, taddr, m0, c_begin, c_end, n0, row, sw, lane, tok, stage_half, tid_half, 2 + hf);
                else if (a.out_dtype == SQAP_BF16) epilogue_tile_coalesced<SQAP_BF16, false>(a, taddr, m0, c_begin, c_end, n0, row, sw, lane, tok, stage_half, tid_half, 2 + hf);
                else epilogue_tile_staged<SQAP_I32, false, 1>(a, taddr, m0, c_begin, c_end, n, n_ok, sw, lane, tok);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(b));
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

}  // namespace tcts

sqap_status launch_linear_tcgen05_ts(const LinearArgs& a, cudaStream_t s) {
    using namespace tcts;
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
    k.swiglu = a.w_up ? 1 : 0;
    k.n_tiles = k.swiglu ? (2 * a.N + BM - 1) / BM : (a.N + BM - 1) / BM;
    choose_token_tiles(a.M, k.n_tiles, sm_count(), BN_MAX, 256, &k.m_tiles, &k.BN);
    k.out_dtype = a.out_dtype;
    k.stages = RING_BYTES / stage_bytes_for(k.BN);
    if (k.stages > S_MAX) k.stages = S_MAX;
    k.a_tiles = (k.BN <= ACC_NARROW && k.stages > U_MAX) ? U_MAX : 2;
    k.status = device_status_word();
    if (!k.status) return SQAP_ERR_CUDA;

    CUtensorMap tm_w, tm_u, tm_x;
    if (!weight_maps(a, k.swiglu != 0, BM, BK / 2, &tm_w, &tm_u)) return SQAP_ERR_CUDA;
    if (!make_map(&tm_x, a.x8, a.M, a.K, k.BN, BKH, CU_TENSOR_MAP_SWIZZLE_128B)) return SQAP_ERR_CUDA;

    static PerDevice<int> setup;
    const sqap_status st = setup.run([](int*) { return set_max_dynamic_smem(w4a4_tc_ts_kernel, SMEM_BYTES); });
    if (st != SQAP_OK) return st;
    const int tiles = k.m_tiles * k.n_tiles;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    const cudaError_t e = launch_dependent(w4a4_tc_ts_kernel, dim3(grid), dim3(THREADS), SMEM_BYTES, s, tm_w, tm_u, tm_x, k);
    if (e != cudaSuccess) note_cuda_error(e);
    count_launch();
    return check_launch();
}

}  // namespace sqap

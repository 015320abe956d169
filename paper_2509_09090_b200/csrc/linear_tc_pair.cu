// tcgen05 kernel of the W4A4 linear on CTA PAIRS (cta_group::2) with the weight operand in tensor memory:
// the large-M kernel.
//
// A cluster of two CTAs (the two SMs of a TPC) computes one 256 x BN tile: D[n][m] = sum_k W[n][k] * X[m][k],
// weights as the MMA-M operand (128 rows per CTA, 256 per pair), tokens as the MMA-N operand (BN <= 192).
// The one-CTA kernels (linear_tc.cu, linear_tc_ts.cu) are bounded by what an SM can pull from L2 (about 58 bytes
// per clock measured): the int8 token tile is their large operand. Here each CTA stages only HALF of the token
// tile (BN/2 rows) and the pair's tensor cores share both halves, so a CTA moves 40 KB instead of 64 KB per 256
// codes of K. As in linear_tc_ts.cu the unpacked weights live in tensor memory (unpack warps: packed TMA tile ->
// registers -> tcgen05.st; the MMA takes A from there), a pipeline stage covers 256 codes of K (one thread issues
// every MMA, and each MMA, commit and wait costs it some 60 cycles), and one barrier per stage ("done") releases
// the shared-memory slot and the tensor-memory weight tile in both CTAs (tcgen05.commit multicast).
// Tensor memory per CTA (512 columns): two accumulators of 192 columns + a ring of two 64-column weight tiles.
//
// Per CTA, warp roles:
//   warp 0      TMA producer: per stage one box of packed weights (128 rows x 128 B) and two boxes of int8
//               activations (BN/2 rows x 128 B), all 128B-swizzled; the activation loads of BOTH CTAs complete
//               on the leader CTA's barrier (the MMA is issued there)
//   warps 2-5   unpack: thread = one tensor-memory lane = one weight row of the CTA's tile; signal the leader
//   warp 1      leader CTA only: 8 x tcgen05.mma.cta_group::2 (M = 256, N = BN, K = 32) per stage
//   warps 6-13  epilogue of the CTA's own 128 accumulator rows
// Every wait on an mbarrier is bounded; on expiry the kernel records SQAP_ERR_TIMEOUT in the device status
// word, drains, and returns through the cluster barrier.
#include "tc_common.cuh"

namespace sqap {
namespace tcpair {

using namespace tc;

constexpr int BM = 128;                   // weight rows per CTA (MMA M = 256 per pair)
constexpr int BKH = 128;                  // codes of K per TMA box / per block of the packed weight layout
constexpr int BK = 2 * BKH;               // codes of K per pipeline stage
constexpr int BN_MAX = 192;               // tokens per pair tile (MMA N), runtime BN <= BN_MAX, multiple of 16
constexpr int S = 5;                      // TMA ring: packed weights + this CTA's half of the token tile
constexpr int U = 2;                      // ring of unpacked weight tiles in tensor memory
constexpr int XH_BYTES = BN_MAX / 2 * BKH;  // 12 KB: one 128-code half of a stage, this CTA's half of the tokens
constexpr int WPH_BYTES = BM * BKH / 2;   // 8 KB: one half of a stage's packed weights
constexpr int OFF_X = 0;
constexpr int OFF_WP = OFF_X + S * 2 * XH_BYTES;
constexpr int OFF_BAR = OFF_WP + S * 2 * WPH_BYTES;
constexpr int OFF_TOK = OFF_BAR + 512;    // per-token epilogue constants, two tiles x BN_MAX x 8 bytes
constexpr int OFF_STAGE = OFF_TOK + 2 * BN_MAX * 8;   // staging of the coalesced epilogue (tc_common.cuh)
constexpr int SMEM_BYTES = OFF_STAGE + EPI_STAGE_TOTAL + 1024;  // + slack for 1024-byte alignment
constexpr int TMEM_A_COL = 2 * BN_MAX;    // columns [0,192) and [192,384): accumulators; from 384: weight tiles
constexpr int A_COLS = BK / 4;            // 64 columns hold 256 int8 per lane
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 32 * (6 + EPI_WARPS);
static_assert(XH_BYTES % 1024 == 0 && OFF_WP % 1024 == 0, "operand tiles must be 1024-byte aligned");
static_assert(TMEM_A_COL + U * A_COLS <= 512, "tensor memory budget");
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
static_assert(S > U, "a stage's done barrier must not wrap before the unpack warps have seen it");

// D (tensor memory) += A (tensor memory: lane = row, 4 int8 per 32-bit column) * B (shared memory descriptor).
// Issued by the lane(s) with issue != 0 of a converged warp.
__device__ __forceinline__ void tc_mma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate,
                                             uint32_t issue) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::2.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
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

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Arrive on a barrier that may live in the peer CTA. Release at CTA scope (the default) is what this needs: what
// the signal stands for is tensor-memory writes already waited for (tcgen05.wait::st) or tensor-memory reads
// already complete; a cluster-scope release was measured to cost about 1300 cycles per arrive.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into this CTA's shared memory whose completion bytes are counted on a barrier that may live in
// the peer CTA (cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar_cluster)
        : "memory");
}
// Arrives (once) on the barrier at this offset in both CTAs of the pair when all MMAs issued so far are done.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint32_t issue) {
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.b32 q, %2, 0;\n\t"
        "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
        ::"r"(bar), "h"(static_cast<uint16_t>(3)), "r"(issue)
        : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
w4a4_tc_pair_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_w_up,
                  const __grid_constant__ CUtensorMap tm_x, Args a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // identical in both CTAs of the pair
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar0 = base + OFF_BAR;
    auto full = [&](int s) { return bar0 + 8u * s; };                  // this CTA's packed weights landed
    auto x_full = [&](int s) { return bar0 + 8u * (3 * S + U + 4 + s); };  // leader's: both CTAs' activation halves landed
    auto done = [&](int s) { return bar0 + 8u * (S + s); };            // the MMAs of the stage in slot s are done
    auto wp_empty = [&](int s) { return bar0 + 8u * (2 * S + s); };    // unpack warps have read the packed weights
    auto a_full = [&](int j) { return bar0 + 8u * (3 * S + j); };      // weight tile j is in tensor memory
    auto acc_full = [&](int b) { return bar0 + 8u * (3 * S + U + b); };
    auto acc_empty = [&](int b) { return bar0 + 8u * (3 * S + U + 2 + b); };
    constexpr int NBAR = 4 * S + U + 4;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + OFF_BAR + 8 * NBAR);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + OFF_BAR + 8 * NBAR + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = leader (issues the MMAs)
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int half_bn = a.BN >> 1;
    const int k_steps = (a.K + BK - 1) / BK;   // a last half-stage past K is zero-filled by TMA and adds nothing
    const int total_tiles = a.m_tiles * a.n_tiles;
    const uint32_t w_tx = static_cast<uint32_t>(2 * WPH_BYTES), x_tx = static_cast<uint32_t>(2 * a.BN * BKH);  // x: both CTAs

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full(s), 1);
            mbar_init(x_full(s), 1);
            mbar_init(done(s), 1);
            mbar_init(wp_empty(s), 4);
        }
        for (int j = 0; j < U; ++j) {
            mbar_init(a_full(j), 8);   // 4 unpack warps of each CTA; the leader's barrier is the one in use
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full(b), 1);
            mbar_init(acc_empty(b), 2 * EPI_WARPS);   // leader's
        }
        abort_flag[0] = 0;
        abort_flag[1] = 0;  // always-zero word for waits that must ignore the abort request
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    pdl_launch_dependents();   // the next kernel of the stream may start its own set-up (it waits before it touches data)
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool failed = false;
    // Everything above is independent of the kernel before this one in the stream; its output (the activations,
    // their sums and scales) is read, and this kernel's output written, only after pdl_wait() below. The packed
    // weights are immutable, so the producer fetches the first stages' weights BEFORE that wait: they travel while
    // the quantizer before this kernel is still running.
    if (warp == 0) {
        // ---------------- TMA producer (one lane)
        if (lane == 0) {
            // packed weights of stage ks of the tile whose weight rows (this CTA's half) start at n0: rows of 128
            // bytes (both 128-code blocks of the stage) in one box
            auto load_weights = [&](int st, int ks, int n0) {
                const uint32_t wp = base + OFF_WP + st * (2 * WPH_BYTES);
                if (a.swiglu) {
                    tma_load_2d(wp, &tm_w, ks * (BK / 2), n0 / 2, full(st));
                    tma_load_2d(wp + WPH_BYTES, &tm_w_up, ks * (BK / 2), n0 / 2, full(st));
                } else {
                    tma_load_2d(wp, &tm_w, ks * (BK / 2), n0, full(st));
                }
            };
            uint32_t early = 0;   // stages of the first tile whose weights are already on their way
            if (pair < total_tiles) {
                early = static_cast<uint32_t>(k_steps < S ? k_steps : S);
                for (uint32_t ks = 0; ks < early; ++ks) {
                    mbar_expect_tx(full(ks), w_tx);
                    load_weights(static_cast<int>(ks), static_cast<int>(ks), (pair % a.n_tiles) * (2 * BM) + static_cast<int>(rank) * BM);
                }
            }
            pdl_wait();
            uint32_t it = 0;
            for (int tile = pair; tile < total_tiles && !failed; tile += n_pairs) {
                const int n0 = (tile % a.n_tiles) * (2 * BM) + static_cast<int>(rank) * BM;
                const int m0 = (tile / a.n_tiles) * a.BN + static_cast<int>(rank) * half_bn;
                for (int ks = 0; ks < k_steps; ++ks, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1u;
                    if (it >= early) {
                        if (!mbar_wait(done(s), ph ^ 1u, abort_flag) || !mbar_wait(wp_empty(s), ph ^ 1u, abort_flag)) { failed = true; break; }
                        mbar_expect_tx(full(s), w_tx);
                        load_weights(s, ks, n0);
                    }
                    if (rank == 0) mbar_expect_tx(x_full(s), x_tx);
                    const uint32_t x_bar = map_to_cta(x_full(s), 0);
#pragma unroll
                    for (int h = 0; h < 2; ++h)
                        tma_load_2d_pair(base + OFF_X + (2 * s + h) * XH_BYTES, &tm_x, ks * BK + h * BKH, m0, x_bar);
                }
            }
            if (failed) {
                // drain: give every armed weight load a bounded chance to land; the activation loads were issued
                // alongside and are counted on the leader's barrier, so wait a further fixed while for them
                for (int s = 0; s < S; ++s) {
                    const uint32_t last = it > static_cast<uint32_t>(s) ? (it - 1 - s) : 0xFFFFFFFFu;
                    if (last != 0xFFFFFFFFu) mbar_wait(full(last % S), (last / S) & 1u, abort_flag + 1);
                }
                const long long t0 = clock64();
                while (clock64() - t0 < 200000) {}
            }
        }
    } else if (warp == 1) {
        pdl_wait();
        // ---------------- MMA issuer (leader CTA): the whole warp walks the loop, one elected lane issues
        if (rank == 0) {
            const uint32_t issue = elect_one();
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a.BN >> 3) << 17) |
                                   (static_cast<uint32_t>((2 * BM) >> 4) << 24);
            uint32_t it = 0, lt = 0;
            for (int tile = pair; tile < total_tiles && !failed; tile += n_pairs, ++lt) {
                const int b = lt & 1;
                if (!__all_sync(0xffffffffu, mbar_wait(acc_empty(b), ((lt >> 1) & 1u) ^ 1u, abort_flag))) { failed = true; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(b * BN_MAX);
                for (int ks = 0; ks < k_steps; ++ks, ++it) {
                    const int s = it % S, j = it % U;
                    const bool ok = mbar_wait(x_full(s), (it / S) & 1u, abort_flag) && mbar_wait(a_full(j), (it / U) & 1u, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                    tc_fence_after();
                    const uint32_t a_tmem = tmem_base + static_cast<uint32_t>(TMEM_A_COL + j * A_COLS);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint64_t bdesc = smem_desc_sw128(base + OFF_X + (2 * s + h) * XH_BYTES);
#pragma unroll
                        for (int k = 0; k < BKH / 32; ++k)
                            tc_mma_i8_ts(d_tmem, a_tmem + 32u * h + 8u * k, bdesc + 2u * k, idesc, (ks | h | k) != 0 ? 1u : 0u, issue);
                    }
                    tc_commit_pair(done(s), issue);
                }
                if (failed) break;
                tc_commit_pair(acc_full(b), issue);
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
        uint32_t it = 0;
        for (int tile = pair; tile < total_tiles && !failed; tile += n_pairs) {
            for (int ks = 0; ks < k_steps; ++ks, ++it) {
                const int s = it % S, j = it % U;
                // weight tile j was last read by the MMAs of stage it - U, whose completion is done((it - U) % S)
                bool ok = mbar_wait(full(s), (it / S) & 1u, abort_flag);
                if (ok && it >= U) ok = mbar_wait(done((it - U) % S), ((it - U) / S) & 1u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
                tc_fence_after();
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint8_t* src = sm + OFF_WP + s * (2 * WPH_BYTES) + src_row * 128;
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
                                static_cast<uint32_t>(TMEM_A_COL + j * A_COLS + 32 * h), r);
                }
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(wp_empty(s));
                    mbar_arrive_cluster(map_to_cta(a_full(j), 0));
                }
            }
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
        for (int tile = pair; tile < total_tiles && !failed; tile += n_pairs, ++lt) {
            const int b = lt & 1;
            const int n0 = (tile % a.n_tiles) * (2 * BM) + static_cast<int>(rank) * BM, m0 = (tile / a.n_tiles) * a.BN;
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
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(b * BN_MAX);
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
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty(b), 0));
        }
    }

    if (failed) {
        *abort_flag = 1;
        atomicOr(a.status, SQAP_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // neither CTA leaves (or frees tensor memory) while the other may still signal it
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
}

}  // namespace tcpair

sqap_status launch_linear_tcgen05_pair(const LinearArgs& a, cudaStream_t s) {
    using namespace tcpair;
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
    k.n_tiles = k.swiglu ? (2 * a.N + 2 * BM - 1) / (2 * BM) : (a.N + 2 * BM - 1) / (2 * BM);
    k.out_dtype = a.out_dtype;
    k.status = device_status_word();
    if (!k.status) return SQAP_ERR_CUDA;

    // Once per device: the shared-memory limit, and the number of CTA pairs that can be resident at once. A pair
    // needs both SMs of one TPC, so this can be fewer than half the SM count; a persistent grid larger than that
    // would run its surplus pairs as a second wave.
    static PerDevice<int> setup;
    const int* max_pairs_p = nullptr;
    const sqap_status st = setup.run(
        [](int* pairs) {
            const sqap_status s0 = set_max_dynamic_smem(w4a4_tc_pair_kernel, SMEM_BYTES);
            if (s0 != SQAP_OK) return s0;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(static_cast<unsigned>(sm_count() / 2 * 2));
            cfg.blockDim = dim3(THREADS);
            cfg.dynamicSmemBytes = SMEM_BYTES;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = 2;
            attr.val.clusterDim.y = 1;
            attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, w4a4_tc_pair_kernel, &cfg) != cudaSuccess || n <= 0) {
                cudaGetLastError();
                n = sm_count() / 2;
            }
            *pairs = n;
            return SQAP_OK;
        },
        &max_pairs_p);
    if (st != SQAP_OK) return st;
    const int max_pairs = *max_pairs_p;
    choose_token_tiles(a.M, k.n_tiles, max_pairs, BN_MAX, 128, &k.m_tiles, &k.BN);
    CUtensorMap tm_w, tm_u, tm_x;
    if (!weight_maps(a, k.swiglu != 0, BM, BK / 2, &tm_w, &tm_u)) return SQAP_ERR_CUDA;
    if (!make_map(&tm_x, a.x8, a.M, a.K, k.BN / 2, BKH, CU_TENSOR_MAP_SWIZZLE_128B)) return SQAP_ERR_CUDA;

    const int tiles = k.m_tiles * k.n_tiles;
    const int pairs = tiles < max_pairs ? tiles : max_pairs;
    const cudaError_t e = launch_dependent(w4a4_tc_pair_kernel, dim3(2 * pairs), dim3(THREADS), SMEM_BYTES, s, tm_w, tm_u, tm_x, k);
    if (e != cudaSuccess) note_cuda_error(e);
    count_launch();
    return check_launch();
}

}  // namespace sqap

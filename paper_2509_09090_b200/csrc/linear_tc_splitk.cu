// tcgen05 kernel of the W4A4 linear for token counts between the weight streamers and the CTA-pair kernel
// (a few dozen to a few hundred rows: one observation before and after pruning): split K across the CTAs of a
// thread-block CLUSTER and add the partial accumulators through distributed shared memory.
//
// Why: with few tokens a tile's main loop is bounded by the rate at which one CTA unpacks weights into tensor
// memory (about 750 cycles per 256 codes of K and 128 weight rows, whatever the tile width), not by the tensor
// core, so the time of a linear is (stages per CTA) x 750 cycles, and with N = 4096 there are only 32 weight tiles
// for 148 SMs. Cutting every tile's K range into `ksplit` slices multiplies the CTA count and divides the chain.
// The partial sums are int32 and exact, so the order of the additions does not matter.
//
// One cluster of `ksplit` (1 to 4) CTAs per 128 x BN output tile; CTA r of the cluster runs the pipeline of
// linear_tc_ts.cu (TMA ring -> unpack warps -> tensor memory -> tcgen05.mma with A from tensor memory) over its
// slice of the K stages, into one accumulator in its own tensor memory. Then, with the main loops of all CTAs of
// the cluster finished (cluster barrier), a reduce-scatter through shared memory: the tile's 16-token chunks are
// dealt round-robin to the CTAs; every CTA writes each chunk of its partial accumulator into the owner's shared
// memory (st.shared::cluster; its own chunks take the same route, locally), a second cluster barrier makes the
// writes visible, and each CTA adds the `ksplit` partials of its own chunks, applies the epilogue and stores them.
// The exchange buffer is the TMA ring, idle by then, so it costs no shared memory; the epilogue's global stores are
// spread over the cluster as well. No global-memory round trip, no atomics, no fences beyond the two barriers.
//
// Not persistent: a cluster computes one tile, the hardware scheduler balances the clusters over the SMs.
// Every wait on an mbarrier is bounded; on expiry the kernel records SQAP_ERR_TIMEOUT in the device status word
// and runs on to the two cluster barriers (which every thread of every CTA reaches on every path), frees its
// tensor memory and returns.
#include "tc_common.cuh"

namespace sqap {
namespace tcsk {

using namespace tc;

constexpr int BM = 128;                   // weight rows per tile (MMA M)
constexpr int BKH = 128;                  // codes of K per TMA box / per block of the packed weight layout
constexpr int BK = 2 * BKH;               // codes of K per pipeline stage
constexpr int BN_MAX = 192;               // tokens per tile (MMA N), runtime BN <= BN_MAX, multiple of 16
constexpr int S_MAX = 8;                  // TMA ring (packed weights + activation tile): depth chosen at launch
constexpr int U_MAX = 4;                  // ring of unpacked weight tiles in tensor memory: 2 to 4
constexpr int KSPLIT_MAX = 4;             // CTAs per cluster
constexpr int W_BYTES = BM * BK / 2;      // 16 KB: a stage's packed weights, 128 rows of 128 bytes
constexpr int RING_BYTES = 222 * 1024;    // stage s: [weights][tokens half 0][tokens half 1]; after the main loop:
constexpr int OFF_XCHG = 0;               //   the exchange buffer (partial accumulators, at most 120 KB)
constexpr int OFF_STAGE = 128 * 1024;     //   and the staging of the coalesced epilogue: 3 groups x 2 buffers x 4 KB
constexpr int OFF_BAR = RING_BYTES;
constexpr int OFF_TOK = OFF_BAR + 512;    // per-token epilogue constants, BN_MAX x 8 bytes
constexpr int SMEM_BYTES = OFF_TOK + BN_MAX * 8 + 1024;  // + slack for 1024-byte alignment
constexpr int A_COLS = BK / 4;            // 64 columns hold 256 int8 per lane
constexpr int TMEM_A_COL = 256;           // accumulator: columns [0, BN); weight tiles from here
constexpr int THREADS = 32 * 14;          // as the other tcgen05 kernels (warps 6-13 have no main-loop role here)
constexpr int EPI_GROUPS = 3;             // groups of four warps (one per tensor-memory lane quadrant) in the epilogue
constexpr int CHUNK_BYTES = BM * 16 * 4;  // one 16-token chunk of a partial accumulator: 128 rows x 16 int32
static_assert(TMEM_A_COL + U_MAX * A_COLS <= 512 && BN_MAX <= TMEM_A_COL, "tensor memory budget");
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
static_assert(8 * (3 * S_MAX + U_MAX + 1) + 16 <= 512, "barrier block");
// every CTA receives ksplit partials of at most ceil(chunks / ksplit) chunks
static_assert((BN_MAX / 16 + KSPLIT_MAX - 1) * CHUNK_BYTES <= OFF_STAGE, "exchange buffer ends before the staging");
static_assert(OFF_STAGE + EPI_GROUPS * 2 * EPI_STAGE_BYTES <= RING_BYTES, "staging fits the ring");

inline __host__ __device__ int stage_bytes_for(int BN) { return W_BYTES + 2 * BN * BKH; }

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
// Barrier among all threads of all CTAs of the cluster; orders (release / acquire at cluster scope) the shared-memory
// writes made before it, distributed ones included, against the reads after it.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Args::stages / a_tiles: ring depths; Args::m_tiles x n_tiles tiles; ksplit = cluster size (gridDim.x = tiles * ksplit).
__global__ void __launch_bounds__(THREADS, 1)
w4a4_tc_splitk_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_w_up,
                      const __grid_constant__ CUtensorMap tm_x, Args a, int ksplit) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // identical in every CTA of the cluster
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar0 = base + OFF_BAR;
    auto full = [&](int s) { return bar0 + 8u * s; };                      // TMA landed (weights + activations)
    auto done = [&](int s) { return bar0 + 8u * (S_MAX + s); };            // the MMAs of the stage in slot s are done
    auto wp_empty = [&](int s) { return bar0 + 8u * (2 * S_MAX + s); };    // unpack warps have read the packed weights
    auto a_full = [&](int j) { return bar0 + 8u * (3 * S_MAX + j); };      // weight tile j is in tensor memory
    const uint32_t acc_full = bar0 + 8u * (3 * S_MAX + U_MAX);            // every MMA of this CTA is done
    constexpr int NBAR = 3 * S_MAX + U_MAX + 1;
    const int S = a.stages, U = a.a_tiles;     // S > U: a stage's done barrier must not wrap before the unpack warps saw it
    const uint32_t xh_bytes = static_cast<uint32_t>(a.BN * BKH);
    const uint32_t stage_bytes = static_cast<uint32_t>(stage_bytes_for(a.BN));
    auto w_addr = [&](int s) { return base + s * stage_bytes; };
    auto x_addr = [&](int s, int h) { return base + s * stage_bytes + W_BYTES + h * xh_bytes; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + OFF_BAR + 8 * NBAR);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + OFF_BAR + 8 * NBAR + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = static_cast<int>(cluster_ctarank());
    const int tile = static_cast<int>(blockIdx.x) / ksplit;
    const int n0 = (tile % a.n_tiles) * BM, m0 = (tile / a.n_tiles) * a.BN;
    const int k_steps = (a.K + BK - 1) / BK;   // a last half-stage past K is zero-filled by TMA and adds nothing
    const int ks_begin = rank * k_steps / ksplit, ks_end = (rank + 1) * k_steps / ksplit;   // ksplit <= k_steps: never empty
    const int my_steps = ks_end - ks_begin;

    // Set-up. Warp 0 initialises the barriers and at once issues the WEIGHT loads of its first stages (fresh ring slots
    // need no waiting), so that the first weights are on their way while tensor memory is allocated and the CTA
    // meets, and, when this kernel was launched as a programmatic dependent, while the kernel before it in the
    // stream is still running: packed weights never change, whereas the tokens are that kernel's output and are
    // fetched after the dependency wait.
    auto issue_weights = [&](int ks, int s, uint32_t issue) {
        mbar_expect_tx_if(full(s), stage_bytes, issue);   // the whole stage's bytes: the tokens follow
        const uint32_t wp = w_addr(s);
        if (a.swiglu) {
            tma_load_2d_if(wp, &tm_w, ks * (BK / 2), n0 / 2, full(s), issue);
            tma_load_2d_if(wp + W_BYTES / 2, &tm_w_up, ks * (BK / 2), n0 / 2, full(s), issue);
        } else {
            tma_load_2d_if(wp, &tm_w, ks * (BK / 2), n0, full(s), issue);
        }
    };
    auto issue_tokens = [&](int ks, int s, uint32_t issue) {
#pragma unroll
        for (int h = 0; h < 2; ++h) tma_load_2d_if(x_addr(s, h), &tm_x, ks * BK + h * BKH, m0, full(s), issue);
    };
    const int pre = my_steps < S ? my_steps : S;   // stages issued before the set-up barrier
    if (warp == 0) {
        if (lane == 0) {
            for (int s = 0; s < S; ++s) {
                mbar_init(full(s), 1);
                mbar_init(done(s), 1);
                mbar_init(wp_empty(s), 4);
            }
            for (int j = 0; j < U; ++j) mbar_init(a_full(j), 4);
            mbar_init(acc_full, 1);
            abort_flag[0] = 0;
            abort_flag[1] = 0;  // always-zero word for waits that must ignore the abort request
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        const uint32_t issue = elect_one();
        for (int it = 0; it < pre; ++it) issue_weights(ks_begin + it, it, issue);
    }
    pdl_launch_dependents();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool failed = false;
    pdl_wait();   // the activations, their sums and scales are read, and the output written, only from here on

    if (warp == 0) {
        // ---------------- TMA producer: the whole warp walks the loop, one elected lane issues
        const uint32_t issue = elect_one();
        for (int it = 0; it < pre; ++it) issue_tokens(ks_begin + it, it, issue);
        int s = pre == S ? 0 : pre;
        uint32_t ph = pre == S ? 1u : 0u;
        int it = pre;
        for (; it < my_steps; ++it) {
            const bool ok = mbar_wait(done(s), ph ^ 1u, abort_flag) && mbar_wait(wp_empty(s), ph ^ 1u, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
            issue_weights(ks_begin + it, s, issue);
            issue_tokens(ks_begin + it, s, issue);
            if (++s == S) { s = 0; ph ^= 1u; }
        }
        if (failed && issue) {
            // drain: give every armed stage a bounded chance to land before shared memory is reused or released
            for (int back = 0; back < S; ++back) {
                const int last = it - 1 - back;
                if (last >= 0) mbar_wait(full(last % S), static_cast<uint32_t>(last / S) & 1u, abort_flag + 1);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer: the whole warp walks the loop, one elected lane issues
        const uint32_t issue = elect_one();
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a.BN >> 3) << 17) |
                               (static_cast<uint32_t>(BM >> 4) << 24);
        int s = 0, j = 0;
        uint32_t jph = 0;
        for (int it = 0; it < my_steps; ++it) {
            // the unpack warps arrive on a_full(j) only after they saw full(s): this wait covers both operands
            if (!__all_sync(0xffffffffu, mbar_wait(a_full(j), jph, abort_flag))) { failed = true; break; }
            tc_fence_after();
            const uint32_t a_tmem = tmem_base + static_cast<uint32_t>(TMEM_A_COL + j * A_COLS);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint64_t bdesc = smem_desc_sw128(x_addr(s, h));
#pragma unroll
                for (int k = 0; k < BKH / 32; ++k)
                    tc_mma_i8_ts(tmem_base, a_tmem + 32u * h + 8u * k, bdesc + 2u * k, idesc, (it | h | k) != 0 ? 1u : 0u, issue);
            }
            tc_commit_if(done(s), issue);
            if (++s == S) s = 0;
            if (++j == U) { j = 0; jph ^= 1u; }
        }
        if (!failed) tc_commit_if(acc_full, issue);
    } else if (warp < 6) {
        // ---------------- unpack warps: thread = one tensor-memory lane = one weight row of the tile
        const int quad = warp & 3;                 // the lane quadrant this warp may write
        const int L = quad * 32 + lane;            // tensor-memory lane
        // Source row of the packed stage. Plain: row L. SwiGLU: the stage holds 64 gate rows then 64 up rows;
        // within each quadrant lanes 0-15 take gate rows and lanes 16-31 the up rows of the same 16 channels.
        const int src_row = a.swiglu ? (quad * 16 + (lane & 15) + ((lane >> 4) << 6)) : L;
        // 128-byte rows under the 128B TMA swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7).
        const int sw = src_row & 7;
        int s = 0, j = 0, sd = 0;
        uint32_t ph = 0, phd = 0;
        for (int it = 0; it < my_steps; ++it) {
            // weight tile j was last read by the MMAs of stage it - U, whose completion is that stage's done barrier
            bool ok = mbar_wait(full(s), ph, abort_flag);
            if (ok && it >= U) ok = mbar_wait(done(sd), phd, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
            tc_fence_after();
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint8_t* src = sm + s * stage_bytes + src_row * 128;
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
                mbar_arrive(a_full(j));
            }
            if (it >= U) {
                if (++sd == S) { sd = 0; phd ^= 1u; }
            }
            if (++s == S) { s = 0; ph ^= 1u; }
            if (++j == U) j = 0;
        }
    }

    // ---------------- reduce-scatter of the partial accumulators, then the epilogue: every warp takes part
    // Chunk c (tokens 16c .. 16c+15 of the tile) belongs to CTA c % ksplit, which keeps the partials of its chunk
    // number c / ksplit from source CTA r at  (r * own_max + c / ksplit) * CHUNK_BYTES, as four planes of
    // [128 rows][16 bytes] (plane q = tokens 4q .. 4q+3): thread = row, so a warp's accesses are contiguous.
    // The work of this part is a chain of short latencies per 16-token chunk (tensor-memory load, distributed
    // store; later shared-memory loads, a few conversions and multiplies, a staging store, a barrier, the global
    // store): measured at several hundred cycles per chunk and warp whatever the instruction mix, so it is spread
    // over as many warps as tensor memory's lane quadrants allow: three groups of four warps (warp % 4 = quadrant).
    const int chunks = a.BN >> 4;
    const int own_max = (chunks + ksplit - 1) / ksplit;
    const int quad = warp & 3, group = warp >> 2;   // warps 12, 13 (group 3) only keep the barriers company
    const int row = quad * 32 + lane;
    int2* tok = reinterpret_cast<int2*>(sm + OFF_TOK);
    if (static_cast<int>(threadIdx.x) < a.BN) {   // the tile's per-token constants
        const int m = m0 + static_cast<int>(threadIdx.x);
        tok[threadIdx.x] = m < a.M ? make_int2(__ldg(a.bias_sum + m) << 7, __float_as_int(__ldg(a.act_scales + m))) : make_int2(0, 0);
    }
    if (!failed && !mbar_wait(acc_full, 0u, abort_flag)) failed = true;
    if (failed) {
        *abort_flag = 1;
        atomicOr(a.status, SQAP_ERR_TIMEOUT);
    }
    failed = __syncthreads_or(failed ? 1 : 0) != 0;   // from here on the whole CTA agrees; tok is complete
    tc_fence_after();
    cluster_sync_all();   // #1: every CTA's MMAs are done (or given up): the rings are idle and may receive partials
    if (group < EPI_GROUPS && !failed) {
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        for (int c = group; c < chunks; c += EPI_GROUPS) {
            uint32_t v[16];
            tc_ld16(taddr + 16 * c, v);
            const uint32_t dst = map_to_cta(base + static_cast<uint32_t>(OFF_XCHG + (rank * own_max + c / ksplit) * CHUNK_BYTES + row * 16),
                                            static_cast<uint32_t>(c % ksplit));
            tc_wait_ld();
#pragma unroll
            for (int q = 0; q < 4; ++q) st_cluster_v4(dst + q * (BM * 16), v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        }
    }
    tc_fence_before();
    __syncwarp();
    cluster_sync_all();   // #2: all partials have arrived; nobody touches another CTA's shared memory from here on
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
    if (group < EPI_GROUPS && !failed) {
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
        const int own = (chunks - rank + ksplit - 1) / ksplit;   // chunks rank, rank + ksplit, ...
        const bool odd = (lane & 16) != 0;
        const int ch = a.swiglu ? quad * 16 + (lane & 15) : row, n_tile0 = a.swiglu ? n0 / 2 : n0;
        for (int lc = group, turn = 0; lc < own; lc += EPI_GROUPS, turn ^= 1) {
            const int c = lc * ksplit + rank;
            const int m_first = m0 + 16 * c;
            const int4* t4 = reinterpret_cast<const int4*>(tok + 16 * c);
            const uint8_t* part = sm + OFF_XCHG + lc * CHUNK_BYTES + row * 16;
            uint32_t v[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0;
            for (int r = 0; r < ksplit; ++r) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint4 p = *reinterpret_cast<const uint4*>(part + r * own_max * CHUNK_BYTES + q * (BM * 16));
                    v[4 * q] += p.x; v[4 * q + 1] += p.y; v[4 * q + 2] += p.z; v[4 * q + 3] += p.w;
                }
            }
            // fp16 / bf16: through shared memory, 16 bytes per thread to global memory; raw int32 (checking): directly
            uint8_t* stage = sm + OFF_STAGE + (group * 2 + turn) * EPI_STAGE_BYTES;
            if (a.swiglu) {
                if (a.out_dtype == SQAP_FP16) epilogue_chunk_coalesced<SQAP_FP16, true>(a, v, m_first, n_tile0, ch, sw, lane, t4, stage, row, 2 + group);
                else epilogue_chunk_coalesced<SQAP_BF16, true>(a, v, m_first, n_tile0, ch, sw, lane, t4, stage, row, 2 + group);
            } else {
                if (a.out_dtype == SQAP_FP16) epilogue_chunk_coalesced<SQAP_FP16, false>(a, v, m_first, n_tile0, ch, sw, lane, t4, stage, row, 2 + group);
                else if (a.out_dtype == SQAP_BF16) epilogue_chunk_coalesced<SQAP_BF16, false>(a, v, m_first, n_tile0, ch, sw, lane, t4, stage, row, 2 + group);
                else epilogue_chunk<SQAP_I32, false, 1>(a, v, m_first, n, n_ok, sw, lane, t4);
            }
            (void)odd;
        }
    }
}

// Resident CTAs the device offers a grid of clusters of `ksplit` CTAs of this kernel (index ksplit; 0 unused).
struct Slots {
    int cta[KSPLIT_MAX + 1];
};

}  // namespace tcsk

// Picks the token tiling and the K split for a shape: the split that minimises
//   rounds of clusters over the device  x  (stages per CTA x cycles per stage + a CTA's fixed cost)  + the exchange.
static void choose_split(int M, int n_tiles, int k_steps, const tcsk::Slots& slots, int forced, int* m_tiles, int* BN,
                         int* ksplit) {
    using namespace tcsk;
    *m_tiles = (M + BN_MAX - 1) / BN_MAX;
    *BN = ((M + *m_tiles - 1) / *m_tiles + 15) / 16 * 16;
    const long tiles = static_cast<long>(*m_tiles) * n_tiles;
    // cycles per 256-code stage: the unpack chain, or the MMAs where the tile is wide (4 cycles per token)
    const double stage = 4.0 * *BN > 750.0 ? 4.0 * *BN : 750.0;
    double best = -1.0;
    *ksplit = 1;
    for (int s = 1; s <= KSPLIT_MAX && s <= k_steps; ++s) {
        if (slots.cta[s] < s) continue;
        if (forced && s != forced) continue;
        const long rounds = (tiles * s + slots.cta[s] - 1) / slots.cta[s];
        const int per = (k_steps + s - 1) / s;
        const double cost = static_cast<double>(rounds) * (per * stage + 2500.0) + (s > 1 ? 600.0 + 200.0 * s : 0.0);
        if (best < 0 || cost < best) {
            best = cost;
            *ksplit = s;
        }
    }
}

sqap_status launch_linear_tcgen05_splitk(const LinearArgs& a, int forced_split, cudaStream_t s) {
    using namespace tcsk;
    if (forced_split < 0 || forced_split > KSPLIT_MAX) return SQAP_ERR_INVALID;
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
    k.out_dtype = a.out_dtype;
    k.status = device_status_word();
    if (!k.status) return SQAP_ERR_CUDA;

    // Once per device: the shared-memory limit, and how many CTAs can be resident for each cluster size (clusters
    // must fit inside one GPC, so the figure drops as the clusters grow).
    static PerDevice<Slots> setup;
    const Slots* slots = nullptr;
    const sqap_status st = setup.run(
        [](Slots* out) {
            const sqap_status s0 = set_max_dynamic_smem(w4a4_tc_splitk_kernel, SMEM_BYTES);
            if (s0 != SQAP_OK) return s0;
            const int sms = sm_count();
            out->cta[0] = 0;
            for (int c = 1; c <= KSPLIT_MAX; ++c) {
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(static_cast<unsigned>(sms / c * c));
                cfg.blockDim = dim3(THREADS);
                cfg.dynamicSmemBytes = SMEM_BYTES;
                cudaLaunchAttribute attr;
                attr.id = cudaLaunchAttributeClusterDimension;
                attr.val.clusterDim.x = static_cast<unsigned>(c);
                attr.val.clusterDim.y = 1;
                attr.val.clusterDim.z = 1;
                cfg.attrs = &attr;
                cfg.numAttrs = 1;
                int n = 0;
                if (cudaOccupancyMaxActiveClusters(&n, w4a4_tc_splitk_kernel, &cfg) != cudaSuccess || n <= 0) {
                    cudaGetLastError();
                    n = c == 1 ? sms : 0;   // unknown: do not use this cluster size
                }
                out->cta[c] = n * c;
            }
            return SQAP_OK;
        },
        &slots);
    if (st != SQAP_OK) return st;

    const int k_steps = (a.K + BK - 1) / BK;
    int ksplit = 1;
    choose_split(a.M, k.n_tiles, k_steps, *slots, forced_split, &k.m_tiles, &k.BN, &ksplit);
    if (forced_split && ksplit != forced_split) return SQAP_ERR_UNSUPPORTED;   // more slices than stages, or no such clusters
    k.stages = RING_BYTES / stage_bytes_for(k.BN);
    if (k.stages > S_MAX) k.stages = S_MAX;
    k.a_tiles = k.stages - 1 < U_MAX ? k.stages - 1 : U_MAX;    // >= 2: three stages fit at 192 tokens

    CUtensorMap tm_w, tm_u, tm_x;
    if (!weight_maps(a, k.swiglu != 0, BM, BK / 2, &tm_w, &tm_u)) return SQAP_ERR_CUDA;
    if (!make_map(&tm_x, a.x8, a.M, a.K, k.BN, BKH, CU_TENSOR_MAP_SWIZZLE_128B)) return SQAP_ERR_CUDA;

    const int tiles = k.m_tiles * k.n_tiles;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(tiles) * static_cast<unsigned>(ksplit));
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(ksplit);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see launch_dependent() in common.cuh
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, w4a4_tc_splitk_kernel, tm_w, tm_u, tm_x, k, ksplit);
    if (e != cudaSuccess) {
        note_cuda_error(e);
        cudaGetLastError();
        return SQAP_ERR_CUDA;
    }
    count_launch();
    return check_launch();
}

}  // namespace sqap

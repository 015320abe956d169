// Quantization-aware visual-token pruning: K_final = K_attn U K_ring U K_fps, then compaction.
//
// One CTA per observation decides the kept set (a few KB of scores; latency-bound, the FPS loop
// is m dependent steps), a second kernel copies the surviving rows (HBM-bound, 2 bytes read and
// 2 written per kept element).
#include "common.cuh"

namespace sqap {

constexpr int PRUNE_MAX_VISUAL = 1024;
constexpr uint32_t FPS_D_INIT = 0x1FFFFFu;  // above any squared distance on a <= 1024-wide grid

// CAND = visual tokens per lane of the FPS warp (token j lives in lane j % 32, slot j / 32).
template <int CAND>
__global__ void __launch_bounds__(512) prune_select_kernel(sqap_prune_params p, const void* __restrict__ scores,
                                                            const int32_t* __restrict__ ring_center,
                                                            int32_t* __restrict__ kept_idx,
                                                            int32_t* __restrict__ n_kept,
                                                            int32_t* __restrict__ row_index, int out_rows) {
    __shared__ float a[PRUNE_MAX_VISUAL];
    __shared__ uint8_t keep[PRUNE_MAX_VISUAL];  // bit 0: in K_attn U K_ring, bit 1: in K_fps
    __shared__ int warp_tot[32];
    __shared__ int s_union;
    const int b = blockIdx.x;
    const int nv = p.n_visual;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;

    // scores: a_j = sum over the R score rows, row 0 first, in fp32
    for (int j = tid; j < nv; j += blockDim.x) {
        float s;
        if (p.score_rows > 0) {
            const __half* A = static_cast<const __half*>(scores) + static_cast<int64_t>(b) * p.score_rows * nv;
            // batches of 8 loads in flight (the rows are nv apart: every load is a separate L2 access), summed in
            // row order
            s = __half2float(A[j]);
            int r = 1;
            for (; r + 8 <= p.score_rows; r += 8) {
                __half h[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) h[i] = A[static_cast<int64_t>(r + i) * nv + j];
#pragma unroll
                for (int i = 0; i < 8; ++i) s = __fadd_rn(s, __half2float(h[i]));
            }
            for (; r < p.score_rows; ++r) s = __fadd_rn(s, __half2float(A[static_cast<int64_t>(r) * nv + j]));
        } else {
            s = static_cast<const float*>(scores)[static_cast<int64_t>(b) * nv + j];
        }
        a[j] = s;
    }
    if (tid == 0) s_union = 0;
    __syncthreads();

    // Strategy 1 (Eq. 1): rank by counting under the order (score descending, index ascending).
    // Strategy 2 (Eq. 4): Chebyshev ball around the projected robot position.
    const bool ring_on = p.ring_radius >= 0 && ring_center != nullptr;
    const int cu = ring_on ? ring_center[2 * b] : 0, cv = ring_on ? ring_center[2 * b + 1] : 0;
    int local_union = 0;
    for (int j = tid; j < nv; j += blockDim.x) {
        const float aj = a[j];
        int rank = 0;
        for (int i = 0; i < nv; ++i) {
            const float ai = a[i];
            rank += (ai > aj) || (ai == aj && i < j);
        }
        bool in = rank < p.k_attn;
        if (ring_on) {
            const int du = abs(j % p.grid_w - cu), dv = abs(j / p.grid_w - cv);
            in |= max(du, dv) <= p.ring_radius;
        }
        keep[j] = in ? 1 : 0;
        local_union += in;
    }
    if (local_union) atomicAdd(&s_union, local_union);
    __syncthreads();

    // Strategy 3 (Eq. 5): farthest-point sampling by one warp. Each candidate keeps ONE word, key = D << 10 |
    // (1023 - j): the maximum key is the largest distance, lowest index on ties, and since the index bits of a
    // candidate never change, min over distances is min over keys, so a step is one min per candidate, one warp
    // max-reduction and no division (the picked token's coordinates come from a reciprocal multiply).
    // D = 0 marks "picked or never a candidate": such keys lose against every live candidate.
    const int m_fps = max(0, p.keep_total - s_union);
    if (warp == 0 && m_fps > 0) {
        uint32_t key[CAND];
        int tu[CAND], tv[CAND];
        // j / grid_w = umulhi(j, inv_w) for j < 2^16 and 2 <= grid_w; a one-token-wide grid (where the 32-bit
        // reciprocal would wrap to 0) has t_v = j, t_u = 0 directly
        const bool one_wide = p.grid_w == 1;
        const uint32_t inv_w = one_wide ? 0u : 0xFFFFFFFFu / static_cast<uint32_t>(p.grid_w) + 1u;
#pragma unroll
        for (int i = 0; i < CAND; ++i) {
            const int j = lane + 32 * i;
            const bool cand = j < nv && keep[j] == 0;
            key[i] = (cand ? (FPS_D_INIT << 10) : 0u) | static_cast<uint32_t>(1023 - (j & 1023));
            tv[i] = j / p.grid_w;
            tu[i] = j - tv[i] * p.grid_w;
        }
        for (int step = 0; step < m_fps; ++step) {
            uint32_t best = 0;
#pragma unroll
            for (int i = 0; i < CAND; ++i) best = max(best, key[i]);
            best = __reduce_max_sync(0xffffffffu, best);
            if ((best >> 10) == 0) break;  // remainder exhausted
            const int pj = 1023 - static_cast<int>(best & 1023u);
            const int pv = one_wide ? pj : static_cast<int>(__umulhi(static_cast<uint32_t>(pj), inv_w));
            const int pu = pj - pv * p.grid_w;
            if ((pj & 31) == lane) keep[pj] = 2;
#pragma unroll
            for (int i = 0; i < CAND; ++i) {
                const int du = tu[i] - pu, dv = tv[i] - pv;
                const uint32_t d2 = static_cast<uint32_t>(du * du + dv * dv);  // 0 exactly for the picked token
                key[i] = min(key[i], (d2 << 10) | (key[i] & 1023u));
            }
        }
    }
    __syncthreads();

    // Compaction: ascending row numbers of the kept rows (non-visual rows always kept).
    int32_t* out = kept_idx + static_cast<int64_t>(b) * p.rows;
    int base = 0;
    for (int r0 = 0; r0 < p.rows; r0 += blockDim.x) {
        const int r = r0 + tid;
        bool k = false;
        if (r < p.rows) {
            const int j = r - p.visual_start;
            k = (j < 0 || j >= nv) ? true : keep[j] != 0;
        }
        const uint32_t bal = __ballot_sync(0xffffffffu, k);
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < nwarps; ++w) {
            const int t = warp_tot[w];
            before += (w < warp) ? t : 0;
            total += t;
        }
        if (k) {
            const int pos = base + before + __popc(bal & ((1u << lane) - 1u));
            out[pos] = r;
            // the same list as source rows of the whole batch, for a quantizer that reads the kept rows in place
            if (row_index && pos < out_rows) row_index[static_cast<int64_t>(b) * out_rows + pos] = b * p.rows + r;
        }
        base += total;
        __syncthreads();
    }
    for (int r = base + tid; r < p.rows; r += blockDim.x) out[r] = -1;
    if (tid == 0) n_kept[b] = base;
    if (row_index) {
        // entries past n_kept repeat the observation's last kept row (its first row if nothing was kept), so that
        // every entry names a row that exists
        const int pad = b * p.rows + (base > 0 ? out[base - 1] : 0);   // written before the last __syncthreads
        for (int i = base + tid; i < out_rows; i += blockDim.x) row_index[static_cast<int64_t>(b) * out_rows + i] = pad;
    }
}

// Row copy: grid (out_rows, batch); CTA (i, b) copies row kept_idx[b][i] of observation b.
__global__ void __launch_bounds__(256) gather_rows_kernel(const __half* __restrict__ x, int64_t ldx, int rows, int K,
                                                          const int32_t* __restrict__ kept_idx,
                                                          const int32_t* __restrict__ n_kept, __half* __restrict__ out,
                                                          int64_t ldo, int out_rows) {
    const int i = blockIdx.x, b = blockIdx.y;
    if (i >= n_kept[b]) return;
    const int src = kept_idx[static_cast<int64_t>(b) * rows + i];
    if (src < 0 || src >= rows) return;
    const uint4* s = reinterpret_cast<const uint4*>(x + (static_cast<int64_t>(b) * rows + src) * ldx);
    uint4* d = reinterpret_cast<uint4*>(out + (static_cast<int64_t>(b) * out_rows + i) * ldo);
    for (int c = threadIdx.x; c < K / 8; c += blockDim.x) d[c] = __ldg(s + c);
}

// ---------------------------------------------------------------------------------------------
// Attention of one task-query token to the visual tokens, from a fused QKV projection output: the
// score rows the criterion above consumes. One CTA per (head, observation); thread = visual token.
// Every floating-point step is an explicitly rounded fp32 operation in a stated order (sqap.h), so
// the scores, and with them the kept set, do not depend on this kernel's thread mapping.
constexpr int ATTN_MAX_HEAD_DIM = 256;
constexpr int ATTN_TILE = 256;   // most tokens whose keys are staged in shared memory at a time

// 2^t for t <= 0: floor / fraction split, degree-9 Taylor polynomial of e^(f ln 2) in Horner form with
// separately rounded multiplies and adds, exact scaling by 2^floor(t); 0 below -126.
__device__ __forceinline__ float exp2_neg(float t) {
    constexpr float c[10] = {1.0f, 6.9314718056e-01f, 2.4022650696e-01f, 5.5504108665e-02f, 9.6181291076e-03f,
                             1.3333558146e-03f, 1.5403530393e-04f, 1.5252733804e-05f, 1.3215486790e-06f,
                             1.0178086009e-07f};
    if (t < -126.0f) return 0.0f;
    const float i = floorf(t);
    const float f = __fsub_rn(t, i);
    float p = c[9];
#pragma unroll
    for (int k = 8; k >= 0; --k) p = __fadd_rn(__fmul_rn(p, f), c[k]);
    return __int_as_float(__float_as_int(p) + (static_cast<int>(i) << 23));   // p in [1, 2], i >= -126: stays normal
}

__global__ void __launch_bounds__(256) attention_scores_kernel(const __half* __restrict__ qkv, int64_t ldq, int rows,
                                                               int query_row, int visual_start, int n_visual,
                                                               int head_dim, int q_col0, int k_col0, float inv_sqrt_d,
                                                               int tile_rows, __half* __restrict__ out) {
    __shared__ float qf[ATTN_MAX_HEAD_DIM];
    __shared__ float lg[PRUNE_MAX_VISUAL];
    __shared__ float red[32];
    __shared__ float s_sum;
    const int h = blockIdx.x, b = blockIdx.y, n_heads = gridDim.x;
    const __half* q = qkv + (static_cast<int64_t>(b) * rows + query_row) * ldq + q_col0 + static_cast<int64_t>(h) * head_dim;
    for (int d = threadIdx.x; d < head_dim; d += blockDim.x) qf[d] = __half2float(q[d]);
    __syncthreads();
    float m = -INFINITY;
    // A thread owns a token (its sum runs in d order, as defined), but a token's key row is only head_dim * 2 bytes of
    // a much longer row of the QKV output: read straight from global memory, the 32 lanes of a load would touch 32
    // separate rows. So the CTA first copies the keys of up to 256 tokens into shared memory with coalesced 16-byte
    // asynchronous copies (consecutive threads take consecutive chunks of a row), rows padded by 16 bytes so that the
    // row-per-thread reads that follow are free of bank conflicts.
    extern __shared__ __align__(16) uint8_t ktile[];
    const int cpr = head_dim / 8, row_stride = head_dim * 2 + 16;
    for (int j0 = 0; j0 < n_visual; j0 += tile_rows) {
        const int tile = min(tile_rows, n_visual - j0);
        const __half* kbase = qkv + (static_cast<int64_t>(b) * rows + visual_start + j0) * ldq + k_col0 + static_cast<int64_t>(h) * head_dim;
        for (int i = threadIdx.x; i < tile * cpr; i += blockDim.x) {
            const int r = i / cpr, c = i - r * cpr;
            const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(ktile + r * row_stride + 16 * c));
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(kbase + static_cast<int64_t>(r) * ldq + 8 * c) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        for (int jj = threadIdx.x; jj < tile; jj += blockDim.x) {
            const uint8_t* k = ktile + jj * row_stride;
            float acc = 0.0f;
            for (int d = 0; d < head_dim; d += 8) {
                const uint4 raw = *reinterpret_cast<const uint4*>(k + 2 * d);
                const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 kv = __half22float2(h2[i]);
                    acc = __fadd_rn(acc, __fmul_rn(qf[d + 2 * i], kv.x));
                    acc = __fadd_rn(acc, __fmul_rn(qf[d + 2 * i + 1], kv.y));
                }
            }
            const float l = __fmul_rn(acc, inv_sqrt_d);
            lg[j0 + jj] = l;
            m = fmaxf(m, l);
        }
        __syncthreads();   // the tile is read: the next one may overwrite it
    }
    // block max (exact, order-free)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    m = red[0];
    for (int i = 1; i < (blockDim.x >> 5); ++i) m = fmaxf(m, red[i]);
    for (int j = threadIdx.x; j < n_visual; j += blockDim.x) lg[j] = exp2_neg(__fmul_rn(__fsub_rn(lg[j], m), 1.44269504f));
    __syncthreads();
    if (threadIdx.x == 0) {   // the sum's order is part of the definition: j ascending
        float s = 0.0f;
        for (int j = 0; j < n_visual; ++j) s = __fadd_rn(s, lg[j]);
        s_sum = s;
    }
    __syncthreads();
    const float s = s_sum;
    __half* o = out + (static_cast<int64_t>(b) * n_heads + h) * n_visual;
    for (int j = threadIdx.x; j < n_visual; j += blockDim.x) o[j] = __float2half_rn(__fdiv_rn(lg[j], s));
}

}  // namespace sqap

extern "C" sqap_status sqap_attention_scores(const void* qkv, int64_t ldq, int batch, int rows, int query_row,
                                             int visual_start, int n_visual, int n_heads, int head_dim, int q_col0,
                                             int k_col0, void* scores_out, void* stream) {
    using namespace sqap;
    if (batch < 0 || rows <= 0 || query_row < 0 || query_row >= rows || visual_start < 0 || n_visual < 0 ||
        static_cast<int64_t>(visual_start) + n_visual > rows || n_heads <= 0 || head_dim <= 0 || q_col0 < 0 || k_col0 < 0)
        return SQAP_ERR_INVALID;
    if (static_cast<int64_t>(q_col0) + static_cast<int64_t>(n_heads) * head_dim > ldq ||
        static_cast<int64_t>(k_col0) + static_cast<int64_t>(n_heads) * head_dim > ldq)
        return SQAP_ERR_INVALID;
    if (n_visual > PRUNE_MAX_VISUAL || head_dim > ATTN_MAX_HEAD_DIM || batch > 65535) return SQAP_ERR_UNSUPPORTED;
    if (batch == 0 || n_visual == 0) return SQAP_OK;
    if (!qkv || !scores_out) return SQAP_ERR_INVALID;
    if (head_dim % 8 != 0 || ldq % 8 != 0 || k_col0 % 8 != 0 || !aligned16(qkv)) return SQAP_ERR_ALIGN;
    const float inv_sqrt_d = static_cast<float>(1.0 / sqrt(static_cast<double>(head_dim)));
    dim3 grid(n_heads, batch);
    // 256 tokens per tile when the grid fits the SMs three CTAs deep (one pass over a 16 x 16 patch grid); half that
    // otherwise, so that more CTAs are resident and the grid runs as one wave
    const int tile_rows = static_cast<int64_t>(n_heads) * batch <= 3 * sm_count() ? ATTN_TILE : ATTN_TILE / 2;
    const size_t smem = static_cast<size_t>(tile_rows) * (head_dim * 2 + 16);
    if (smem > 48 * 1024) {
        static PerDevice<int> setup;   // the limit covers the longest supported head
        const sqap_status st = setup.run([](int*) { return set_max_dynamic_smem(attention_scores_kernel, ATTN_TILE * (ATTN_MAX_HEAD_DIM * 2 + 16)); });
        if (st != SQAP_OK) return st;
    }
    attention_scores_kernel<<<grid, 256, smem, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __half*>(qkv), ldq, rows, query_row, visual_start, n_visual, head_dim, q_col0, k_col0, inv_sqrt_d,
        tile_rows, static_cast<__half*>(scores_out));
    count_launch();
    return check_launch();
}

namespace sqap {

static sqap_status prune_check(const sqap_prune_params* p, const void* scores, const int32_t* kept_idx, const int32_t* n_kept) {
    if (!p) return SQAP_ERR_INVALID;
    if (p->batch < 0 || p->rows < 0 || p->n_visual < 0 || p->visual_start < 0 ||
        static_cast<int64_t>(p->visual_start) + p->n_visual > p->rows)
        return SQAP_ERR_INVALID;
    if (p->k_attn < 0 || p->keep_total < 0 || p->score_rows < 0 || p->flags != 0) return SQAP_ERR_INVALID;
    if (p->n_visual > 0 && (p->grid_w <= 0 || p->grid_h <= 0 ||
                            static_cast<int64_t>(p->grid_w) * p->grid_h != p->n_visual))
        return SQAP_ERR_INVALID;
    if (p->n_visual > PRUNE_MAX_VISUAL) return SQAP_ERR_UNSUPPORTED;
    if (p->batch > 65535) return SQAP_ERR_UNSUPPORTED;
    if (p->batch == 0) return SQAP_OK;
    if (!kept_idx || !n_kept || (p->n_visual > 0 && !scores)) return SQAP_ERR_INVALID;
    return SQAP_OK;
}

static sqap_status launch_select(const sqap_prune_params* p, const void* scores, const int32_t* ring_center,
                                 int32_t* kept_idx, int32_t* n_kept, int32_t* row_index, int out_rows, cudaStream_t s) {
    sqap_prune_params q = *p;
    if (q.n_visual == 0) q.grid_w = q.grid_h = 1;
    int threads = (q.n_visual + 31) / 32 * 32;
    if (threads < 128) threads = 128;
    if (threads > 512) threads = 512;
    if (q.n_visual <= 256)
        prune_select_kernel<8><<<q.batch, threads, 0, s>>>(q, scores, ring_center, kept_idx, n_kept, row_index, out_rows);
    else
        prune_select_kernel<32><<<q.batch, threads, 0, s>>>(q, scores, ring_center, kept_idx, n_kept, row_index, out_rows);
    count_launch();
    return check_launch();
}

}  // namespace sqap

extern "C" sqap_status sqap_prune_select(const sqap_prune_params* p, const void* scores, const int32_t* ring_center,
                                         int out_rows, int32_t* kept_idx, int32_t* n_kept, int32_t* row_index,
                                         void* stream) {
    using namespace sqap;
    const sqap_status st = prune_check(p, scores, kept_idx, n_kept);
    if (st != SQAP_OK || p->batch == 0) return st;
    if (out_rows < 0 || (out_rows > 0 && !row_index)) return SQAP_ERR_INVALID;
    if (static_cast<int64_t>(p->batch) * p->rows > 0x7FFFFFFFll) return SQAP_ERR_UNSUPPORTED;   // row numbers are int32
    return launch_select(p, scores, ring_center, kept_idx, n_kept, out_rows > 0 ? row_index : nullptr, out_rows,
                         static_cast<cudaStream_t>(stream));
}

extern "C" sqap_status sqap_prune_tokens(const sqap_prune_params* p, const void* scores, const int32_t* ring_center,
                                         const void* x, int64_t ldx, int K, void* x_out, int64_t ldo, int out_rows,
                                         int32_t* kept_idx, int32_t* n_kept, void* stream) {
    using namespace sqap;
    sqap_status st = prune_check(p, scores, kept_idx, n_kept);
    if (st != SQAP_OK || p->batch == 0) return st;
    if (x) {
        if (!x_out || K <= 0 || ldx < K || ldo < K || out_rows < 0) return SQAP_ERR_INVALID;
        if (K % 8 != 0 || ldx % 8 != 0 || ldo % 8 != 0 || !aligned16(x) || !aligned16(x_out)) return SQAP_ERR_ALIGN;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = launch_select(p, scores, ring_center, kept_idx, n_kept, nullptr, 0, s);
    if (st != SQAP_OK) return st;
    if (x && out_rows > 0) {
        dim3 grid(out_rows, p->batch);
        gather_rows_kernel<<<grid, 256, 0, s>>>(static_cast<const __half*>(x), ldx, p->rows, K, kept_idx, n_kept,
                                                static_cast<__half*>(x_out), ldo, out_rows);
        count_launch();
        st = check_launch();
    }
    return st;
}

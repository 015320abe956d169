/*
 * sqap.h — C ABI of the SQAP-VLA hot path for NVIDIA B200 (sm_100a).
 *
 * The path is the part of a W4A4 vision-language-action model that the paper speeds up:
 * the 4-bit-weight / 4-bit-activation linear layers of the language backbone, run on a
 * visual-token set reduced by the paper's quantization-aware pruning criterion
 * (K_final = K_attn U K_ring U K_fps).
 *
 * General rules for every call
 *   - "device" pointers are CUDA device pointers owned by the CALLER; the library never
 *     frees or keeps them. "host" pointers are ordinary host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Calls
 *     validate their arguments on the host, enqueue work on `stream` and return without
 *     synchronising, unless stated otherwise.
 *   - Sizes are `int`, row strides `int64_t`, both counted in ELEMENTS of the array's type.
 *   - Return value is a sqap_status; nothing throws, aborts or prints. Nothing runs on the CPU
 *     in place of a kernel: without a usable sm_100 device the compute calls fail.
 *   - Inputs must be finite. Non-finite activations or scores give unspecified codes /
 *     indices, never a fault.
 */
#ifndef SQAP_H
#define SQAP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SQAP_OK = 0,
    SQAP_ERR_INVALID = 1,     /* null pointer, negative or inconsistent size */
    SQAP_ERR_RANGE = 2,       /* weight code outside [-8,7]; scale not finite or <= 0 */
    SQAP_ERR_ALIGN = 3,       /* pointer or stride not 16-byte aligned; K not a multiple of 32 */
    SQAP_ERR_UNSUPPORTED = 4, /* e.g. rotation with K not a power of two; n_visual > 1024 */
    SQAP_ERR_NOMEM = 5,       /* device allocation failed, or workspace too small */
    SQAP_ERR_CUDA = 6,        /* a CUDA call failed; see sqap_last_cuda_error() */
    SQAP_ERR_TIMEOUT = 7,     /* a bounded wait inside a kernel ran out (reported by sqap_device_status) */
    SQAP_ERR_TOO_LARGE = 8    /* the problem does not fit a fixed-size resource (sqap_w4a4_linear_static) */
} sqap_status;

/* Output element types of sqap_w4a4_linear. */
#define SQAP_FP16 0
#define SQAP_BF16 1
#define SQAP_I32 2 /* raw int32 accumulators (checking only; SwiGLU not allowed) */

/* Flags of sqap_quantize_act. */
#define SQAP_Q_ROTATE 1u /* apply the orthonormal Hadamard rotation to each row first (Eq. 6) */
#define SQAP_Q_PER_TENSOR 2u /* sqap_quantize_act_ex: one scale for the whole tensor ("tensor-wise quantization") */

/* Flags of sqap_pack_weights. */
#define SQAP_W_ROTATED 1u /* bookkeeping only: the codes are those of W·H^T (Eq. 6, weight side) */

/* Flags of sqap_w4a4_linear (0 = let the library choose the kernel). */
#define SQAP_L_FORCE_SIMT 1u    /* the plain CUDA-core kernel */
#define SQAP_L_FORCE_TCGEN05 2u /* the tcgen05 tensor-core kernel (needs K % 128 == 0) */
#define SQAP_L_FORCE_GEMV 4u    /* the weight-streaming kernel for very few rows (M <= 8) */
#define SQAP_L_FORCE_TCGEN05_TS 16u /* the tcgen05 kernel that keeps the unpacked weights in tensor memory
                                       (needs K % 128 == 0) */
#define SQAP_L_FORCE_TCGEN05_PAIR 32u /* the same on CTA pairs (tcgen05 cta_group::2) */
#define SQAP_L_FORCE_MMA 64u /* the register-MMA weight streamer for a handful of rows (M <= 32, K % 128 == 0) */
#define SQAP_L_FORCE_TCGEN05_SPLITK 128u /* the tcgen05 kernel that splits K over the CTAs of a cluster (needs
                                            K % 128 == 0); SQAP_L_KSPLIT(n), n = 1..4, also fixes the cluster size */
#define SQAP_L_KSPLIT(n) ((uint32_t)(n) << 8)
#define SQAP_L_KSPLIT_MASK 0x700u
#define SQAP_L_FORCE_MASK                                                                                          \
    (SQAP_L_FORCE_SIMT | SQAP_L_FORCE_TCGEN05 | SQAP_L_FORCE_GEMV | SQAP_L_FORCE_TCGEN05_TS | SQAP_L_FORCE_TCGEN05_PAIR | \
     SQAP_L_FORCE_MMA | SQAP_L_FORCE_TCGEN05_SPLITK)
#define SQAP_L_REUSE_EXPANDED 8u /* the workspace still holds the expanded form of these same M x K activations
                                    from the previous call that used it (one activation feeding several weight
                                    matrices): skip the expand pass */

/* Opaque packed weight matrix; owned by the LIBRARY, released by sqap_free_weights. Immutable
 * after creation and usable from any stream once the creating stream has reached the pack. */
typedef struct sqap_weights sqap_weights;

/*
 * Offline weight side of W4A4 ("4-bit weights", introduction; Eq. 6 for rotated layers):
 * takes INT4 codes [N rows = output channels][K] (row-major, one int8 per code, values -8..7)
 * and one fp16 scale per output channel (bits as uint16, finite, > 0) and stores them in the
 * library's private nibble-packed device layout (N*K/2 bytes + 2N bytes of scales). `codes` and `scales_fp16` may each be host or device memory. The call allocates
 * device memory, synchronises `stream` before returning (it validates the codes), and writes the
 * handle to *out. Errors: INVALID (null, N <= 0, K <= 0), ALIGN (K % 32), RANGE, NOMEM, CUDA.
 */
sqap_status sqap_pack_weights(const int8_t* codes, const uint16_t* scales_fp16, int N, int K, uint32_t flags,
                              void* stream, sqap_weights** out);

/*
 * Offline weight quantizer ("4-bit weights", per-output-channel symmetric round-to-nearest; with
 * SQAP_Q_ROTATE the weight side of Eq. 6: the codes are those of W H^T, H = Sylvester-Hadamard / sqrt(K),
 * to be multiplied with activations quantized with SQAP_Q_ROTATE). For every output channel n:
 *   v = fp32(W[n])  [channel_mul: v[k] *= channel_mul[k]]  [rotated: H v] ; amax = max|v|
 *   scale = fp16(amax / 7)  (fp16(1) for an all-zero row; the smallest positive fp16 if that underflows)
 *   code  = clamp(round_half_even(v / fp32(scale)), -8, 7)
 * w_fp16: device fp16 [N rows, ldw elements apart]; channel_mul: device fp32 [K] or NULL (the reciprocal of the
 * activation side's per-channel multiplier, see sqap_quantize_act_ex); codes_out: device int8 [N*K];
 * scales_out_fp16: device [N].
 * K % 32 == 0, K <= 32768; rotation needs K a power of two >= 64. The outputs are what sqap_pack_weights takes
 * (pass SQAP_W_ROTATED there for rotated weights). Weights whose amax / 7 exceeds the fp16 range give an
 * infinite scale, which sqap_pack_weights rejects (SQAP_ERR_RANGE). Enqueues on `stream`, does not synchronise.
 */
sqap_status sqap_quantize_weights(const void* w_fp16, int N, int K, int64_t ldw, uint32_t flags, const float* channel_mul,
                                  int8_t* codes_out, uint16_t* scales_out_fp16, void* stream);

/* Releases a handle (NULL is accepted). Synchronises the device. */
sqap_status sqap_free_weights(sqap_weights* w);

/* Shape and flags of a handle. */
sqap_status sqap_weights_info(const sqap_weights* w, int* N, int* K, uint32_t* flags);

/* Inverse of the packing, for checking: writes the original codes [N*K] and scale bits [N] to
 * HOST memory. Synchronises. */
sqap_status sqap_unpack_weights(const sqap_weights* w, int8_t* codes_out_host, uint16_t* scales_out_host);

/*
 * Online activation side of W4A4 ("4-bit activations"; Section "Pruning-Targeted Quantizer
 * Enhancement"): per-token symmetric INT4 quantization of fp16 rows.
 *   v = fp32(x[row])                    ; with SQAP_Q_ROTATE: v = H v, H = Sylvester-Hadamard / sqrt(K)
 *   amax = max|v| ; scale = amax / 7 (1 if the row is all zero) ; inv = 7 / amax
 *   q = clamp(round_half_even(v * inv), -8, 7)
 * x: device fp16, row i starts at x + src*ldx with src = row_index ? row_index[i] : i.
 * row_index: device int32 [M] or NULL. K % 32 == 0; ROTATE needs K a power of two, 64 <= K <= 16384.
 * q_packed: device [M][K/2] bytes, PUBLIC layout: byte j of a row = (q[2j] & 15) | (q[2j+1] & 15) << 4
 * (two's-complement nibbles). scales: device fp32 [M]. M = 0 is a no-op.
 * x, q_packed 16-byte aligned; ldx % 8 == 0.
 */
sqap_status sqap_quantize_act(const void* x, int M, int K, int64_t ldx, const int32_t* row_index, uint32_t flags,
                              uint8_t* q_packed, float* scales, void* stream);

/*
 * The activation quantizer in the other granularities the paper names (Sections 2.2, 3, 3.3):
 *   SQAP_Q_PER_TENSOR  "tensor-wise": amax is taken over all M rows; every scales[i] receives the one scale, so
 *                      sqap_w4a4_linear is used unchanged
 *   channel_mul != NULL  "channel-wise", read as a static per-input-channel multiplier (device fp32 [K]) applied to
 *                      fp32(x) before the rotation and the max-abs (smoothing); put its reciprocal into the weights
 *                      with sqap_quantize_weights
 * Everything else (arguments, layout, rounding, SQAP_Q_ROTATE) is as in sqap_quantize_act, to which the call
 * falls through when neither extension is requested. channel_mul is 16-byte aligned. Both forms run in the
 * per-token quantizer's kernels; the tensor-wise form takes two launches (max-abs of the tensor, then the codes; x is
 * read twice) and keeps the max-abs between them in a word of a 64-slot pool owned by the library, cleared on
 * `stream`: up to 64 such calls may be in flight on different streams at once.
 */
sqap_status sqap_quantize_act_ex(const void* x, int M, int K, int64_t ldx, const int32_t* row_index, uint32_t flags,
                                 const float* channel_mul, uint8_t* q_packed, float* scales, void* stream);

/* Bytes of caller-provided scratch that sqap_w4a4_linear needs for M rows against a K-column
 * weight matrix (independent of N). Always a multiple of 256. */
size_t sqap_workspace_bytes(int M, int N, int K, uint32_t flags);

/*
 * The W4A4 linear (Q = W_q^T X on integer codes, then dequantisation):
 *   acc[m][n] = sum_k q[m][k] * w[n][k]                       exact int32
 *   out[m][n] = round( (float(acc) * act_scales[m]) * float(w_scale[n]) )       fp16 or bf16
 * With w_up != NULL (the gated MLP; w = gate projection, same N and K):
 *   g, u as above in fp32 from w and w_up;  out = round( g / (1 + exp(-g)) * u )
 * q_packed / act_scales: device, as written by sqap_quantize_act (K = the handle's K).
 * out: device [M rows, ldo elements apart] of out_dtype; 16-byte aligned, ldo*elemsize % 16 == 0.
 * workspace: device scratch of at least sqap_workspace_bytes(M, N, K, flags) bytes, 256-byte
 * aligned; its contents are undefined afterwards; two calls in flight at once need two workspaces.
 * flags: SQAP_L_* or 0 (at most one FORCE flag). Errors: INVALID, ALIGN, UNSUPPORTED (forced kernel cannot run the shape),
 * NOMEM (workspace too small), CUDA.
 */
sqap_status sqap_w4a4_linear(const uint8_t* q_packed, const float* act_scales, int M, const sqap_weights* w,
                             const sqap_weights* w_up, void* out, int64_t ldo, int out_dtype, uint32_t flags,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * Quantizer and linear as one call: what a W4A4 layer does with an fp16 activation ("4-bit activations" then
 * Q = W_q^T X, Section 3.3; Eq. 6 when SQAP_Q_ROTATE is set). The result is exactly that of
 *   sqap_quantize_act(x, M, K = w's K, ldx, row_index, qflags, q, s) ; sqap_w4a4_linear(q, s, M, w, w_up, out, ...)
 * but the codes go straight from the quantizer's registers into the form the GEMM reads, so the nibble-packed
 * intermediate is never written or re-read (3 bytes of HBM traffic per activation element instead of 4, one
 * launch fewer). Arguments as in those two calls; lflags may hold a SQAP_L_FORCE_* flag (REUSE_EXPANDED is
 * rejected). workspace: device scratch of at least sqap_quantize_linear_workspace_bytes(M, N, K) bytes,
 * 256-byte aligned; afterwards it holds the expanded codes of these activations, so further weight matrices
 * that take the SAME activations can follow with sqap_w4a4_linear(..., SQAP_L_REUSE_EXPANDED, workspace, ...)
 * and act_scales = (const float*)((char*)workspace + sqap_workspace_bytes(M, N, K, 0)).
 * Errors: those of the two calls.
 */
size_t sqap_quantize_linear_workspace_bytes(int M, int N, int K);
sqap_status sqap_quantize_linear(const void* x, int M, int64_t ldx, const int32_t* row_index, uint32_t qflags,
                                 const sqap_weights* w, const sqap_weights* w_up, void* out, int64_t ldo,
                                 int out_dtype, uint32_t lflags, void* workspace, size_t workspace_bytes,
                                 void* stream);

/*
 * The same linear for callers that must not allocate. (The paper has no counterpart: this entry point
 * exists only for the sake of such callers.)
 *
 * Who needs it: code that runs where device allocation is forbidden or would be harmful — a real-time
 * control loop that may not touch the allocator between robot actions, a process whose device memory
 * has all been handed to another component's pool, a host runtime that gives the library a fixed memory
 * budget and nothing more. Those callers
 * cannot size and cudaMalloc the workspace that sqap_w4a4_linear asks for, so here the scratch is an
 * array of SQAP_STATIC_WORKSPACE_BYTES bytes built into the library image (every GPU that loads the
 * library holds that much until the process exits). Inputs and outputs are still the caller's.
 *
 * Semantics, results and argument rules are exactly those of sqap_w4a4_linear; the differences:
 *   - no workspace arguments, and SQAP_L_REUSE_EXPANDED is rejected (INVALID);
 *   - the problem must satisfy sqap_workspace_bytes(M, N, K, flags) <= SQAP_STATIC_WORKSPACE_BYTES
 *     (about M * K <= 4 Mi, e.g. 288 rows at K = 11008 or 1020 rows at K = 4096); anything larger
 *     returns SQAP_ERR_TOO_LARGE and launches nothing;
 *   - the call itself calls no cudaMalloc / cudaFree and no allocating library routine;
 *   - the FIRST call on each device looks up the array's device address (a one-time query, with that
 *     device current); make that first call during set-up, before any stream capture begins;
 *   - all calls on a device share the one array, which simply keeps what the last call left in it (no
 *     part of it has to be cleared: each call rewrites everything it reads). Two calls whose kernels can
 *     overlap on the GPU — different streams, no dependency between them — race on it; serialise them.
 */
#define SQAP_STATIC_WORKSPACE_BYTES (4 * 1024 * 1024 + 8192)
sqap_status sqap_w4a4_linear_static(const uint8_t* q_packed, const float* act_scales, int M, const sqap_weights* w,
                                    const sqap_weights* w_up, void* out, int64_t ldo, int out_dtype, uint32_t flags,
                                    void* stream);

/*
 * Parameters of the pruning criterion (Section "Quantization-aware Pruning Strategies").
 * An observation is `rows` consecutive token rows; rows [visual_start, visual_start + n_visual)
 * are the visual tokens, laid out row-major on a grid_w x grid_h token grid
 * (token j has t_u = j % grid_w, t_v = j / grid_w); all other rows are never pruned.
 */
typedef struct {
    int batch;        /* observations */
    int rows;         /* token rows per observation */
    int visual_start; /* first visual row */
    int n_visual;     /* N_v = grid_w * grid_h, at most 1024 */
    int grid_w, grid_h;
    int score_rows;  /* R > 0: scores are fp16 [batch][R][n_visual], summed over R in fp32, row 0 first;
                        R = 0: scores are fp32 [batch][n_visual] */
    int k_attn;      /* |K_attn|: tokens kept for their score (Eq. 1); ties -> lower index */
    int keep_total;  /* visual tokens to keep in all; FPS fills keep_total - |K_attn U K_ring| */
    int ring_radius; /* R_t of Eq. 4; < 0: no ring */
    uint32_t flags;  /* 0 */
} sqap_prune_params;

/*
 * Quantization-aware visual-token pruning and compaction.
 *   K_attn = the k_attn highest-scoring visual tokens                                  (Eq. 1)
 *   K_ring = tokens within Chebyshev distance ring_radius of ring_center                (Eq. 4)
 *   K_fps  = farthest-point sampling of the quota's remainder from the other tokens     (Eq. 5)
 *            (squared Euclidean grid distance; first pick = lowest remaining index; ties -> lower index)
 *   kept rows = all non-visual rows + visual_start + j for j in K_attn U K_ring U K_fps, ascending.
 * scores: device (see score_rows). ring_center: device int32 [batch][2] = (t_u, t_v), may lie off the
 * grid; NULL or ring_radius < 0 disables the ring. x: device fp16 [batch*rows rows, ldx apart], or NULL
 * for indices only; x_out: device fp16, observation b's kept rows are written contiguously starting at
 * row b*out_rows (ldo apart), in ascending original order — the caller guarantees n_kept <= out_rows
 * (rows beyond out_rows are dropped, never written). kept_idx: device int32 [batch][rows], first
 * n_kept[b] entries valid (row numbers within the observation), the rest -1. n_kept: device int32 [batch].
 * K % 8 == 0; x, x_out 16-byte aligned; ldx, ldo % 8 == 0.
 */
sqap_status sqap_prune_tokens(const sqap_prune_params* p, const void* scores, const int32_t* ring_center,
                              const void* x, int64_t ldx, int K, void* x_out, int64_t ldo, int out_rows,
                              int32_t* kept_idx, int32_t* n_kept, void* stream);

/*
 * The same criterion and compaction without the row copy (the paper only needs the reduced sequence to reach the next
 * layer; Section 4.3's speed-up is end to end, so a pass over the activations that can be avoided is avoided):
 * besides kept_idx / n_kept as above, writes the kept rows as SOURCE ROW NUMBERS of the whole batch,
 *   row_index[b*out_rows + i] = b*rows + kept_idx[b][i]      for i < min(n_kept[b], out_rows),
 * which sqap_quantize_act / sqap_quantize_linear take as their `row_index` with M = batch*out_rows: the first linear
 * after the pruning then reads the surviving rows where they are. Entries from n_kept[b] on (only when fewer rows
 * were kept than out_rows) repeat the observation's last kept row, so every entry names an existing row.
 * row_index: device int32 [batch*out_rows]; batch*rows must fit int32. Errors: as sqap_prune_tokens.
 */
sqap_status sqap_prune_select(const sqap_prune_params* p, const void* scores, const int32_t* ring_center, int out_rows,
                              int32_t* kept_idx, int32_t* n_kept, int32_t* row_index, void* stream);

/*
 * Attention scores of one task-query token over the visual tokens (strategy 1 of Section "Quantization-aware
 * Pruning Strategies" scores the visual tokens by the attention of a task-query token), computed from the fp16
 * output of a fused QKV projection. For observation b, head h and visual token j:
 *   l_j = ( sum_d fp32(q[d]) * fp32(k_j[d]) ) * fp32(1/sqrt(head_dim))     fp32 products and sums, d ascending
 *   e_j = 2^((l_j - max_j l_j) * 1.44269504f)     2^t = P(t - floor t) * 2^floor(t), P the degree-9 Taylor polynomial
 *                                                 of e^(f ln 2) in Horner form, fp32, unfused; 0 for t < -126
 *   a_j = fp16( e_j / sum_j e_j )                 sum over j ascending, fp32 division
 * i.e. a softmax over the visual tokens only. q = row query_row of the observation, columns q_col0 + h*head_dim ...;
 * k_j = row visual_start + j, columns k_col0 + h*head_dim ... . qkv: device fp16 [batch*rows rows, ldq apart].
 * scores_out: device fp16 [batch][n_heads][n_visual] — exactly the `scores` input of sqap_prune_tokens with
 * score_rows = n_heads. Every step is an individually rounded fp32 operation in the stated order, so the result is
 * bit-reproducible. head_dim % 8 == 0, head_dim <= 256, n_visual <= 1024, ldq % 8 == 0, k_col0 % 8 == 0, qkv
 * 16-byte aligned.
 */
sqap_status sqap_attention_scores(const void* qkv, int64_t ldq, int batch, int rows, int query_row, int visual_start,
                                  int n_visual, int n_heads, int head_dim, int q_col0, int k_col0, void* scores_out,
                                  void* stream);

/*
 * Host helper (no GPU): robot-aware protection, Eq. 2-3. Projects the world point xyz through the
 * intrinsics Kmat (3x3 row-major) and extrinsics Rt = [R|t] (3x4 row-major) and maps the pixel to
 * token coordinates with the patch size (patch_w, patch_h), in double precision:
 * t_u = floor(u / patch_w), t_v = floor(v / patch_h). *in_front = 0 when the point is not in front
 * of the camera (lambda <= 0); the coordinates are then 0 and no ring should be used.
 */
sqap_status sqap_project_center(const double Kmat[9], const double Rt[12], const double xyz[3], double patch_w,
                                double patch_h, int32_t out_tu_tv[2], int* in_front);

/* Synchronises `stream`, then returns and clears the status word that kernels on the current
 * device set when one of their bounded waits runs out (SQAP_ERR_TIMEOUT) — SQAP_OK otherwise. */
sqap_status sqap_device_status(void* stream);

/*
 * Self-test of the bounded waits (the paper has no counterpart; this is the library's own failure-detection
 * mechanism). Every wait on a barrier inside the tensor-core kernels gives up after a fixed number of clocks,
 * records SQAP_ERR_TIMEOUT in the device status word, drains and returns. This call launches one warp that runs that
 * same wait, with the limit `limit_clocks` (1e3 .. 2e8 SM clocks, i.e. at most about 0.1 s), on a barrier nothing
 * will ever arrive on. Afterwards sqap_device_status(stream) must return SQAP_ERR_TIMEOUT once and SQAP_OK on the next
 * call, and the device stays fully usable. Touches no caller memory. Errors: INVALID (limit out of range),
 * UNSUPPORTED (not an sm_100 device), CUDA.
 */
sqap_status sqap_selftest_bounded_wait(int64_t limit_clocks, void* stream);

/* cudaError_t of the most recent failing CUDA call on this thread (0 if none). */
int sqap_last_cuda_error(void);

const char* sqap_status_string(sqap_status s);

/* Number of kernels this library has launched in this process (all threads). */
int64_t sqap_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SQAP_H */

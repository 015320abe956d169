/*
 * CPU oracle for the SQAP-VLA hot path (W4A4 linears on a pruned visual-token set).
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain restatement of what the path
 * computes, written from the paper's text; the parity tests, the smoke check and the
 * bench's cpu_baseline leg are its only callers. It shares no code with the CUDA library
 * and the library never calls it.
 *
 * Conventions: scalar loops in the order the method states them; fp32 where the method's
 * arithmetic is fp32 (compiled with -ffp-contract=off so no multiply-add is fused), exact
 * integers elsewhere, fp64 for the SiLU gate and the camera projection. OpenMP is used only
 * across rows / output rows, which are independent, so threading cannot change a result.
 *
 * Parity with the authors' own implementation is unpinned for: the activation quantizer's
 * rounding/scale convention, the Hadamard stage order, the choices of k, R_t, the FPS seed
 * point and tie rules (the paper prints none of them). Every function below is pinned in
 * the CPU test-suite against closed forms, brute force, invariants or library routines.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <limits.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------------------------------------------------------------- fp16 / bf16 bit helpers */

/* IEEE binary16 bits -> binary32 value (exact). */
static float half_bits_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t exp = (h >> 10) & 0x1Fu;
    uint32_t man = h & 0x3FFu;
    uint32_t bits;
    if (exp == 0) {
        if (man == 0) {
            bits = sign;
        } else { /* subnormal: value = man * 2^-24 */
            float f = (float)man * 0x1p-24f;
            memcpy(&bits, &f, 4);
            bits |= sign;
        }
    } else if (exp == 31) {
        bits = sign | 0x7F800000u | (man << 13);
    } else {
        bits = sign | ((exp + 112u) << 23) | (man << 13);
    }
    float out;
    memcpy(&out, &bits, 4);
    return out;
}

/* binary32 -> binary16 bits, round to nearest, ties to even; overflow -> inf. */
static uint16_t float_to_half_bits(float f)
{
    uint32_t x;
    memcpy(&x, &f, 4);
    uint32_t sign = (x >> 16) & 0x8000u;
    uint32_t absx = x & 0x7FFFFFFFu;
    if (absx >= 0x7F800000u) { /* inf / nan */
        return (uint16_t)(sign | 0x7C00u | ((absx > 0x7F800000u) ? 0x200u : 0u));
    }
    if (absx >= 0x47800000u) { /* >= 65536 -> certainly inf (65520 rounds to inf too, handled below) */
        return (uint16_t)(sign | 0x7C00u);
    }
    if (absx < 0x33000000u) { /* < 2^-25 -> rounds to zero (2^-25 itself ties to even = 0) */
        return (uint16_t)sign;
    }
    int32_t e = (int32_t)(absx >> 23) - 127; /* unbiased exponent */
    uint32_t m = (absx & 0x7FFFFFu) | 0x800000u; /* 24-bit significand */
    uint32_t shift;                           /* bits to drop */
    uint32_t base;                            /* half bits before adding the kept significand */
    if (e < -14) {                            /* half subnormal: unit = 2^-24 */
        shift = (uint32_t)(13 + (-14 - e));
        base = 0;
        /* kept = m >> shift, including the (former) implicit bit */
        uint32_t kept = m >> shift;
        uint32_t rem = m & ((1u << shift) - 1u);
        uint32_t halfway = 1u << (shift - 1);
        if (rem > halfway || (rem == halfway && (kept & 1u))) kept++;
        return (uint16_t)(sign | (base + kept));
    }
    shift = 13;
    base = (uint32_t)(e + 15) << 10;
    uint32_t kept = (m >> shift) & 0x3FFu;
    uint32_t rem = m & 0x1FFFu;
    uint32_t hb = base | kept;
    if (rem > 0x1000u || (rem == 0x1000u && (hb & 1u))) hb++; /* carry may roll into exponent / inf: correct */
    return (uint16_t)(sign | hb);
}

/* binary32 -> bfloat16 bits, round to nearest even. */
static uint16_t float_to_bf16_bits(float f)
{
    uint32_t x;
    memcpy(&x, &f, 4);
    if ((x & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((x >> 16) | 0x40u);
    uint32_t lsb = (x >> 16) & 1u;
    x += 0x7FFFu + lsb;
    return (uint16_t)(x >> 16);
}

void oracle_half_to_float(const uint16_t *h, int64_t n, float *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = half_bits_to_float(h[i]);
}

void oracle_float_to_half(const float *f, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = float_to_half_bits(f[i]);
}

void oracle_float_to_bf16(const float *f, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = float_to_bf16_bits(f[i]);
}

/* ---------------------------------------------------------------- Hadamard rotation (Eq. 6) */

/*
 * In-place fast Walsh-Hadamard transform of one fp32 row, Sylvester order, unnormalised.
 * Stages h = 1, 2, 4, ..., K/2; in stage h every pair (j, j+h) with bit h of j clear becomes
 * (a+b, a-b). Each output of a stage is one fp32 add of two fixed inputs, so the result is
 * defined bit for bit by the stage order alone.
 */
void oracle_fwht_f32(float *v, int K)
{
    for (int h = 1; h < K; h <<= 1) {
        for (int i = 0; i < K; i += 2 * h) {
            for (int j = i; j < i + h; ++j) {
                float a = v[j];
                float b = v[j + h];
                v[j] = a + b;
                v[j + h] = a - b;
            }
        }
    }
}

/* Same transform in fp64, used by the Eq. 6 identity checks. */
void oracle_fwht_f64(double *v, int K)
{
    for (int h = 1; h < K; h <<= 1)
        for (int i = 0; i < K; i += 2 * h)
            for (int j = i; j < i + h; ++j) {
                double a = v[j], b = v[j + h];
                v[j] = a + b;
                v[j + h] = a - b;
            }
}

/* Normalisation that makes H orthonormal (H^T H = I, the property Eq. 6 relies on). */
float oracle_hadamard_norm(int K) { return (float)(1.0 / sqrt((double)K)); }

/* ---------------------------------------------------------------- activation quantizer */

/*
 * Symmetric INT4 quantization of fp16 activations (Sec. "Pruning-Targeted Quantizer Enhancement";
 * 4-bit activations of the W4A4 model), with the optional Hadamard rotation of Eq. 6 applied to
 * the row first, in the three granularities the paper names:
 *   per token   (the default; one scale per row)
 *   per tensor  ("tensor-wise quantization", Sec. 2.2 / 3): one scale from the amax over ALL rows,
 *               reported in every scales[i]
 *   per channel ("channel-wise quantization for activations", Sec. 3.3), read as a static
 *               multiplier m[k] per input channel applied before anything else (smoothing); the
 *               reciprocal belongs into the weights (oracle_quantize_weights takes it)
 *
 * Row i reads x[src*ldx .. +K) with src = row_index ? row_index[i] : i.
 *   v       = fp32(x)                        [ch_mul: v[k] = v[k] * m[k], one fp32 multiply]
 *                                            [rotate: v = FWHT(v) * (1/sqrt K)]
 *   amax    = max |v|  over the row, or over all M rows (per_tensor)
 *   amax==0 : scale 1, all codes 0
 *   else    : scale = amax / 7 ; inv = 7 / amax           (two fp32 divisions)
 *   q       = clamp( rint(v * inv), -8, 7 )               (fp32 multiply, ties to even)
 *   packed byte j = (q[2j] & 15) | (q[2j+1] & 15) << 4
 * Returns 0, or -1 on bad arguments.
 */
static void act_row(const uint16_t *xr, int K, int rotate, const float *ch_mul, float norm, float *v)
{
    for (int k = 0; k < K; ++k) v[k] = half_bits_to_float(xr[k]);
    if (ch_mul)
        for (int k = 0; k < K; ++k) v[k] = v[k] * ch_mul[k];
    if (rotate) {
        oracle_fwht_f32(v, K);
        for (int k = 0; k < K; ++k) v[k] = v[k] * norm;
    }
}

int oracle_quantize_act_ex(const uint16_t *x, int M, int K, int64_t ldx, const int32_t *row_index,
                           int rotate, int per_tensor, const float *ch_mul, uint8_t *q_packed, float *scales,
                           int8_t *codes_out /* nullable [M*K] */)
{
    if (M < 0 || K <= 0 || (K & 1)) return -1;
    if (rotate && (K & (K - 1))) return -1;
    const float norm = oracle_hadamard_norm(K);
    int err = 0;
    float tensor_amax = 0.0f;
    if (per_tensor) {
        float *v = (float *)malloc(sizeof(float) * (size_t)K);
        if (!v) return -2;
        for (int i = 0; i < M; ++i) {
            int64_t src = row_index ? (int64_t)row_index[i] : (int64_t)i;
            act_row(x + src * ldx, K, rotate, ch_mul, norm, v);
            for (int k = 0; k < K; ++k) {
                float a = fabsf(v[k]);
                if (a > tensor_amax) tensor_amax = a;
            }
        }
        free(v);
    }
#pragma omp parallel for schedule(static)
    for (int i = 0; i < M; ++i) {
        float *v = (float *)malloc(sizeof(float) * (size_t)K);
        if (!v) { err = 1; continue; }
        int64_t src = row_index ? (int64_t)row_index[i] : (int64_t)i;
        act_row(x + src * ldx, K, rotate, ch_mul, norm, v);
        float amax = 0.0f;
        if (per_tensor) {
            amax = tensor_amax;
        } else {
            for (int k = 0; k < K; ++k) {
                float a = fabsf(v[k]);
                if (a > amax) amax = a;
            }
        }
        float scale, inv;
        if (amax == 0.0f) {
            scale = 1.0f;
            inv = 0.0f;
        } else {
            scale = amax / 7.0f;
            inv = 7.0f / amax;
        }
        scales[i] = scale;
        uint8_t *qr = q_packed + (int64_t)i * (K / 2);
        for (int k = 0; k < K; k += 2) {
            int q0 = (int)rintf(v[k] * inv);
            int q1 = (int)rintf(v[k + 1] * inv);
            if (q0 < -8) q0 = -8;
            if (q0 > 7) q0 = 7;
            if (q1 < -8) q1 = -8;
            if (q1 > 7) q1 = 7;
            qr[k / 2] = (uint8_t)((q0 & 0xF) | ((q1 & 0xF) << 4));
            if (codes_out) {
                codes_out[(int64_t)i * K + k] = (int8_t)q0;
                codes_out[(int64_t)i * K + k + 1] = (int8_t)q1;
            }
        }
        free(v);
    }
    return err ? -2 : 0;
}

/* The per-token quantizer without smoothing: the form the hot path uses. */
int oracle_quantize_act(const uint16_t *x, int M, int K, int64_t ldx, const int32_t *row_index,
                        int rotate, uint8_t *q_packed, float *scales, int8_t *codes_out /* nullable [M*K] */)
{
    return oracle_quantize_act_ex(x, M, K, ldx, row_index, rotate, 0, NULL, q_packed, scales, codes_out);
}

/* The rotated (or plain) fp32 row the quantizer sees, exposed for the pins. */
void oracle_rotate_rows(const uint16_t *x, int M, int K, int64_t ldx, int rotate, float *out)
{
    const float norm = oracle_hadamard_norm(K);
    for (int i = 0; i < M; ++i) {
        float *v = out + (int64_t)i * K;
        for (int k = 0; k < K; ++k) v[k] = half_bits_to_float(x[(int64_t)i * ldx + k]);
        if (rotate) {
            oracle_fwht_f32(v, K);
            for (int k = 0; k < K; ++k) v[k] = v[k] * norm;
        }
    }
}

/* ---------------------------------------------------------------- offline weight quantizer */

/*
 * Offline side of W4A4 ("4-bit weights"; Eq. 6 for rotated layers): per-output-channel symmetric
 * round-to-nearest INT4 quantization of an fp16 weight matrix W [N][K] (row n = output channel n).
 *   v     = fp32(W[n])                 [ch_mul: v[k] = v[k] * d[k], the reciprocal of the activation
 *                                        side's channel multiplier, one fp32 multiply]
 *                                      [rotate: v = FWHT(v) * (1/sqrt K), i.e. row n of W H^T; the
 *                                        Sylvester matrix is symmetric, so H applied to the row is that]
 *   amax  = max |v|
 *   amax==0 : scale = fp16(1), codes 0
 *   else    : s16 = fp16_rn(amax / 7), raised to the smallest positive fp16 if that rounds to zero
 *   sf    = fp32(s16)
 *   q     = clamp( rint(v / sf), -8, 7 )              (fp32 division, ties to even)
 * The scale is rounded to fp16 BEFORE the codes are taken, because fp16 is what the linear
 * multiplies with. Returns 0, -1 on bad arguments, -3 if a scale is not finite.
 */
int oracle_quantize_weights(const uint16_t *w, int N, int K, int64_t ldw, int rotate, const float *ch_mul,
                            int8_t *codes, uint16_t *scales_fp16)
{
    if (N < 0 || K <= 0) return -1;
    if (rotate && (K & (K - 1))) return -1;
    const float norm = oracle_hadamard_norm(K);
    int err = 0;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        float *v = (float *)malloc(sizeof(float) * (size_t)K);
        if (!v) { err = 1; continue; }
        act_row(w + (int64_t)n * ldw, K, rotate, ch_mul, norm, v);
        float amax = 0.0f;
        for (int k = 0; k < K; ++k) {
            float a = fabsf(v[k]);
            if (a > amax) amax = a;
        }
        uint16_t s16;
        if (amax == 0.0f) {
            s16 = 0x3C00; /* 1.0 */
        } else {
            s16 = float_to_half_bits(amax / 7.0f);
            if ((s16 & 0x7FFF) == 0) s16 = 0x0001;
            if ((s16 & 0x7C00) == 0x7C00) err = 3; /* inf / nan: weights out of the fp16 range of scales */
        }
        scales_fp16[n] = s16;
        const float sf = half_bits_to_float(s16);
        for (int k = 0; k < K; ++k) {
            int q = (int)rintf(v[k] / sf);
            if (q < -8) q = -8;
            if (q > 7) q = 7;
            codes[(int64_t)n * K + k] = (int8_t)q;
        }
        free(v);
    }
    return err == 1 ? -2 : (err == 3 ? -3 : 0);
}

/* Two's-complement nibble pairs -> int8 codes (even index in the low nibble). */
void oracle_unpack_nibbles(const uint8_t *packed, int64_t n_codes, int8_t *codes)
{
    for (int64_t j = 0; j < n_codes / 2; ++j) {
        int lo = packed[j] & 0xF;
        int hi = packed[j] >> 4;
        codes[2 * j] = (int8_t)(lo >= 8 ? lo - 16 : lo);
        codes[2 * j + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
    }
}

void oracle_pack_nibbles(const int8_t *codes, int64_t n_codes, uint8_t *packed)
{
    for (int64_t j = 0; j < n_codes / 2; ++j)
        packed[j] = (uint8_t)((codes[2 * j] & 0xF) | ((codes[2 * j + 1] & 0xF) << 4));
}

/* ---------------------------------------------------------------- weights */

/*
 * Offline weight side (4-bit weights of the W4A4 model): the codes are given; the oracle
 * only validates them (every code in [-8,7], every scale finite and > 0).
 * Returns 0 if valid, 1 if a code is out of range, 2 if a scale is bad.
 */
int oracle_check_weights(const int8_t *codes, const uint16_t *scales_fp16, int N, int K)
{
    for (int64_t i = 0; i < (int64_t)N * K; ++i)
        if (codes[i] < -8 || codes[i] > 7) return 1;
    for (int n = 0; n < N; ++n) {
        float s = half_bits_to_float(scales_fp16[n]);
        if (!(s > 0.0f) || isinf(s)) return 2;
    }
    return 0;
}

/* ---------------------------------------------------------------- W4A4 GEMM */

/*
 * acc[m][n] = sum_k qx[m][k] * qw[n][k], exact in int32: the plain definition of the
 * product of the two code matrices (Q = W_q^T X in the paper's notation).
 */
void oracle_gemm_i32(const int8_t *qx, const int8_t *qw, int M, int N, int K, int32_t *acc)
{
#pragma omp parallel for schedule(static)
    for (int64_t mn = 0; mn < (int64_t)M * N; ++mn) {
        int m = (int)(mn / N);
        int n = (int)(mn % N);
        const int8_t *a = qx + (int64_t)m * K;
        const int8_t *b = qw + (int64_t)n * K;
        int32_t s = 0;
        for (int k = 0; k < K; ++k) s += (int32_t)a[k] * (int32_t)b[k];
        acc[mn] = s;
    }
}

/* One accumulator, for sampled checks at sizes where the full product is too slow. */
int32_t oracle_dot_i32(const int8_t *a, const int8_t *b, int K)
{
    int32_t s = 0;
    for (int k = 0; k < K; ++k) s += (int32_t)a[k] * (int32_t)b[k];
    return s;
}

/*
 * Dequantising epilogue: y = round16( (float(acc) * sx[m]) * float(sw[n]) ).
 * out_kind: 0 = fp16 bits, 1 = bf16 bits. |acc| < 2^24 for every K the path uses, so
 * float(acc) is exact.
 */
void oracle_epilogue(const int32_t *acc, const float *sx, const uint16_t *sw_fp16, int M, int N,
                     int out_kind, uint16_t *out)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            float t = (float)acc[(int64_t)m * N + n] * sx[m];
            float y = t * half_bits_to_float(sw_fp16[n]);
            out[(int64_t)m * N + n] = out_kind ? float_to_bf16_bits(y) : float_to_half_bits(y);
        }
}

/*
 * SiLU-gated product of the gate and up projections:
 *   g = (float(acc_g)*sx)*sw_g ; u = (float(acc_u)*sx)*sw_u   (fp32, as above)
 *   h = round16( g / (1 + exp(-g)) * u )                      (gate evaluated in fp64)
 */
void oracle_epilogue_swiglu(const int32_t *acc_g, const int32_t *acc_u, const float *sx,
                            const uint16_t *swg_fp16, const uint16_t *swu_fp16, int M, int N,
                            int out_kind, uint16_t *out)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            float tg = (float)acc_g[(int64_t)m * N + n] * sx[m];
            float g = tg * half_bits_to_float(swg_fp16[n]);
            float tu = (float)acc_u[(int64_t)m * N + n] * sx[m];
            float u = tu * half_bits_to_float(swu_fp16[n]);
            double h = ((double)g / (1.0 + exp(-(double)g))) * (double)u;
            float hf = (float)h;
            out[(int64_t)m * N + n] = out_kind ? float_to_bf16_bits(hf) : float_to_half_bits(hf);
        }
}

/* ---------------------------------------------------------------- pruning criterion */

/*
 * Robot-aware protection, Eq. 2-3: project a world point through K[R|t] and map the pixel
 * to a token coordinate. Kmat 3x3 row-major, Rt 3x4 row-major. in_front = 0 when the
 * homogeneous scale lambda <= 0 (point behind the camera; no ring).
 */
void oracle_project_center(const double Kmat[9], const double Rt[12], const double xyz[3],
                           double patch_w, double patch_h, int32_t out_tu_tv[2], int *in_front)
{
    double cam[3];
    for (int r = 0; r < 3; ++r)
        cam[r] = Rt[4 * r + 0] * xyz[0] + Rt[4 * r + 1] * xyz[1] + Rt[4 * r + 2] * xyz[2] + Rt[4 * r + 3];
    double p[3];
    for (int r = 0; r < 3; ++r)
        p[r] = Kmat[3 * r + 0] * cam[0] + Kmat[3 * r + 1] * cam[1] + Kmat[3 * r + 2] * cam[2];
    double lambda = p[2];
    if (!(lambda > 0.0)) {
        *in_front = 0;
        out_tu_tv[0] = 0;
        out_tu_tv[1] = 0;
        return;
    }
    *in_front = 1;
    double u = p[0] / lambda;
    double v = p[1] / lambda;
    out_tu_tv[0] = (int32_t)floor(u / patch_w);
    out_tu_tv[1] = (int32_t)floor(v / patch_h);
}

/* ---------------------------------------------------------------- attention scores of the query token */

/*
 * 2^t for t <= 0 in fp32, defined operation by operation so that any implementation gives the same
 * bits: i = floor(t), f = t - i in [0, 1) (exact), p = the degree-9 Taylor polynomial of 2^f = e^(f ln 2)
 * in Horner form with separately rounded multiplies and adds, result = p * 2^i (exact). t < -126 gives 0.
 * Truncation error below 1e-8, so the value is within a few ulp of the true 2^t.
 */
static const float EXP2_C[10] = {1.0f, 6.9314718056e-01f, 2.4022650696e-01f, 5.5504108665e-02f, 9.6181291076e-03f,
                                 1.3333558146e-03f, 1.5403530393e-04f, 1.5252733804e-05f, 1.3215486790e-06f,
                                 1.0178086009e-07f};
float oracle_exp2_neg(float t)
{
    if (t < -126.0f) return 0.0f;
    float i = floorf(t);
    float f = t - i;
    float p = EXP2_C[9];
    for (int k = 8; k >= 0; --k) {
        p = p * f;
        p = p + EXP2_C[k];
    }
    return ldexpf(p, (int)i);
}

/*
 * Importance of the visual tokens as seen from one task-query token (Sec. 3.2, strategy 1: "attention
 * scores ... of a task-query token"), computed from a fused QKV projection output (fp16):
 * for observation b, head h and visual token j
 *   l_j  = ( sum_{d} fp32(q[d]) * fp32(k_j[d]) ) * (1/sqrt D)     products and sums fp32, d ascending
 *   e_j  = 2^((l_j - max_j l) * log2(e))                         oracle_exp2_neg
 *   a_j  = fp16( e_j / sum_j e_j )                               sum j ascending, fp32 division
 * (softmax over the visual tokens only). q = row query_row of the observation, columns q_col0 + h*D ..;
 * k_j = row visual_start + j, columns k_col0 + h*D .. . Output A [batch][n_heads][n_visual] fp16: the
 * "score rows" that oracle_prune_tokens sums per token.
 */
int oracle_attention_scores(const uint16_t *qkv, int64_t ldq, int batch, int rows, int query_row, int visual_start,
                            int n_visual, int n_heads, int head_dim, int q_col0, int k_col0, uint16_t *scores_fp16)
{
    if (batch < 0 || rows <= 0 || query_row < 0 || query_row >= rows || visual_start < 0 || n_visual < 0 ||
        visual_start + n_visual > rows || n_heads <= 0 || head_dim <= 0)
        return -1;
    const float inv_sqrt_d = (float)(1.0 / sqrt((double)head_dim));
    const float log2e = 1.44269504f;
    float *l = (float *)malloc(sizeof(float) * (size_t)(n_visual + 1));
    if (!l) return -2;
    for (int b = 0; b < batch; ++b)
        for (int h = 0; h < n_heads; ++h) {
            const uint16_t *q = qkv + ((int64_t)b * rows + query_row) * ldq + q_col0 + (int64_t)h * head_dim;
            float m = -INFINITY;
            for (int j = 0; j < n_visual; ++j) {
                const uint16_t *k = qkv + ((int64_t)b * rows + visual_start + j) * ldq + k_col0 + (int64_t)h * head_dim;
                float acc = 0.0f;
                for (int d = 0; d < head_dim; ++d) {
                    float prod = half_bits_to_float(q[d]) * half_bits_to_float(k[d]);
                    acc = acc + prod;
                }
                l[j] = acc * inv_sqrt_d;
                if (l[j] > m) m = l[j];
            }
            float sum = 0.0f;
            for (int j = 0; j < n_visual; ++j) {
                float t = (l[j] - m) * log2e;
                l[j] = oracle_exp2_neg(t);
                sum = sum + l[j];
            }
            uint16_t *out = scores_fp16 + ((int64_t)b * n_heads + h) * n_visual;
            for (int j = 0; j < n_visual; ++j) out[j] = float_to_half_bits(l[j] / sum);
        }
    free(l);
    return 0;
}

/* a_j = A[0][j] + A[1][j] + ... + A[R-1][j], left to right in fp32 (the per-head rows of
 * attention from the task-query token to the visual tokens, summed). */
void oracle_score_sum(const uint16_t *A_fp16, int R, int n_visual, float *a)
{
    for (int j = 0; j < n_visual; ++j) {
        float s = half_bits_to_float(A_fp16[j]);
        for (int r = 1; r < R; ++r) s = s + half_bits_to_float(A_fp16[(int64_t)r * n_visual + j]);
        a[j] = s;
    }
}

/* Strategy 1, Eq. 1: mark the k tokens with the largest scores; equal scores -> lower index first. */
void oracle_topk_mask(const float *a, int n, int k, uint8_t *mask)
{
    memset(mask, 0, (size_t)n);
    if (k > n) k = n;
    for (int pick = 0; pick < k; ++pick) {
        int best = -1;
        for (int j = 0; j < n; ++j) {
            if (mask[j]) continue;
            if (best < 0 || a[j] > a[best]) best = j;
        }
        mask[best] = 1;
    }
}

/* Strategy 2, Eq. 4: tokens within Chebyshev distance R_t of the centre (c_u, c_v). */
void oracle_ring_mask(int grid_w, int grid_h, int c_u, int c_v, int radius, uint8_t *mask)
{
    for (int j = 0; j < grid_w * grid_h; ++j) {
        int tu = j % grid_w, tv = j / grid_w;
        int du = abs(tu - c_u), dv = abs(tv - c_v);
        int d = du > dv ? du : dv;
        mask[j] = (uint8_t)(radius >= 0 && d <= radius);
    }
}

/*
 * Strategy 3, Eq. 5: farthest-point sampling of m tokens from the tokens with remain[j] != 0,
 * squared Euclidean distance on integer grid coordinates. D starts at "infinite" so the
 * first pick is the lowest-index remaining token; afterwards each pick is the token whose
 * distance to the picked set is largest, lowest index on ties.
 */
void oracle_fps_mask(int grid_w, int grid_h, const uint8_t *remain, int m, uint8_t *picked)
{
    int n = grid_w * grid_h;
    int *D = (int *)malloc(sizeof(int) * (size_t)n);
    memset(picked, 0, (size_t)n);
    for (int j = 0; j < n; ++j) D[j] = INT_MAX;
    for (int step = 0; step < m; ++step) {
        int p = -1;
        for (int j = 0; j < n; ++j) {
            if (!remain[j] || picked[j]) continue;
            if (p < 0 || D[j] > D[p]) p = j;
        }
        if (p < 0) break; /* remainder exhausted */
        picked[p] = 1;
        int pu = p % grid_w, pv = p / grid_w;
        for (int j = 0; j < n; ++j) {
            if (!remain[j] || picked[j]) continue;
            int du = j % grid_w - pu, dv = j / grid_w - pv;
            int d2 = du * du + dv * dv;
            if (d2 < D[j]) D[j] = d2;
        }
    }
    free(D);
}

typedef struct {
    int batch, rows, visual_start, n_visual, grid_w, grid_h, score_rows, k_attn, keep_total, ring_radius;
    uint32_t flags;
} oracle_prune_params;

/*
 * The whole criterion for a batch of observations: K_final = K_attn U K_ring U K_fps, where
 * FPS fills the quota keep_total - |K_attn U K_ring| (nothing if already exceeded). Kept
 * rows = every non-visual row plus visual_start + j for j in K_final, ascending.
 * scores: fp16 [batch][R][n_visual] when score_rows = R > 0, else fp32 [batch][n_visual].
 * ring_center: [batch][2] = (c_u, c_v); ignored when ring_radius < 0 or NULL.
 * kept_idx: [batch][rows] (first n_kept[b] entries valid, the rest set to -1).
 * masks_out (nullable): [batch][3][n_visual] = attn, ring, fps membership.
 */
int oracle_prune_tokens(const oracle_prune_params *p, const void *scores, const int32_t *ring_center,
                        int32_t *kept_idx, int32_t *n_kept, uint8_t *masks_out)
{
    int nv = p->n_visual;
    if (p->batch < 0 || p->rows < 0 || nv < 0 || p->visual_start < 0 || p->visual_start + nv > p->rows) return -1;
    if (nv > 0 && p->grid_w * p->grid_h != nv) return -1;
    if (p->k_attn < 0 || p->keep_total < 0) return -1;
    float *a = (float *)malloc(sizeof(float) * (size_t)(nv + 1));
    uint8_t *attn = (uint8_t *)malloc((size_t)nv + 1), *ring = (uint8_t *)malloc((size_t)nv + 1);
    uint8_t *remain = (uint8_t *)malloc((size_t)nv + 1), *fps = (uint8_t *)malloc((size_t)nv + 1);
    for (int b = 0; b < p->batch; ++b) {
        if (p->score_rows > 0)
            oracle_score_sum((const uint16_t *)scores + (int64_t)b * p->score_rows * nv, p->score_rows, nv, a);
        else
            memcpy(a, (const float *)scores + (int64_t)b * nv, sizeof(float) * (size_t)nv);
        oracle_topk_mask(a, nv, p->k_attn, attn);
        if (p->ring_radius >= 0 && ring_center)
            oracle_ring_mask(p->grid_w, p->grid_h, ring_center[2 * b], ring_center[2 * b + 1], p->ring_radius, ring);
        else
            memset(ring, 0, (size_t)nv);
        int n_union = 0;
        for (int j = 0; j < nv; ++j) {
            int in_u = attn[j] | ring[j];
            n_union += in_u;
            remain[j] = (uint8_t)!in_u;
        }
        int m = p->keep_total - n_union;
        if (m < 0) m = 0;
        oracle_fps_mask(p->grid_w, p->grid_h, remain, m, fps);
        int cnt = 0;
        int32_t *out = kept_idx + (int64_t)b * p->rows;
        for (int r = 0; r < p->rows; ++r) {
            int keep = 1;
            if (r >= p->visual_start && r < p->visual_start + nv) {
                int j = r - p->visual_start;
                keep = attn[j] | ring[j] | fps[j];
            }
            if (keep) out[cnt++] = r;
        }
        n_kept[b] = cnt;
        for (int r = cnt; r < p->rows; ++r) out[r] = -1;
        if (masks_out) {
            memcpy(masks_out + ((int64_t)b * 3 + 0) * nv, attn, (size_t)nv);
            memcpy(masks_out + ((int64_t)b * 3 + 1) * nv, ring, (size_t)nv);
            memcpy(masks_out + ((int64_t)b * 3 + 2) * nv, fps, (size_t)nv);
        }
    }
    free(a); free(attn); free(ring); free(remain); free(fps);
    return 0;
}

/* Compaction: out row i of observation b = x row kept_idx[b][i] of observation b (bit copy). */
void oracle_gather_rows(const uint16_t *x, int batch, int rows, int K, int64_t ldx, const int32_t *kept_idx,
                        const int32_t *n_kept, int out_rows, int64_t ldo, uint16_t *out)
{
    for (int b = 0; b < batch; ++b)
        for (int i = 0; i < n_kept[b] && i < out_rows; ++i) {
            int32_t src = kept_idx[(int64_t)b * rows + i];
            memcpy(out + ((int64_t)b * out_rows + i) * ldo, x + ((int64_t)b * rows + src) * ldx,
                   sizeof(uint16_t) * (size_t)K);
        }
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

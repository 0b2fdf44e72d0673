/*
 * CPU oracle for the FP8 Smooth-SwiGLU MLP block (forward + backward).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
 * block computes, written from the paper; the CUDA library never includes, links or
 * calls it, and it shares no code with the CUDA library.  Only the tests, the smoke
 * check and the CPU-baseline leg of the benchmark may use it.
 *
 * What it follows (paper = "Scaling FP8 training to trillion-token LLMs"):
 *   - Section 2: E4M3 for weights/activations, E5M2 for gradients; per-tensor scaling
 *     from the tensor's range; just-in-time ("current amax") versus delayed ("given")
 *     scale selection.
 *   - Section 4.1: SwiGLU(x) = (x.w1) * Swish(x.w2), Swish(z) = z*sigma(z).
 *     w1 is the linear branch, w2 the Swish (gate) branch, w3 the last linear layer.
 *   - Section 4.4, Eq. (2): Smooth-SwiGLU_i(x) = s_i^-1 * Q(s_i * (w1_i.Q(x)) * Swish(w2_i.Q(x)))
 *     with a per-channel s_i derived from the per-channel maximum, and the merge
 *     w3~_i = Q(s_i^-1 * w3_i) that moves s_i^-1 onto the rows of W3.
 *   - Proof of Theorem 1: the factor sigma(z) + z*sigma'(z) of the gate derivative.
 *   - Section 6.2: high-precision master weights quantised each step, E4M3 operands in
 *     the forward phase and E5M2 gradients in the backward phase.
 *
 * Arithmetic: fp32 exactly as written, one operation per statement (compile with
 * -ffp-contract=off), GEMMs accumulate in fp32 sequentially over the contraction
 * index starting from 0.  FP8 encoding is done on the integer bits of the float:
 * round-to-nearest-even onto the format's grid (subnormals included), saturating to
 * the largest finite value (448 for E4M3, 57344 for E5M2); NaN stays NaN.
 *
 * Readings of points the paper leaves open are listed where they are taken
 * (search "READING").
 *
 * Parity status: the number formats, quantisation, GEMMs, SwiGLU, its derivative and
 * the Smooth-SwiGLU identities are each pinned by tests that do not go through this
 * file's own formulas (exhaustive code round trips, a library FP8 cast, fp64 brute
 * force, closed forms, finite differences).  The block as a whole has no worked
 * numeric example in the paper: whole-block parity unpinned beyond those pins.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_E4M3 0
#define ORC_E5M2 1

#define ORC_FLAG_SMOOTH      1u  /* per-channel s_i (Eq. 2); otherwise one per-tensor scale for H */
#define ORC_FLAG_Q_IDENTITY  2u  /* Q(v) = v: skip the FP8 rounding (pins only)                  */
#define ORC_FLAG_NO_BF16     4u  /* keep G, U, Y, dX in fp32 instead of rounding to bf16 (pins)  */
#define ORC_FLAG_H_BF16      8u  /* the paper's "SwiGLU output in BF16" variant (Section 4.3): the
                                    last linear layer is not quantised - its input H, its weight W3
                                    and the dY it meets in backward are bf16; everything else FP8   */
#define ORC_FLAG_GU_FP8     16u  /* the activations kept for backward, G and U, are stored as E4M3
                                    codes with one per-tensor scale instead of bf16 (the paper does
                                    not say how they are kept: a reading, offered as an option)     */

#define ORC_SCALE_GIVEN   0
#define ORC_SCALE_CURRENT 1

/* ------------------------------------------------------------------ bit helpers */

static uint32_t f2u(float v) { uint32_t u; memcpy(&u, &v, 4); return u; }
static float    u2f(uint32_t u) { float v; memcpy(&v, &u, 4); return v; }

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ FP8 formats
 * Section 2 names the two formats by their bit split and cites the FP8 standard:
 *   E4M3: 1-4-3, bias 7, no infinity, S.1111.111 is NaN, largest finite 448 (0x7E).
 *   E5M2: 1-5-2, bias 15, IEEE-like (0x7C inf, 0x7D..0x7F NaN), largest finite 57344 (0x7B).
 */
static int fmt_mbits(int fmt) { return fmt == ORC_E4M3 ? 3 : 2; }
static int fmt_bias(int fmt)  { return fmt == ORC_E4M3 ? 7 : 15; }
static int fmt_maxcode(int fmt) { return fmt == ORC_E4M3 ? 0x7E : 0x7B; }

float orc_fmt_max(int fmt) { return fmt == ORC_E4M3 ? 448.0f : 57344.0f; }

float orc_decode(int fmt, uint8_t code) {
    const int M = fmt_mbits(fmt), B = fmt_bias(fmt);
    const int sign = code >> 7;
    const int e = (code & 0x7F) >> M;
    const int m = code & ((1 << M) - 1);
    float v;
    if (fmt == ORC_E4M3) {
        if ((code & 0x7F) == 0x7F) return NAN;
    } else {
        if (e == 31) return m ? NAN : (sign ? -INFINITY : INFINITY);
    }
    if (e == 0) v = ldexpf((float)m, 1 - B - M);                 /* subnormal: m * 2^(emin-M) */
    else        v = ldexpf((float)((1 << M) + m), e - B - M);    /* (1.m) * 2^(e-B)           */
    return sign ? -v : v;
}

/* Round-to-nearest-even of a 32-bit significand shifted right by sh (sh >= 1). */
static uint32_t rne_shift(uint32_t sig, int sh) {
    if (sh > 31) return 0;            /* below half of the smallest step: rounds to 0 */
    uint32_t q    = sig >> sh;
    uint32_t rem  = sig & ((1u << sh) - 1u);
    uint32_t half = 1u << (sh - 1);
    if (rem > half || (rem == half && (q & 1u))) q += 1u;
    return q;
}

uint8_t orc_encode(int fmt, float v) {
    const int M = fmt_mbits(fmt), B = fmt_bias(fmt);
    const uint32_t u = f2u(v);
    const uint8_t sign = (uint8_t)((u >> 31) << 7);
    const uint32_t a = u & 0x7FFFFFFFu;
    if (a > 0x7F800000u) return (uint8_t)(sign | 0x7F);                    /* NaN stays NaN     */
    if (a == 0x7F800000u) return (uint8_t)(sign | fmt_maxcode(fmt));       /* inf saturates     */
    const int fe = (int)(a >> 23);                                         /* float exp field   */
    if (fe == 0) return sign;                       /* float subnormals are far below half the smallest FP8 step */
    const int e = fe - 127;                                                /* unbiased exponent */
    const uint32_t sig = (a & 0x7FFFFFu) | 0x800000u;                      /* 1.frac, 24 bits   */
    const int emin = 1 - B;
    int code;
    if (e >= emin) {
        /* normal range: keep M fraction bits; a carry out of the significand moves into the exponent */
        uint32_t q = rne_shift(sig, 23 - M);                               /* in [2^M, 2^(M+1)] */
        code = ((e + B) << M) + (int)q - (1 << M);
    } else {
        /* subnormal range: integer multiple of 2^(emin-M); q == 2^M is the smallest normal */
        uint32_t q = rne_shift(sig, (23 - M) + (emin - e));
        code = (int)q;
    }
    if (code > fmt_maxcode(fmt)) code = fmt_maxcode(fmt);                  /* saturate to finite */
    return (uint8_t)(sign | code);
}

void orc_encode_array(int fmt, const float* v, int64_t n, uint8_t* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = orc_encode(fmt, v[i]);
}
void orc_decode_array(int fmt, const uint8_t* c, int64_t n, float* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = orc_decode(fmt, c[i]);
}

/* bf16: round-to-nearest-even on the upper 16 bits of the float. */
uint16_t orc_f32_to_bf16(float v) {
    uint32_t u = f2u(v);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}
float orc_bf16_to_f32(uint16_t h) { return u2f(((uint32_t)h) << 16); }

void orc_bf16_to_f32_array(const uint16_t* h, int64_t n, float* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = orc_bf16_to_f32(h[i]);
}
void orc_f32_to_bf16_array(const float* v, int64_t n, uint16_t* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = orc_f32_to_bf16(v[i]);
}

/* ------------------------------------------------------------------ scaling (Section 2)
 * READING: Section 2 describes per-tensor scaling only as a factor chosen from the range of the
 * tensor's values; it is taken as scale = fmt_max / max|v| with no margin; a zero or non-finite
 * amax gives scale 1.
 */
float orc_amax(const float* v, int64_t n) {
    float a = 0.0f;
    for (int64_t i = 0; i < n; ++i) { float t = fabsf(v[i]); if (t > a) a = t; }
    return a;
}

float orc_scale_from_amax(int fmt, float amax) {
    if (!(amax > 0.0f) || isinf(amax)) return 1.0f;
    float s = orc_fmt_max(fmt) / amax;
    if (isinf(s) || isnan(s)) return 1.0f;
    return s;
}

/* READING (Section 4.4, third step of the recipe: the per-channel maxima decide the per-channel
 * factors, no formula given): s is the largest power of two p with p*amax <= fmt_max.
 * A power of two makes s * s^-1 exact, so the scaled block is the same function.
 * fmt_max = 0.875 * 2^E with E = 9 (E4M3) or 16 (E5M2); amax = m * 2^e, m in [0.5, 1).
 */
float orc_pow2_scale(int fmt, float amax) {
    if (!(amax > 0.0f) || isinf(amax)) return 1.0f;
    const int E = fmt == ORC_E4M3 ? 9 : 16;
    int e;
    float m = frexpf(amax, &e);
    int k = (m <= 0.875f) ? (E - e) : (E - 1 - e);
    if (k > 100) k = 100;
    if (k < -100) k = -100;
    return ldexpf(1.0f, k);
}

/* Q(v * scale): returns the decoded value and, if code != NULL, the 8-bit code. */
static float quant1(int fmt, float v, float scale, unsigned flags, uint8_t* code) {
    float t = v * scale;
    if (flags & ORC_FLAG_Q_IDENTITY) { if (code) *code = 0; return t; }
    uint8_t c = orc_encode(fmt, t);
    if (code) *code = c;
    return orc_decode(fmt, c);
}

/* Quantise a rows x cols tensor; row_mul (nullable) multiplies row r before scaling
 * (used for W3' = diag(s^-1) W3).  amax_out (nullable) receives max|v * row_mul|.
 * dst codes are written with leading dimension ld_dst; deq (nullable) gets the decoded
 * values contiguously.
 */
void orc_quantize(const float* src, int64_t rows, int64_t cols, const float* row_mul,
                  int fmt, float scale, unsigned flags,
                  uint8_t* dst, int64_t ld_dst, float* deq, float* amax_out) {
    float a = 0.0f;
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t c = 0; c < cols; ++c) {
            float v = src[r * cols + c];
            if (row_mul) v = v * row_mul[r];
            float t = fabsf(v);
            if (t > a) a = t;
            uint8_t code;
            float q = quant1(fmt, v, scale, flags, &code);
            if (dst) dst[r * ld_dst + c] = code;
            if (deq) deq[r * cols + c] = q;
        }
    }
    if (amax_out) *amax_out = a;
}

/* How the range of a format was used by a tensor of codes (Section 4.3 looks at exactly this for the SwiGLU
 * output: values lost to underflow next to values at the top of the range): the number of codes that are
 * zero (+0 or -0) and the number at the largest finite magnitude (where the saturating cast puts everything
 * beyond it).  codes is [rows, cols] with row stride ld. */
void orc_code_stats(int fmt, const uint8_t* codes, int64_t rows, int64_t cols, int64_t ld, int64_t* zero, int64_t* top) {
    const uint8_t top_code = fmt == ORC_E4M3 ? 0x7E : 0x7B;
    int64_t z = 0, t = 0;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            const uint8_t mag = codes[r * ld + c] & 0x7F;
            if (mag == 0) ++z;
            if (mag == top_code) ++t;
        }
    *zero = z; *top = t;
}

float orc_amax_rows(const float* src, int64_t rows, int64_t cols, const float* row_mul) {
    float a = 0.0f;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            float v = src[r * cols + c];
            if (row_mul) v = v * row_mul[r];
            float t = fabsf(v);
            if (t > a) a = t;
        }
    return a;
}

/* ------------------------------------------------------------------ GEMM
 * C[m,n] = sum_k A(m,k) * B(k,n), fp32, k ascending from an accumulator of 0.
 * A(m,k) = A[m*a_rs + k*a_cs], B(k,n) = B[k*b_rs + n*b_cs].  The loop nest is m, k, n
 * with a row of accumulators, which leaves every C[m,n] a sequential sum over k.
 */
void orc_gemm(int64_t M, int64_t N, int64_t K,
              const float* A, int64_t a_rs, int64_t a_cs,
              const float* B, int64_t b_rs, int64_t b_cs,
              float* C) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        float* acc = C + m * N;
        for (int64_t n = 0; n < N; ++n) acc[n] = 0.0f;
        for (int64_t k = 0; k < K; ++k) {
            const float a = A[m * a_rs + k * a_cs];
            const float* b = B + k * b_rs;
            if (b_cs == 1) { for (int64_t n = 0; n < N; ++n) acc[n] = acc[n] + a * b[n]; }
            else           { for (int64_t n = 0; n < N; ++n) acc[n] = acc[n] + a * b[n * b_cs]; }
        }
    }
}

/* ------------------------------------------------------------------ SwiGLU pieces (Section 4.1) */
static float sigmoidf_(float z) { return 1.0f / (1.0f + expf(-z)); }

float orc_swiglu(float u_lin, float g_gate) {            /* (x.w1) * (x.w2) * sigma(x.w2) */
    float sig = sigmoidf_(g_gate);
    float sw = g_gate * sig;
    return u_lin * sw;
}

/* d/du and d/dg of u * g * sigma(g); the gate factor is sigma(g) + g*sigma'(g)
 * = sigma(g) * (1 + g*(1 - sigma(g)))  (proof of Theorem 1). */
void orc_swiglu_grad(float u_lin, float g_gate, float dh, float* du, float* dg) {
    float sig = sigmoidf_(g_gate);
    float sw = g_gate * sig;
    *du = dh * sw;
    float one_m = 1.0f - sig;
    float t = g_gate * one_m;
    float t1 = 1.0f + t;
    float dsw = sig * t1;
    float dhu = dh * u_lin;
    *dg = dhu * dsw;
}

/* ------------------------------------------------------------------ forward
 * Inputs : x bf16 [T,d]; master weights fp32 W1,W2 [d,f], W3 [f,d].
 * Scales : sx, sw12, sw3 scalars, s_h[f].  ORC_SCALE_GIVEN reads them;
 *          ORC_SCALE_CURRENT derives them from this call's data and writes them back.
 * Outputs (any may be NULL): amax values; codes Xq [T,d], W12q [d,2f] (gate W2 in columns
 *          [0,f), linear W1 in [f,2f)), W3q [f,d], Hq [T,f]; saved G,U (bf16 bits, [T,f]);
 *          H fp32 (unscaled SwiGLU output); Y (bf16 bits) and Y as fp32.
 * READING: W1 and W2 share one scale (they are one concatenated operand).
 * READING: saved activations for backward are the bf16-rounded G and U; with ORC_FLAG_GU_FP8 they
 *          are GUq [T,2f] = Q_e4m3(sgu * [G | U]) instead, sgu one scale for both (448 / max(|G|,|U|)
 *          in current-amax mode), and backward takes G~ = decode(code) * (1 / sgu).
 * READING: with Smooth off, H gets one per-tensor scale sh = 448/max_i amax_h[i] held in
 *          every s_h[i]; W3 is quantised unscaled and 1/sh joins the output dequantisation.
 */
int orc_forward(int64_t T, int64_t d, int64_t f, unsigned flags, int scale_mode,
                const uint16_t* x_bf16, const float* W1, const float* W2, const float* W3,
                float* sx, float* sw12, float* s_h, float* sw3,
                float* amax_x, float* amax_w1, float* amax_w2, float* amax_w3, float* amax_h,
                uint8_t* Xq, uint8_t* W12q, uint8_t* W3q, uint8_t* Hq,
                uint16_t* G_bf16, uint16_t* U_bf16, float* H_f32,
                uint16_t* Y_bf16, float* Y_f32,
                float* xq_f, float* w12q_f, float* w3q_f, float* hq_f, float* G_f32, float* U_f32,
                float* sgu, float* amax_gu, uint8_t* GUq) {
    const int smooth = (flags & ORC_FLAG_SMOOTH) != 0;
    float* xf   = (float*)malloc(sizeof(float) * T * d);
    float* xq   = (float*)malloc(sizeof(float) * T * d);
    float* w2q  = (float*)malloc(sizeof(float) * d * f);
    float* w1q  = (float*)malloc(sizeof(float) * d * f);
    float* w3q  = (float*)malloc(sizeof(float) * f * d);
    float* accG = (float*)malloc(sizeof(float) * T * f);
    float* accU = (float*)malloc(sizeof(float) * T * f);
    float* H    = (float*)malloc(sizeof(float) * T * f);
    float* hq   = (float*)malloc(sizeof(float) * T * f);
    float* accY = (float*)malloc(sizeof(float) * T * d);
    float* rmul = (float*)malloc(sizeof(float) * f);
    float* ah   = (float*)malloc(sizeof(float) * f);
    if (!xf || !xq || !w2q || !w1q || !w3q || !accG || !accU || !H || !hq || !accY || !rmul || !ah) return -1;

    /* quantise x (E4M3) */
    orc_bf16_to_f32_array(x_bf16, T * d, xf);
    float ax = orc_amax(xf, T * d);
    if (scale_mode == ORC_SCALE_CURRENT) *sx = orc_scale_from_amax(ORC_E4M3, ax);
    orc_quantize(xf, T, d, NULL, ORC_E4M3, *sx, flags, Xq, d, xq, NULL);
    if (amax_x) *amax_x = ax;

    /* quantise W2 (gate) and W1 (linear) with one shared scale */
    float a1 = orc_amax(W1, d * f), a2 = orc_amax(W2, d * f);
    if (scale_mode == ORC_SCALE_CURRENT) *sw12 = orc_scale_from_amax(ORC_E4M3, a1 > a2 ? a1 : a2);
    orc_quantize(W2, d, f, NULL, ORC_E4M3, *sw12, flags, W12q, 2 * f, w2q, NULL);
    orc_quantize(W1, d, f, NULL, ORC_E4M3, *sw12, flags, W12q ? W12q + f : NULL, 2 * f, w1q, NULL);
    if (amax_w1) *amax_w1 = a1;
    if (amax_w2) *amax_w2 = a2;

    /* gate/up projections, dequantised */
    orc_gemm(T, f, d, xq, d, 1, w2q, f, 1, accG);
    orc_gemm(T, f, d, xq, d, 1, w1q, f, 1, accU);
    const float inv_sx = 1.0f / *sx, inv_sw12 = 1.0f / *sw12;
    const float dq1 = inv_sx * inv_sw12;
    for (int64_t i = 0; i < f; ++i) ah[i] = 0.0f;
    if (flags & ORC_FLAG_GU_FP8) {
        /* G and U kept as E4M3 codes: their common maximum, the scale, the codes */
        float agu = 0.0f;
        for (int64_t j = 0; j < T * f; ++j) {
            float a = fabsf(accG[j] * dq1); if (a > agu) agu = a;
            a = fabsf(accU[j] * dq1);       if (a > agu) agu = a;
        }
        if (amax_gu) *amax_gu = agu;
        if (scale_mode == ORC_SCALE_CURRENT) *sgu = orc_scale_from_amax(ORC_E4M3, agu);
        if (GUq)
            for (int64_t t = 0; t < T; ++t)
                for (int64_t i = 0; i < f; ++i) {
                    quant1(ORC_E4M3, accG[t * f + i] * dq1, *sgu, flags, &GUq[t * 2 * f + i]);
                    quant1(ORC_E4M3, accU[t * f + i] * dq1, *sgu, flags, &GUq[t * 2 * f + f + i]);
                }
    }
    for (int64_t t = 0; t < T; ++t)
        for (int64_t i = 0; i < f; ++i) {
            float g = accG[t * f + i] * dq1;
            float u = accU[t * f + i] * dq1;
            float h = orc_swiglu(u, g);
            H[t * f + i] = h;
            float ab = fabsf(h);
            if (ab > ah[i]) ah[i] = ab;                      /* per-channel max (Section 4.4, steps 1-2) */
            if (G_bf16) G_bf16[t * f + i] = (flags & ORC_FLAG_NO_BF16) ? 0 : orc_f32_to_bf16(g);
            if (U_bf16) U_bf16[t * f + i] = (flags & ORC_FLAG_NO_BF16) ? 0 : orc_f32_to_bf16(u);
            if (G_f32) G_f32[t * f + i] = g;
            if (U_f32) U_f32[t * f + i] = u;
        }
    if (amax_h) memcpy(amax_h, ah, sizeof(float) * f);
    if (H_f32) memcpy(H_f32, H, sizeof(float) * T * f);

    /* per-channel scale s_i (step 3) or the per-tensor scale */
    if (scale_mode == ORC_SCALE_CURRENT) {
        if (smooth) {
            for (int64_t i = 0; i < f; ++i) s_h[i] = orc_pow2_scale(ORC_E4M3, ah[i]);
        } else {
            float a = 0.0f;
            for (int64_t i = 0; i < f; ++i) if (ah[i] > a) a = ah[i];
            float sh = orc_scale_from_amax(ORC_E4M3, a);
            for (int64_t i = 0; i < f; ++i) s_h[i] = sh;
        }
    }
    /* Q(s_i * H) (Eq. 2) */
    const int h_bf16 = (flags & ORC_FLAG_H_BF16) != 0;
    if (h_bf16) {
        /* READING (Section 4.3: the experiment that leaves the last linear layer's input unquantised):
         * that layer runs in bf16 - H and W3 are rounded to bf16 (no scales), products accumulate in fp32. */
        for (int64_t i = 0; i < f; ++i) s_h[i] = 1.0f;
        for (int64_t i = 0; i < T * f; ++i) {
            hq[i] = orc_bf16_to_f32(orc_f32_to_bf16(H[i]));
            if (Hq) Hq[i] = 0;
        }
    } else
    for (int64_t t = 0; t < T; ++t)
        for (int64_t i = 0; i < f; ++i) {
            uint8_t code;
            hq[t * f + i] = quant1(ORC_E4M3, H[t * f + i], s_h[i], flags, &code);
            if (Hq) Hq[t * f + i] = code;
        }

    /* W3' = diag(s^-1) W3 and its quantisation (the merge of Section 4.4) */
    float dq2;
    if (h_bf16) {
        float a3 = orc_amax(W3, f * d);
        for (int64_t i = 0; i < f * d; ++i) w3q[i] = orc_bf16_to_f32(orc_f32_to_bf16(W3[i]));
        if (W3q) memset(W3q, 0, (size_t)(f * d));
        if (amax_w3) *amax_w3 = a3;
        *sw3 = 1.0f;
        dq2 = 1.0f;
    } else if (smooth) {
        for (int64_t i = 0; i < f; ++i) rmul[i] = 1.0f / s_h[i];
        float a3 = orc_amax_rows(W3, f, d, rmul);
        if (scale_mode == ORC_SCALE_CURRENT) *sw3 = orc_scale_from_amax(ORC_E4M3, a3);
        orc_quantize(W3, f, d, rmul, ORC_E4M3, *sw3, flags, W3q, d, w3q, NULL);
        if (amax_w3) *amax_w3 = a3;
        dq2 = 1.0f / *sw3;
    } else {
        float a3 = orc_amax(W3, f * d);
        if (scale_mode == ORC_SCALE_CURRENT) *sw3 = orc_scale_from_amax(ORC_E4M3, a3);
        orc_quantize(W3, f, d, NULL, ORC_E4M3, *sw3, flags, W3q, d, w3q, NULL);
        if (amax_w3) *amax_w3 = a3;
        float inv_sw3 = 1.0f / *sw3, inv_sh = 1.0f / s_h[0];
        dq2 = inv_sw3 * inv_sh;
    }

    /* down projection */
    orc_gemm(T, d, f, hq, f, 1, w3q, d, 1, accY);
    for (int64_t i = 0; i < T * d; ++i) {
        float y = accY[i] * dq2;
        if (Y_bf16) Y_bf16[i] = (flags & ORC_FLAG_NO_BF16) ? 0 : orc_f32_to_bf16(y);
        if (Y_f32)  Y_f32[i]  = (flags & ORC_FLAG_NO_BF16) ? y : orc_bf16_to_f32(orc_f32_to_bf16(y));
    }

    /* decoded operands, for callers that want to look at them (and for the Q = identity pins) */
    if (xq_f) memcpy(xq_f, xq, sizeof(float) * T * d);
    if (w3q_f) memcpy(w3q_f, w3q, sizeof(float) * f * d);
    if (hq_f) memcpy(hq_f, hq, sizeof(float) * T * f);
    if (w12q_f)
        for (int64_t k = 0; k < d; ++k)
            for (int64_t i = 0; i < f; ++i) {
                w12q_f[k * 2 * f + i] = w2q[k * f + i];
                w12q_f[k * 2 * f + f + i] = w1q[k * f + i];
            }

    free(xf); free(xq); free(w2q); free(w1q); free(w3q); free(accG); free(accU);
    free(H); free(hq); free(accY); free(rmul); free(ah);
    return 0;
}

/* ------------------------------------------------------------------ backward
 * Takes what forward left behind: codes Xq, W12q, W3q, Hq, saved G,U (bf16 bits, or fp32
 * arrays G_f32/U_f32 when ORC_FLAG_NO_BF16, or E4M3 codes GUq with their scale when
 * ORC_FLAG_GU_FP8), and the forward scales.
 * READING: every Q is straight-through and s_i is a constant; weights and activations
 * keep their E4M3 codes in the backward GEMMs, only dY and dZ = [dG|dU] are E5M2.
 * The header above lists what pins this.
 * READING: dG and dU share one scale sdz (one concatenated operand), a power of two
 * derived from max(|dG|,|dU|) in current-amax mode.
 * For ORC_FLAG_Q_IDENTITY the "codes" are unused and the decoded operands are passed as
 * fp32 arrays instead (xq_f, w12q_f [d,2f], w3q_f, hq_f).
 * dH_out / dZ_out (nullable) receive the fp32 intermediates dH and [dG | dU] as they stand before
 * the E5M2 cast (tests derive tolerance bounds from them; nothing else reads them).
 */
int orc_backward(int64_t T, int64_t d, int64_t f, unsigned flags, int scale_mode,
                 const uint16_t* dy_bf16,
                 const uint8_t* Xq, const uint8_t* W12q, const uint8_t* W3q, const uint8_t* Hq,
                 const float* xq_f, const float* w12q_f, const float* w3q_f, const float* hq_f,
                 const uint16_t* G_bf16, const uint16_t* U_bf16, const float* G_f32, const float* U_f32,
                 float sx, float sw12, const float* s_h, float sw3,
                 float* sdy, float* sdz, float* amax_dy, float* amax_dz,
                 uint8_t* dYq, uint8_t* dZq /*[T,2f]: dG | dU*/,
                 uint16_t* dX_bf16, float* dX_f32, float* dW1, float* dW2, float* dW3,
                 const uint8_t* GUq, float sgu,
                 float* dH_out /*[T,f], nullable*/, float* dZ_out /*[T,2f] = dG | dU before scaling, nullable*/) {
    const int smooth = (flags & ORC_FLAG_SMOOTH) != 0;
    const int qid = (flags & ORC_FLAG_Q_IDENTITY) != 0;
    float* dyf  = (float*)malloc(sizeof(float) * T * d);
    float* dyq  = (float*)malloc(sizeof(float) * T * d);
    float* xq   = (float*)malloc(sizeof(float) * T * d);
    float* w12q = (float*)malloc(sizeof(float) * d * 2 * f);
    float* w3q  = (float*)malloc(sizeof(float) * f * d);
    float* hq   = (float*)malloc(sizeof(float) * T * f);
    float* accH = (float*)malloc(sizeof(float) * T * f);
    float* dG   = (float*)malloc(sizeof(float) * T * f);
    float* dU   = (float*)malloc(sizeof(float) * T * f);
    float* dzq  = (float*)malloc(sizeof(float) * T * 2 * f);
    float* accX = (float*)malloc(sizeof(float) * T * d);
    float* acc  = (float*)malloc(sizeof(float) * (f * d > d * 2 * f ? f * d : d * 2 * f));
    if (!dyf || !dyq || !xq || !w12q || !w3q || !hq || !accH || !dG || !dU || !dzq || !accX || !acc) return -1;

    const int h_bf16 = (flags & ORC_FLAG_H_BF16) != 0;
    if (qid) {
        memcpy(xq, xq_f, sizeof(float) * T * d);
        memcpy(w12q, w12q_f, sizeof(float) * d * 2 * f);
        memcpy(w3q, w3q_f, sizeof(float) * f * d);
        memcpy(hq, hq_f, sizeof(float) * T * f);
    } else {
        orc_decode_array(ORC_E4M3, Xq, T * d, xq);
        orc_decode_array(ORC_E4M3, W12q, d * 2 * f, w12q);
        if (h_bf16) {                       /* the bf16 operands of the unquantised last layer */
            memcpy(w3q, w3q_f, sizeof(float) * f * d);
            memcpy(hq, hq_f, sizeof(float) * T * f);
        } else {
            orc_decode_array(ORC_E4M3, W3q, f * d, w3q);
            orc_decode_array(ORC_E4M3, Hq, T * f, hq);
        }
    }

    /* quantise dY (E5M2) */
    orc_bf16_to_f32_array(dy_bf16, T * d, dyf);
    float ady = orc_amax(dyf, T * d);
    if (h_bf16) {                           /* dY only meets the bf16 layer: used as it is */
        *sdy = 1.0f;
        memcpy(dyq, dyf, sizeof(float) * T * d);
        if (dYq) memset(dYq, 0, (size_t)(T * d));
    } else {
    if (scale_mode == ORC_SCALE_CURRENT) *sdy = orc_scale_from_amax(ORC_E5M2, ady);
    orc_quantize(dyf, T, d, NULL, ORC_E5M2, *sdy, flags, dYq, d, dyq, NULL);
    }
    if (amax_dy) *amax_dy = ady;
    const float inv_sdy = 1.0f / *sdy, inv_sw3 = 1.0f / sw3;

    /* dH~ = dY W3'^T.  Smooth on: W3' carries s_i^-1, so dH = s (.) dH~ (chain rule through
     * Hq = Q(s_i H)).  Smooth off: W3' = W3 and the 1/sh of the forward dequantisation cancels
     * against Hq = Q(sh H), so dH = dH~. */
    orc_gemm(T, f, d, dyq, d, 1, w3q, 1, d, accH);
    const float dqh = inv_sdy * inv_sw3;
    float adz = 0.0f;
    for (int64_t t = 0; t < T; ++t)
        for (int64_t i = 0; i < f; ++i) {
            float dht = accH[t * f + i] * dqh;
            float dh = smooth ? dht * s_h[i] : dht;
            float g, u;
            if (flags & ORC_FLAG_GU_FP8) {          /* kept as E4M3 codes with the scale sgu */
                g = orc_decode(ORC_E4M3, GUq[t * 2 * f + i]) * (1.0f / sgu);
                u = orc_decode(ORC_E4M3, GUq[t * 2 * f + f + i]) * (1.0f / sgu);
            } else if (flags & ORC_FLAG_NO_BF16) {
                g = G_f32[t * f + i]; u = U_f32[t * f + i];
            } else {
                g = orc_bf16_to_f32(G_bf16[t * f + i]); u = orc_bf16_to_f32(U_bf16[t * f + i]);
            }
            float du, dg;
            orc_swiglu_grad(u, g, dh, &du, &dg);
            dG[t * f + i] = dg;
            dU[t * f + i] = du;
            if (dH_out) dH_out[t * f + i] = dh;
            if (dZ_out) { dZ_out[t * 2 * f + i] = dg; dZ_out[t * 2 * f + f + i] = du; }
            float a = fabsf(dg); if (a > adz) adz = a;
            a = fabsf(du);       if (a > adz) adz = a;
        }
    if (amax_dz) *amax_dz = adz;
    if (scale_mode == ORC_SCALE_CURRENT) *sdz = orc_pow2_scale(ORC_E5M2, adz);
    for (int64_t t = 0; t < T; ++t)
        for (int64_t i = 0; i < f; ++i) {
            uint8_t cg, cu;
            dzq[t * 2 * f + i]     = quant1(ORC_E5M2, dG[t * f + i], *sdz, flags, &cg);
            dzq[t * 2 * f + f + i] = quant1(ORC_E5M2, dU[t * f + i], *sdz, flags, &cu);
            if (dZq) { dZq[t * 2 * f + i] = cg; dZq[t * 2 * f + f + i] = cu; }
        }
    const float inv_sdz = 1.0f / *sdz, inv_sw12 = 1.0f / sw12, inv_sx = 1.0f / sx;

    /* dW3[i,j] = (sum_t Hq[t,i] dYq[t,j]) / sdy / s_i   (gradient w.r.t. the master W3) */
    if (dW3) {
        orc_gemm(f, d, T, hq, 1, f, dyq, d, 1, acc);
        for (int64_t i = 0; i < f; ++i) {
            float rs = 1.0f / s_h[i];                 /* H = Hq / s_i in both modes */
            float dq = inv_sdy * rs;
            for (int64_t j = 0; j < d; ++j) dW3[i * d + j] = acc[i * d + j] * dq;
        }
    }

    /* dX = dZ [W2|W1]^T : one contraction over the 2f concatenated channels */
    orc_gemm(T, d, 2 * f, dzq, 2 * f, 1, w12q, 1, 2 * f, accX);
    const float dqx = inv_sdz * inv_sw12;
    for (int64_t i = 0; i < T * d; ++i) {
        float v = accX[i] * dqx;
        if (dX_bf16) dX_bf16[i] = (flags & ORC_FLAG_NO_BF16) ? 0 : orc_f32_to_bf16(v);
        if (dX_f32)  dX_f32[i]  = (flags & ORC_FLAG_NO_BF16) ? v : orc_bf16_to_f32(orc_f32_to_bf16(v));
    }

    /* [dW2|dW1] = Xq^T dZq */
    if (dW1 || dW2) {
        orc_gemm(d, 2 * f, T, xq, 1, d, dzq, 2 * f, 1, acc);
        const float dqw = inv_sx * inv_sdz;
        for (int64_t k = 0; k < d; ++k)
            for (int64_t i = 0; i < f; ++i) {
                if (dW2) dW2[k * f + i] = acc[k * 2 * f + i] * dqw;
                if (dW1) dW1[k * f + i] = acc[k * 2 * f + f + i] * dqw;
            }
    }

    free(dyf); free(dyq); free(xq); free(w12q); free(w3q); free(hq); free(accH);
    free(dG); free(dU); free(dzq); free(accX); free(acc);
    return 0;
}

/* ------------------------------------------------------------------ fp64 definition of the block
 * The unquantised block in double precision, by the definitions alone: used to pin the
 * quantised path (Q = identity must reproduce it; Smooth-SwiGLU must not change it).
 * s (nullable) applies Eq. (2) with Q = identity: H*s_i, then W3 rows times 1/s_i.
 */
void orc_mlp_f64(int64_t T, int64_t d, int64_t f,
                 const double* x, const double* W1, const double* W2, const double* W3,
                 const double* s, double* H_out, double* Y) {
    for (int64_t t = 0; t < T; ++t) {
        for (int64_t j = 0; j < d; ++j) Y[t * d + j] = 0.0;
        for (int64_t i = 0; i < f; ++i) {
            double u = 0.0, g = 0.0;
            for (int64_t k = 0; k < d; ++k) {
                u += x[t * d + k] * W1[k * f + i];
                g += x[t * d + k] * W2[k * f + i];
            }
            double h = u * g * (1.0 / (1.0 + exp(-g)));
            if (H_out) H_out[t * f + i] = h;
            double hs = s ? h * s[i] : h;
            for (int64_t j = 0; j < d; ++j) {
                double w = s ? (1.0 / s[i]) * W3[i * d + j] : W3[i * d + j];
                Y[t * d + j] += hs * w;
            }
        }
    }
}

/* Analytic gradients of L = sum_{t,j} dY[t,j] * Y[t,j] for the fp64 block. */
void orc_mlp_f64_backward(int64_t T, int64_t d, int64_t f,
                          const double* x, const double* W1, const double* W2, const double* W3,
                          const double* dY, double* dX, double* dW1, double* dW2, double* dW3) {
    for (int64_t i = 0; i < T * d; ++i) dX[i] = 0.0;
    for (int64_t i = 0; i < d * f; ++i) { dW1[i] = 0.0; dW2[i] = 0.0; }
    for (int64_t i = 0; i < f * d; ++i) dW3[i] = 0.0;
    for (int64_t t = 0; t < T; ++t)
        for (int64_t i = 0; i < f; ++i) {
            double u = 0.0, g = 0.0, dh = 0.0;
            for (int64_t k = 0; k < d; ++k) {
                u += x[t * d + k] * W1[k * f + i];
                g += x[t * d + k] * W2[k * f + i];
            }
            double sig = 1.0 / (1.0 + exp(-g));
            double h = u * g * sig;
            for (int64_t j = 0; j < d; ++j) {
                dh += dY[t * d + j] * W3[i * d + j];
                dW3[i * d + j] += h * dY[t * d + j];
            }
            double du = dh * g * sig;
            double dg = dh * u * (sig + g * sig * (1.0 - sig));
            for (int64_t k = 0; k < d; ++k) {
                dX[t * d + k] += du * W1[k * f + i] + dg * W2[k * f + i];
                dW1[k * f + i] += x[t * d + k] * du;
                dW2[k * f + i] += x[t * d + k] * dg;
            }
        }
}

/*
 * CPU oracle for Adam with FP8 moments (first moment E4M3, second moment E5M2).
 *
 * TEST INFRASTRUCTURE ONLY: the CUDA library never includes, links or calls this file and shares
 * no code with it.  Only the tests and the benchmark's CPU-baseline leg may use it.
 *
 * What it follows (paper = "Scaling FP8 training to trillion-token LLMs", Section 5): both Adam
 * moments are stored in FP8 - the first moment (estimate of the gradient mean) in E4M3, the second
 * moment (estimate of the uncentred gradient variance) in E5M2, because the update divides by the
 * square root of the second moment, so its smallest values matter most and it needs the wider
 * exponent range.  The paper fixes nothing else, so the update itself is the textbook one
 * (Kingma & Ba's Adam with bias correction; decoupled weight decay as in AdamW), and:
 *
 * READING A1  per-tensor scaling of each moment, like every other FP8 tensor of the recipe
 *             (Section 2): code = Q(value * scale), value = decode(code) / scale.  The scale a
 *             step stores with ("out") is given by the caller (delayed scaling: from the maximum
 *             the previous step reported); the scale it decodes with ("in") is the one the
 *             previous step stored with.
 * READING A2  rounding to nearest even, saturating (the recipe's cast everywhere else).
 * READING A3  the moments are updated in fp32 from the decoded FP8 values; the weight update
 *             uses the fp32 moments of this step (before they are rounded for storage).
 * READING A4  master weights and gradients are fp32.
 *
 * Arithmetic: fp32, one operation per statement in the order written (compile with
 * -ffp-contract=off); sqrtf and the division are correctly rounded.  The FP8 encoder / decoder are
 * this file's own (integer-bit arithmetic), written separately from the MLP oracle's so that the
 * two can be checked against each other.
 *
 * Parity status: pinned against a library Adam/AdamW in fp64 with the quantisation switched off,
 * and against the MLP oracle's independently written FP8 encoder for the stored codes.  The paper
 * prints no numeric example of a quantised optimizer step: the quantised step as a whole is
 * parity unpinned beyond those pins.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

enum {
    ADAM_Q_IDENTITY = 1,   /* keep the moments in fp32 (no FP8 storage), for the pins                   */
    ADAM_M_AS_E5M2 = 2,    /* store the first moment in E5M2 instead  } the other cells of the paper's  */
    ADAM_V_AS_E4M3 = 4     /* store the second moment in E4M3 instead } format grid, for the pins       */
};

static float bits_f(uint32_t u) { float v; memcpy(&v, &u, 4); return v; }
static uint32_t f_bits(float v) { uint32_t u; memcpy(&u, &v, 4); return u; }

/* value of an FP8 code: sign, E exponent bits (bias B), M mantissa bits */
static float fp8_value(uint8_t code, int E, int M, int B) {
    const int sign = code >> 7;
    const int ex = (code >> M) & ((1 << E) - 1);
    const int man = code & ((1 << M) - 1);
    float mag;
    if (ex == 0) mag = ldexpf((float)man, 1 - B - M);                 /* subnormal */
    else mag = ldexpf((float)((1 << M) + man), ex - B - M);
    return sign ? -mag : mag;
}

/* nearest code (ties to the even code), saturating at max_code; v finite */
static uint8_t fp8_nearest(float v, int E, int M, int B, int max_code) {
    const uint8_t sign = (f_bits(v) >> 31) ? 0x80 : 0x00;
    const float a = fabsf(v);
    /* walk the non-negative codes by bisection: codes are monotone in value */
    int lo = 0, hi = max_code;
    if (a >= fp8_value((uint8_t)max_code, E, M, B)) return sign | (uint8_t)max_code;
    while (hi - lo > 1) {
        const int mid = (lo + hi) / 2;
        if (fp8_value((uint8_t)mid, E, M, B) <= a) lo = mid; else hi = mid;
    }
    /* a lies in [value(lo), value(hi)): pick the nearer, the even code on a tie (exact in fp64) */
    const double dl = (double)a - (double)fp8_value((uint8_t)lo, E, M, B);
    const double dh = (double)fp8_value((uint8_t)hi, E, M, B) - (double)a;
    int pick;
    if (dl < dh) pick = lo; else if (dh < dl) pick = hi; else pick = (lo & 1) ? hi : lo;
    return sign | (uint8_t)pick;
}

static float dec_m(uint8_t c) { return fp8_value(c, 4, 3, 7); }            /* E4M3 */
static float dec_v(uint8_t c) { return fp8_value(c, 5, 2, 15); }           /* E5M2 */
static uint8_t enc_m(float v) { return fp8_nearest(v, 4, 3, 7, 0x7E); }    /* max 448 */
static uint8_t enc_v(float v) { return fp8_nearest(v, 5, 2, 15, 0x7B); }   /* max 57344 */

float adam_decode(int second_moment, uint8_t code) { return second_moment ? dec_v(code) : dec_m(code); }
uint8_t adam_encode(int second_moment, float v) { return second_moment ? enc_v(v) : enc_m(v); }

/* bias corrections 1 / (1 - beta^t), evaluated in fp64 and rounded once */
float adam_bias_correction(float beta, int64_t step) {
    return (float)(1.0 / (1.0 - pow((double)beta, (double)step)));
}

/*
 * One Adam step on n parameters (Section 5; textbook Adam / AdamW).
 *   w, g            fp32 master weights (updated in place) and gradients
 *   mq, vq          FP8 codes of the moments (E4M3 / E5M2), updated in place
 *   m32, v32        with ADAM_Q_IDENTITY: the moments in fp32 instead (mq, vq unused)
 *   sm_in, sv_in    scales the stored codes were written with
 *   sm_out, sv_out  scales the new codes are written with
 *   amax_m, amax_v  out: max |m|, max v of the new fp32 moments (for the next step's scales)
 */
void adam_step(int64_t n, unsigned flags, float* w, const float* g, uint8_t* mq, uint8_t* vq, float* m32, float* v32,
               float lr, float beta1, float beta2, float eps, float weight_decay, int64_t step,
               float sm_in, float sv_in, float sm_out, float sv_out, float* amax_m, float* amax_v) {
    const float omb1 = 1.0f - beta1;
    const float omb2 = 1.0f - beta2;
    const float c1 = adam_bias_correction(beta1, step);
    const float c2 = adam_bias_correction(beta2, step);
    const float inv_sm = 1.0f / sm_in;
    const float inv_sv = 1.0f / sv_in;
    float am = 0.0f, av = 0.0f;
    for (int64_t i = 0; i < n; ++i) {
        float m_prev, v_prev;
        if (flags & ADAM_Q_IDENTITY) { m_prev = m32[i]; v_prev = v32[i]; }
        else {
            m_prev = ((flags & ADAM_M_AS_E5M2) ? dec_v(mq[i]) : dec_m(mq[i])) * inv_sm;
            v_prev = ((flags & ADAM_V_AS_E4M3) ? dec_m(vq[i]) : dec_v(vq[i])) * inv_sv;
        }
        const float gi = g[i];
        const float t1 = beta1 * m_prev;
        const float t2 = omb1 * gi;
        const float m = t1 + t2;                      /* first moment: running mean of g */
        const float g2 = gi * gi;
        const float t3 = beta2 * v_prev;
        const float t4 = omb2 * g2;
        const float v = t3 + t4;                      /* second moment: running mean of g^2 */
        const float mhat = m * c1;
        const float vhat = v * c2;
        const float root = sqrtf(vhat);
        const float den = root + eps;
        float upd = mhat / den;
        if (weight_decay != 0.0f) {
            const float wdw = weight_decay * w[i];
            upd = upd + wdw;
        }
        const float stepv = lr * upd;
        w[i] = w[i] - stepv;
        if (flags & ADAM_Q_IDENTITY) { m32[i] = m; v32[i] = v; }
        else {
            const float ms = m * sm_out;
            const float vs = v * sv_out;
            mq[i] = (flags & ADAM_M_AS_E5M2) ? enc_v(ms) : enc_m(ms);
            vq[i] = (flags & ADAM_V_AS_E4M3) ? enc_m(vs) : enc_v(vs);
        }
        const float absm = fabsf(m);
        if (absm > am) am = absm;
        if (v > av) av = v;
    }
    *amax_m = am;
    *amax_v = av;
}

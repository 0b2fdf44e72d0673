/*
 * fp8mlp — FP8 Smooth-SwiGLU MLP block (forward + backward) for NVIDIA B200 (sm_100a).
 *
 * C ABI of libfp8mlp.so.  The block is the Llama-style MLP
 *     Y = (Swish(x W2) * (x W1)) W3
 * trained in FP8 as in "Scaling FP8 training to trillion-token LLMs": E4M3 operands in the
 * forward phase, E5M2 gradients in the backward phase, per-tensor scales taken from amax
 * buffers, and the paper's Smooth-SwiGLU (Section 4.4, Eq. 2): a per-channel scale s_i is
 * applied to the SwiGLU output before it is quantised and s_i^-1 is folded into row i of W3
 * before W3 is quantised.  Naming follows the paper (Section 4.1): W1 is the linear branch,
 * W2 the Swish (gate) branch, W3 the last linear layer.  T = tokens, d = d_model, f = d_ff.
 *
 * Conventions for every entry point
 *   - All tensor / amax / scale pointers are DEVICE pointers owned by the caller, row-major,
 *     16-byte aligned; the library never frees or reallocates them.  d and f must be
 *     multiples of 16 (FP8MLP_ERR_SHAPE otherwise); T is any value >= 0 and <= T_max.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work on it and return; nothing synchronises the device.  The kernels are launched with
 *     programmatic stream serialisation (each waits for its predecessor in the stream before it touches
 *     global memory), which is invisible to the caller: the stream behaves as an in-order stream, and
 *     work the caller enqueues before or after a call is ordered as usual.
 *   - Results are deterministic: the same inputs, scales and shapes give the same bits in every call.
 *   - The return value is FP8MLP_OK (0) or a negative FP8MLP_ERR_* code.  Argument errors are
 *     detected before anything is launched.  Nothing throws or aborts across this boundary.
 *   - bf16 tensors are passed as void* (2 bytes per element); FP8 codes as uint8_t.
 *   - Rounding: FP8 casts are round-to-nearest-even and saturate to the largest finite value
 *     (448 for E4M3, 57344 for E5M2); bf16 outputs are round-to-nearest-even from fp32.
 */
#ifndef FP8MLP_H_
#define FP8MLP_H_

#include <stdint.h>

#if defined(__GNUC__)
#define FP8MLP_API __attribute__((visibility("default")))
#else
#define FP8MLP_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fp8mlp_ctx fp8mlp_ctx; /* opaque: owns the FP8 operand copies, saved activations, status word */

enum {
    FP8MLP_OK = 0,
    FP8MLP_ERR_ARG = -1,     /* null pointer / bad enum value                                   */
    FP8MLP_ERR_SHAPE = -2,   /* negative size, d or f not a multiple of 16, T > T_max           */
    FP8MLP_ERR_ALIGN = -3,   /* a tensor pointer is not 16-byte aligned                         */
    FP8MLP_ERR_CUDA = -4,    /* a CUDA runtime/driver call failed (see fp8mlp_last_cuda_error)  */
    FP8MLP_ERR_TIMEOUT = -5, /* a kernel gave up on a bounded wait (device status word)         */
    FP8MLP_ERR_STATE = -6,   /* backward without a matching forward that saved activations; merged forward
                                without merged weights; the context's device is not the current one */
    FP8MLP_ERR_TOO_LARGE = -7 /* fp8mlp_forward_static: the problem does not fit the built-in scratch */
};
enum { FP8MLP_E4M3 = 0, FP8MLP_E5M2 = 1 };
enum { FP8MLP_BF16 = 0, FP8MLP_F32 = 1 };
enum {
    FP8MLP_SMOOTH = 1,       /* per-channel Smooth-SwiGLU scales; without it one per-tensor scale for H */
    FP8MLP_SAVE_FOR_BWD = 2, /* forward keeps bf16 G = x W2 and U = x W1 for backward               */
    FP8MLP_H_BF16 = 4,       /* the paper's "SwiGLU output in BF16" variant (Section 4.3): the last linear
                                layer is not quantised - H, W3 and, in backward, dY are bf16 operands and
                                scales.h / scales.w3 / scales.dy are unused; not with FP8MLP_SMOOTH        */
    FP8MLP_GU_FP8 = 8        /* with FP8MLP_SAVE_FOR_BWD: G and U are kept as E4M3 codes Q(sgu [G | U]) with one
                                per-tensor scale (scales.gu, amax.gu) instead of bf16 - half the saved bytes.
                                The paper does not say how these activations are kept; this is an option in
                                the spirit of its FP8 memory savings (Section 5).  Not with FP8MLP_H_BF16     */
};
enum {
    FP8MLP_SCALE_GIVEN = 0,              /* delayed scaling: use the scale buffers as they are  */
    FP8MLP_SCALE_FROM_CURRENT_AMAX = 1,  /* just-in-time: derive every scale from this call's data */
    FP8MLP_SCALE_GIVEN_WEIGHTS_CAST = 2  /* fp8mlp_forward only: as SCALE_GIVEN, and the context's FP8 weight buffers
                                            already hold this step's codes (fp8mlp_adam_step_cast wrote them): the
                                            weight pass is skipped, W1/W2/W3 are not read (may be null), amax.w* stay */
};
enum { /* fp8mlp_workspace: internal buffers, for inspection by tests */
    FP8MLP_WS_XQ = 0,   /* E4M3 [T,d]   quantised x                                   */
    FP8MLP_WS_W12Q = 1, /* E4M3 [d,2f]  quantised [W2 | W1]: gate columns [0,f), linear [f,2f) */
    FP8MLP_WS_W3Q = 2,  /* E4M3 [f,d]   quantised diag(s^-1) W3                        */
    FP8MLP_WS_HQ = 3,   /* E4M3 [T,f]   Q(s_i * SwiGLU)                                */
    FP8MLP_WS_GU = 4,   /* bf16 [T,2f]  saved G | U  (E4M3 [T,2f] with FP8MLP_GU_FP8)  */
    FP8MLP_WS_DYQ = 5,  /* E5M2 [T,d]   quantised dY                                   */
    FP8MLP_WS_DZQ = 6,  /* E5M2 [T,2f]  quantised [dG | dU]                            */
    FP8MLP_WS_HB = 7,   /* bf16 [T,f]   SwiGLU output, FP8MLP_H_BF16 contexts only      */
    FP8MLP_WS_W3B = 8   /* bf16 [f,d]   W3 rounded to bf16, FP8MLP_H_BF16 contexts only */
};

enum { /* phases of one step, for fp8mlp_profile_read (SMOOTH-mode kernel sequence) */
    FP8MLP_PH_QUANT_X = 0,    /* x -> E4M3 (+ amax)                                   */
    FP8MLP_PH_QUANT_W12 = 1,  /* W2, W1 -> E4M3 [W2|W1] (+ amax); with given scales W3' too */
    FP8MLP_PH_QUANT_W3 = 2,   /* diag(1/s) W3 -> E4M3 (+ amax), just-in-time scales only */
    FP8MLP_PH_GEMM1 = 3,      /* gate/up GEMM + SwiGLU / Smooth-SwiGLU epilogue       */
    FP8MLP_PH_GEMM2 = 4,      /* down projection                                      */
    FP8MLP_PH_QUANT_DY = 5,   /* dY -> E5M2 (+ amax)                                  */
    FP8MLP_PH_DGRAD2 = 6,     /* dY W3'^T + SwiGLU-backward epilogue                  */
    FP8MLP_PH_WGRAD3 = 7,     /* dW3                                                  */
    FP8MLP_PH_DGRAD1 = 8,     /* dX                                                   */
    FP8MLP_PH_WGRAD12 = 9,    /* dW2 | dW1                                            */
    FP8MLP_PH_MISC = 10,      /* amax resets, scale updates                           */
    FP8MLP_PH_COUNT = 11
};

/* The paper's scaling state (Section 2: per-tensor scaling, delayed or just-in-time; Section 4.4:
 * per-channel s_i).  Every member is a device pointer to float(s), caller-owned; the library
 * keeps no history.  A scale multiplies the tensor before the cast: code = Q(v * scale).
 *   scales.h[f]: Smooth on  -> s_i, powers of two;  Smooth off -> the per-tensor scale, repeated.
 *   amax.h[f]  : per-channel max |SwiGLU output| before scaling (Section 4.4, steps 1-2).
 *   amax.w3    : max |W3[i,j] / s_i|  (the tensor that is actually quantised).
 *   w12 / dz   : one scale for the concatenated [W2|W1] and [dG|dU] operands; amax of W1 and
 *                W2 are still reported separately.
 *   gu         : FP8MLP_GU_FP8 contexts only (may be NULL otherwise): scale of the saved [G | U] and
 *                max(|G|, |U|). */
typedef struct { float *x, *w12, *w3, *dy, *dz, *h, *gu; } fp8mlp_scales;
typedef struct { float *x, *w1, *w2, *w3, *dy, *dz, *h, *gu; } fp8mlp_amax;

/* Creates a context for T <= T_max tokens.  Allocates its workspace on the current device
 * (about T_max*(2d + 7f) + 3*d*f bytes).  Host call; may synchronise. */
FP8MLP_API int fp8mlp_create(fp8mlp_ctx** out, int64_t T_max, int64_t d_model, int64_t d_ff, uint32_t flags);
FP8MLP_API int fp8mlp_destroy(fp8mlp_ctx* ctx);
FP8MLP_API const char* fp8mlp_strerror(int code);
/* Text of the last CUDA error this thread's calls ran into ("" if none). */
FP8MLP_API const char* fp8mlp_last_cuda_error(void);
/* Synchronises `stream`, then returns FP8MLP_ERR_TIMEOUT if any kernel of this context gave up on
 * a bounded wait since the last call (and clears the word), else FP8MLP_OK. */
FP8MLP_API int fp8mlp_status(fp8mlp_ctx* ctx, void* stream);
/* Self-test of the failure path (the paper has no counterpart).  Every wait inside the kernels is bounded; this
 * launches a one-thread kernel that waits, for at most timeout_us microseconds (1 .. 1e6), on a barrier nothing
 * will ever complete.  The wait must give up, raise the context's status word and let the kernel end normally:
 * returns FP8MLP_OK if it did (the next fp8mlp_status then reports FP8MLP_ERR_TIMEOUT once and clears the word,
 * and the context stays usable), FP8MLP_ERR_STATE if the wait claimed success.  Synchronises `stream`. */
FP8MLP_API int fp8mlp_selftest_wait_timeout(fp8mlp_ctx* ctx, int64_t timeout_us, void* stream);
/* Device pointer and size in bytes of one of the FP8MLP_WS_* buffers (sized for T_max). */
FP8MLP_API int fp8mlp_workspace(fp8mlp_ctx* ctx, int which, void** ptr, int64_t* bytes);
/* Per-phase device timing (no counterpart in the paper; measurement support).  While enabled,
 * forward/backward record a CUDA event pair around every phase on the caller's stream.
 * fp8mlp_profile_read waits for the recorded events, adds their elapsed times into ms[phase]
 * (milliseconds) and the number of recorded brackets into count[phase] (both arrays of
 * FP8MLP_PH_COUNT entries, overwritten), and forgets them. */
FP8MLP_API int fp8mlp_profile_enable(fp8mlp_ctx* ctx, int on);
FP8MLP_API int fp8mlp_profile_read(fp8mlp_ctx* ctx, double* ms, int64_t* count);
/* Number of kernels this library has launched in this process so far (all contexts). */
FP8MLP_API int64_t fp8mlp_launch_count(void);

/* Per-tensor quantisation (Section 2: every tensor gets its own scale, chosen from its own
 * range of values; Section 4.4 for row_mul).
 *   dst[r, c] = Q_fmt( (src[r, c] * row_mul[r]) * scale ),  r < rows, c < cols
 *   src       rows x cols, src_dtype FP8MLP_BF16 or FP8MLP_F32, contiguous.
 *   dst       FP8 codes, leading dimension ld_dst >= cols (bytes), ld_dst % 16 == 0.
 *   row_mul   nullable; per-row multiplier (s_i^-1 for W3' = diag(s^-1) W3).
 *   scale     device float.  SCALE_GIVEN: read.  SCALE_FROM_CURRENT_AMAX: written first, as
 *             fmt_max / amax (1 if amax is 0 or not finite), then used; costs a second pass
 *             over src.
 *   amax      device float, receives max |src * row_mul|.  Nullable in SCALE_GIVEN mode,
 *             required in SCALE_FROM_CURRENT_AMAX mode.
 * cols % 16 == 0.  rows == 0 is allowed (amax becomes 0). */
FP8MLP_API int fp8mlp_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols, int fp8_fmt,
                    int scale_mode, float* scale, float* amax, const float* row_mul,
                    uint8_t* dst, int64_t ld_dst, void* stream);

/* amax -> scale bookkeeping between steps (Section 2, delayed scaling; Section 4.4 step 3).
 *   x, w3, dy : scale = fmt_max / amax.     w12 : 448 / max(amax.w1, amax.w2).
 *   h[i]      : Smooth on: largest power of two p with p * amax.h[i] <= 448; off: 448 / max_i amax.h[i].
 *   dz        : largest power of two p with p * amax.dz <= 57344.
 *   gu        : 448 / amax.gu.
 * A zero or non-finite amax gives scale 1.  Members of `amax` that are NULL are skipped together
 * with their scale. */
FP8MLP_API int fp8mlp_update_scales(fp8mlp_ctx* ctx, const fp8mlp_amax* amax, fp8mlp_scales* scales, void* stream);

/* Forward (Eq. 2 and the merge of Section 4.4; Section 6.2 for the operand formats).
 *   x_bf16 [T,d]; W1, W2 [d,f], W3 [f,d] fp32 master weights; y_bf16 [T,d] output.
 *   1. Xq = Q(x sx); [W2q|W1q] = Q(W sw12); G = Xq W2q / (sx sw12), U likewise (fp32 accumulate)
 *   2. H = U * G * sigma(G); amax.h[i] = max_t |H[t,i]|; Hq = Q(H * s_i)   (never stored unquantised)
 *   3. W3q = Q((W3[i,:] / s_i) sw3)  (Smooth off: Q(W3 sw3));  Y = Hq W3q / sw3  (Smooth off: / (sw3 sh))
 *   SCALE_GIVEN: `scales` are read; `amax` (nullable, members nullable) receives this call's maxima.
 *   SCALE_FROM_CURRENT_AMAX: both structs must be complete; scales.x/w12/h/w3 are overwritten from
 *   this call's data first (runs step 1-2 twice: once for the per-channel maxima, once for the codes).
 *   With FP8MLP_SAVE_FOR_BWD in the context flags, bf16 G and U are kept for fp8mlp_backward; with
 *   FP8MLP_GU_FP8 as well they are kept as Q_e4m3([G | U] sgu) (scales.gu required; amax.gu = max(|G|, |U|),
 *   required in SCALE_FROM_CURRENT_AMAX mode, which derives sgu = 448 / amax.gu first). */
FP8MLP_API int fp8mlp_forward(fp8mlp_ctx* ctx, int64_t T, const void* x_bf16,
                   const float* W1, const float* W2, const float* W3,
                   int scale_mode, fp8mlp_scales* scales, fp8mlp_amax* amax,
                   void* y_bf16, void* stream);

/* Backward (Section 6.2: E5M2 gradients; proof of Theorem 1 for the gate derivative
 * sigma(g) + g sigma'(g)).  Needs the preceding fp8mlp_forward on the same context, same T, with
 * FP8MLP_SAVE_FOR_BWD (FP8MLP_ERR_STATE otherwise); uses the same `scales` the forward used.
 *   dYq = Q_e5m2(dY sdy);  dH = s (.) (dYq W3q^T) / (sdy sw3)  (Smooth off: no s)
 *   dU = dH * G sigma(G);  dG = dH * U * sigma(G) (1 + G (1 - sigma(G)));  dZq = Q_e5m2([dG|dU] sdz)
 *   dX = dZq [W2q|W1q]^T / (sdz sw12)  -> bf16 [T,d]
 *   [dW2|dW1] = Xq^T dZq / (sx sdz)    -> fp32 [d,f] each, overwritten
 *   dW3[i,:] = (Hq^T dYq)[i,:] / (sdy s_i) -> fp32 [f,d], overwritten
 * Every Q is straight-through and s is a constant.  scale_mode as in forward, for dy and dz.
 * FP8MLP_GU_FP8: G and U above are the decoded saved codes times 1 / sgu (scales.gu as in the forward). */
FP8MLP_API int fp8mlp_backward(fp8mlp_ctx* ctx, int64_t T, const void* dy_bf16,
                    int scale_mode, fp8mlp_scales* scales, fp8mlp_amax* amax,
                    void* dx_bf16, float* dW1, float* dW2, float* dW3, void* stream);

/* Inference form of Smooth-SwiGLU (end of Section 4.4): once s_i is fixed it is folded into the weights,
 *   w1~_i = Q(s_i w1_i),   w3~_i = Q(s_i^-1 w3_i),
 * and the block becomes an ordinary FP8 SwiGLU MLP on the merged weights with one per-tensor scale for the
 * SwiGLU output - the per-channel scaling costs nothing at run time.
 * fp8mlp_merge_weights quantises [W2 | W1 diag(s)] (one scale, scales.w12) and diag(1/s) W3 (scales.w3) into the
 * context, once; s[f] device floats.  SCALE_GIVEN reads the two scales, SCALE_FROM_CURRENT_AMAX derives them
 * (amax.w1 = max |W1 diag(s)|, amax.w2, amax.w3 = max |diag(1/s) W3|; `amax` and its members nullable).
 * fp8mlp_forward_merged then runs  Xq = Q(x sx);  G = Xq W2q, U~ = Xq W1~q (dequantised);  H~ = U~ G sigma(G);
 * Hq = Q(H~ sh);  Y = Hq W3~q / (sw3 sh)  with sh = scales.h[0] (scales.h[f] holds sh repeated, as with
 * Smooth off).  SCALE_FROM_CURRENT_AMAX derives sx and sh from this call's data (amax.x, amax.h[f] required);
 * with SCALE_GIVEN amax and its members are optional and the per-channel maxima are only computed if amax.h is
 * given.  FP8MLP_ERR_STATE unless the context holds merged weights (fp8mlp_forward replaces them). */
FP8MLP_API int fp8mlp_merge_weights(fp8mlp_ctx* ctx, const float* W1, const float* W2, const float* W3, const float* s,
                                    int scale_mode, fp8mlp_scales* scales, fp8mlp_amax* amax, void* stream);
FP8MLP_API int fp8mlp_forward_merged(fp8mlp_ctx* ctx, int64_t T, const void* x_bf16, int scale_mode,
                                     fp8mlp_scales* scales, fp8mlp_amax* amax, void* y_bf16, void* stream);

/* Adam step with both moments stored in FP8 (Section 5: first moment E4M3, second moment E5M2 -
 * the update divides by the square root of the second moment, so its smallest values matter and it
 * needs the wider exponent range).  The step after fp8mlp_backward: it consumes dW1, dW2, dW3.
 * The update is the textbook one (bias-corrected Adam, decoupled weight decay); per parameter i,
 * in fp32 in this order - the moments, codes and maxima with one rounding per operation (they are
 * bit-exact against a plain CPU evaluation); the square root and the division of `upd` run on the
 * special-function unit and are approximate to a few 2^-23 relative, which reaches only w:
 *   m_prev = dec_e4m3(m[i]) * (1 / *scale_m_in);     v_prev = dec_e5m2(v[i]) * (1 / *scale_v_in)
 *   mi = beta1 * m_prev + (1 - beta1) * g[i];        vi = beta2 * v_prev + (1 - beta2) * (g[i] * g[i])
 *   upd = (mi * c1) / (sqrt(vi * c2) + eps) [+ weight_decay * w[i]],   c = 1 / (1 - beta^step) (fp64, rounded once)
 *   w[i] = w[i] - lr * upd
 *   m[i] = Q_e4m3(mi * *scale_m_out);                v[i] = Q_e5m2(vi * *scale_v_out)
 *   *amax_m = max |mi|;  *amax_v = max vi            (of the fp32 moments, for the next step's scales)
 * Scaling is per tensor and delayed, like the rest of the recipe: the caller keeps, per tensor, the
 * scale the stored codes were written with (`in`) and chooses the scale to write with (`out`), e.g.
 * with fp8mlp_scale_from_amax on the maxima of the previous step; `in` and `out` may be the same
 * buffer.  A zero state is codes 0 with scales 1.
 * Up to 8 tensors per call (one launch); n % 16 == 0; w, g fp32 and m, v FP8 codes, device pointers,
 * 16-byte aligned, updated in place; scales and maxima device floats.  step >= 1. */
typedef struct {
    float* w;                  /* [n] master weights, updated in place        */
    const float* g;            /* [n] gradients                                */
    uint8_t* m;                /* [n] first moment, E4M3 codes, in place       */
    uint8_t* v;                /* [n] second moment, E5M2 codes, in place      */
    int64_t n;
    const float* scale_m_in;   /* scales the stored codes were written with    */
    const float* scale_v_in;
    const float* scale_m_out;  /* scales the new codes are written with        */
    const float* scale_v_out;
    float* amax_m;             /* out: max |m|, max v of this step's moments   */
    float* amax_v;
} fp8mlp_adam_tensor;
FP8MLP_API int fp8mlp_adam_step(const fp8mlp_adam_tensor* tensors, int count, float lr, float beta1, float beta2,
                                float eps, float weight_decay, int64_t step, void* stream);
/* The same step, which also casts the updated master weights to the E4M3 operands of the next forward
 * (Section 6.2: high-precision master weights, quantised to E4M3 for the forward phase): the pass already reads
 * and writes every weight, so the cast costs one more byte written per parameter instead of a pass of its own
 * (4 bytes read + 1 written).  Per tensor i, casts[i] describes the codes (dst = null: none for this tensor):
 *   the tensor is a [n / cols, cols] matrix; code[r, c] = Q_e4m3((w_new[r, c] / row_div[r]) * *scale) at
 *   dst[r * ld_dst + c]; *amax = max |w_new[r, c] / row_div[r]|   (row_div nullable = no division; the
 *   division is a multiplication by the fp32 reciprocal, as in the forward's own quantise pass).
 * With dst pointing into the context's FP8 weight buffers (fp8mlp_workspace: W1 at FP8MLP_WS_W12Q + d_ff with
 * ld_dst = 2 d_ff, W2 at FP8MLP_WS_W12Q with ld_dst = 2 d_ff, both with scales.w12; W3 at FP8MLP_WS_W3Q with
 * scales.w3 and row_div = scales.h for Smooth-SwiGLU) the next fp8mlp_forward can be called with
 * FP8MLP_SCALE_GIVEN_WEIGHTS_CAST and skips its weight pass.  cols, ld_dst multiples of 16; dst 16-byte aligned. */
typedef struct {
    uint8_t* dst;              /* [n / cols, ld_dst] E4M3 codes, or null         */
    int64_t cols;
    int64_t ld_dst;
    const float* scale;        /* device float                                   */
    const float* row_div;      /* device [n / cols], nullable                    */
    float* amax;               /* device float out, nullable                     */
} fp8mlp_adam_cast;
FP8MLP_API int fp8mlp_adam_step_cast(const fp8mlp_adam_tensor* tensors, const fp8mlp_adam_cast* casts, int count,
                                     float lr, float beta1, float beta2, float eps, float weight_decay, int64_t step,
                                     void* stream);
/* *scale = fmt_max / *amax (Section 2, per-tensor scaling; 1 if *amax is zero or not finite).
 * fp8_fmt FP8MLP_E4M3 or FP8MLP_E5M2; both pointers device floats. */
FP8MLP_API int fp8mlp_scale_from_amax(const float* amax, int fp8_fmt, float* scale, void* stream);

/* Forward without any allocation (the paper has no counterpart; this is a deployment aid).
 *
 * Some callers cannot create a context because they cannot allocate device memory at all: a plug-in
 * running inside a host application whose own pool already owns the whole GPU (cudaMalloc would
 * fail or fight that pool), or a serving loop that must not hit the device-wide synchronisation
 * and unpredictable latency a cudaMalloc / cudaFree can bring.  For them this entry point runs the
 * same forward as fp8mlp_forward (same kernels, forward only, nothing saved for backward) with the
 * internal buffers - the FP8 copies of x, [W2|W1], W3', the SwiGLU codes and the status word -
 * placed in a fixed array that is part of the library image:
 *   FP8MLP_STATIC_SCRATCH_BYTES (4 MiB) of device memory, held by every GPU that loads the library
 *   until the process exits.  The problem fits when
 *       T*d + 3*d*f + T*f + 8*f + 4096 <= FP8MLP_STATIC_SCRATCH_BYTES
 *   (e.g. T=128, d=256, f=704, or T=256, d=512, f=1536); otherwise FP8MLP_ERR_TOO_LARGE is returned and
 *   nothing is launched.
 * Arguments are those of fp8mlp_forward, with the shape and `flags` (FP8MLP_SMOOTH or 0) passed
 * directly instead of a context.  The caller still owns x, the weights, y, `scales` and `amax`.
 * It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - Every call asks the runtime for the array's address on the current device (the array exists once
 *     per GPU; the device that is current at the call is the one used).  The first call on a device is
 *     the one that makes the runtime set the array up there: make that first call outside any stream
 *     capture.  Argument errors are found before the lookup and before anything is enqueued.
 *   - All calls share the one array, and it keeps whatever the previous call left in it; each call
 *     rewrites or clears everything it reads (the status word and the maxima start from zero).
 *     Two calls that overlap on the GPU (different streams, or different host threads without
 *     ordering) race on it: serialise them.
 *   - A bounded-wait timeout inside a kernel cannot be reported through a context here; the word is
 *     cleared at the start of every call and is not readable by the caller. */
#define FP8MLP_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
FP8MLP_API int fp8mlp_forward_static(int64_t T, int64_t d_model, int64_t d_ff, uint32_t flags,
                                     const void* x_bf16, const float* W1, const float* W2, const float* W3,
                                     int scale_mode, fp8mlp_scales* scales, fp8mlp_amax* amax,
                                     void* y_bf16, void* stream);

/* One FP8 GEMM of the kind the block is made of, exposed for tests and tuning (Section 6.2:
 * quantised operands, high-precision accumulation and output).
 *   out[m, n] = (sum_k A(m,k) B(n,k)) * ((1 / *scale_a) * (1 / *scale_b)),  fp32 accumulate,
 *   out fp32 [M,N] row-major.  scale_a / scale_b: device floats, nullable (= 1).
 *   a_kmajor != 0: A is stored [M,K] (K contiguous); == 0: stored [K,M] (M contiguous).
 *   b_kmajor != 0: B is stored [N,K];                == 0: stored [K,N].
 *   a_fmt / b_fmt: FP8MLP_E4M3 or FP8MLP_E5M2.  M, N, K multiples of 16 and > 0. */
FP8MLP_API int fp8mlp_gemm_fp8(int64_t M, int64_t N, int64_t K,
                    const uint8_t* A, int a_kmajor, int a_fmt,
                    const uint8_t* B, int b_kmajor, int b_fmt,
                    const float* scale_a, const float* scale_b, float* out, void* stream);

/* How a tensor of FP8 codes used its format's range (Section 4.3 motivates Smooth-SwiGLU with exactly this view of the
 * SwiGLU output: ordinary channels lost to underflow next to outlier channels at the top of the range):
 *   *zero_count = codes that are +0 or -0;  *top_count = codes at the largest finite magnitude (448 / 57344), which is
 *   where the saturating cast puts every value beyond it.
 * codes: device, [rows, cols] with row stride ld (cols, ld multiples of 16; 16-byte aligned), e.g. a context's
 * FP8MLP_WS_HQ buffer; the two counters are 8-byte aligned device words, overwritten.  One pass, 1 byte read per code. */
FP8MLP_API int fp8mlp_code_stats(const uint8_t* codes, int64_t rows, int64_t cols, int64_t ld, int fp8_fmt,
                                 uint64_t* zero_count, uint64_t* top_count, void* stream);

/* How the library would run one of the block's GEMMs on a device with `sm_count` SMs: host arithmetic only, nothing
 * is launched and no device is needed (for tests of the tiling rules and for tuning).  kind: 0 = fp32 output
 * (weight gradients), 1 = bf16 output (down projection, input gradient), 2 = gate/up GEMM with the SwiGLU epilogue
 * (N = d_ff), 3 = dgrad-2 with the SwiGLU-backward epilogue (N = d_ff).  with_workspace != 0: as inside a context
 * (a split contraction is possible).  Returns FP8MLP_ERR_ARG for a bad kind or a null plan. */
typedef struct {
    int cta_pairs;          /* 1: 256-row tiles on CTA pairs (cta_group::2); 0: 128-row tiles on single CTAs      */
    int tile_rows, tile_cols;
    int m_tiles, n_tiles, k_stages;      /* k_stages: 128-byte steps of the contraction                            */
    int split_k;            /* shares the contraction of a tile is cut into (1 = none)                             */
    int stages_per_share;
    int band_along_n, band_tiles;        /* rasterisation: bands of band_tiles tiles along m (0) or n (1)          */
    int staged_stores;      /* output through shared memory and bulk tensor stores (fp32: short contractions;      */
                            /* bf16: 256 x 512 tiles)                                                              */
    int64_t work_items;     /* tiles x split_k                                                                      */
} fp8mlp_gemm_plan_t;
FP8MLP_API int fp8mlp_gemm_plan(int kind, int64_t M, int64_t N, int64_t K, int sm_count, int with_workspace,
                                fp8mlp_gemm_plan_t* plan);

/* The same for bf16 operands (the unquantised last layer of FP8MLP_H_BF16 contexts): A, B bf16, no scales. */
FP8MLP_API int fp8mlp_gemm_bf16(int64_t M, int64_t N, int64_t K, const void* A, int a_kmajor, const void* B,
                                int b_kmajor, float* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FP8MLP_H_ */

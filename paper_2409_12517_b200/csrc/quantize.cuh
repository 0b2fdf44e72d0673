// Host-side launchers of the amax / cast / scale kernels (quantize.cu).
#pragma once

#include "common.cuh"

namespace fp8mlp {

// Tensors of one source dtype and FP8 format quantised together in one launch (e.g. W2 and W1, the
// two column halves of one FP8 operand, and W3'), each with its own amax and scale pointer.
constexpr int kMaxQuantSegs = 3;
struct QuantTensor {
    const void* src;        // rows x cols, contiguous, 16-byte aligned
    int64_t rows, cols;     // cols % 16 == 0
    uint8_t* dst;           // codes, leading dimension ld_dst (cast passes)
    int64_t ld_dst;
    float* amax;            // raised atomically to max |src * multiplier| (amax passes; zeroed by the caller)
    const float* row_mul;   // nullable: row r is multiplied by row_mul[r] first
    const float* row_div;   // nullable: row r is multiplied by 1 / row_div[r] first (W3' = diag(s^-1) W3)
    const float* col_mul;   // nullable: column c is multiplied by col_mul[c] first (merged w1~ = s_i w1_i)
    const float* scale;     // nullable: overrides the launch's scale for this tensor
};
// what the kernel sees
struct QuantSeg {
    const void* src; uint8_t* dst; float* amax; const float* row_mul; const float* row_div; const float* col_mul;
    const float* scale;
    int64_t ld_dst; uint32_t units_per_row, n_units;
};
struct QuantLaunch { QuantSeg seg[kMaxQuantSegs]; int nseg; int wide; uint32_t units_per_block; const float* scale; };
int run_quantize_segments(bool cast, bool amax, int src_dtype, int fmt, const QuantTensor* t, int nseg,
                          const float* scale, int sm_count, cudaStream_t st);

// One streaming pass over a rows x cols tensor (cols % 16 == 0).
//   cast: write FP8 codes dst[r*ld_dst + c] = Q((src*row_mul[r]) * *scale)
//   amax: atomically raise *amax_out to max |src*row_mul| (the caller zeroes it first)
int run_quantize_pass(bool cast, bool amax, const void* src, int src_dtype, int64_t rows, int64_t cols, int fmt,
                      const float* row_mul, const float* scale, uint8_t* dst, int64_t ld_dst, float* amax_out,
                      int sm_count, cudaStream_t st);

// dst[i] = bf16(src[i]) (n % 8 == 0), *amax_out raised to max |src| (nullable; zeroed by the caller)
int run_code_stats(const uint8_t* codes, int64_t rows, int64_t cols, int64_t ld, int fmt, unsigned long long* zero,
                   unsigned long long* top, int sm_count, cudaStream_t st);
int run_cast_bf16(const float* src, uint16_t* dst, int64_t n, float* amax_out, int sm_count, cudaStream_t st);

// *scale = fmt_max / max(*amax_a, *amax_b)  (amax_b nullable), 1 for a zero / non-finite amax
int run_scale_from_amax(int fmt, const float* amax_a, const float* amax_b, float* scale, cudaStream_t st);

struct UpdateScalesArgs {
    const float *amax_x, *amax_w1, *amax_w2, *amax_w3, *amax_dy, *amax_dz, *amax_h, *amax_gu;
    float *scale_x, *scale_w12, *scale_w3, *scale_dy, *scale_dz, *scale_h, *scale_gu;
    int64_t f;
    int smooth;
};
int run_update_scales(const UpdateScalesArgs& a, int sm_count, cudaStream_t st);


}  // namespace fp8mlp

// Host-side launchers of the amax / cast / scale kernels (quantize.cu).
#pragma once

#include "common.cuh"

namespace fp8mlp {

// One streaming pass over a rows x cols tensor (cols % 16 == 0).
//   cast: write FP8 codes dst[r*ld_dst + c] = Q((src*row_mul[r]) * *scale)
//   amax: atomically raise *amax_out to max |src*row_mul| (the caller zeroes it first)
int run_quantize_pass(bool cast, bool amax, const void* src, int src_dtype, int64_t rows, int64_t cols, int fmt,
                      const float* row_mul, const float* scale, uint8_t* dst, int64_t ld_dst, float* amax_out,
                      int sm_count, cudaStream_t st);

// *scale = fmt_max / max(*amax_a, *amax_b)  (amax_b nullable), 1 for a zero / non-finite amax
int run_scale_from_amax(int fmt, const float* amax_a, const float* amax_b, float* scale, cudaStream_t st);

struct UpdateScalesArgs {
    const float *amax_x, *amax_w1, *amax_w2, *amax_w3, *amax_dy, *amax_dz, *amax_h;
    float *scale_x, *scale_w12, *scale_w3, *scale_dy, *scale_dz, *scale_h;
    int64_t f;
    int smooth;
};
int run_update_scales(const UpdateScalesArgs& a, int sm_count, cudaStream_t st);

// out[i] = 1 / s[i]
int run_reciprocal(const float* s, float* out, int64_t n, cudaStream_t st);

}  // namespace fp8mlp

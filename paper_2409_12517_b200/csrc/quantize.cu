// amax reduction, saturating round-to-nearest-even FP8 cast, and amax -> scale kernels.
// All of them stream through HBM once: 128-bit loads and stores, warp-shuffle reductions,
// one atomic per block.  Per-tensor scaling as in the paper's Section 2; the per-row multiplier
// is the s_i^-1 of Section 4.4 (W3' = diag(s^-1) W3).
#include "quantize.cuh"

namespace fp8mlp {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float fmt_max_dev(int fmt) { return fmt == FP8MLP_E4M3 ? 448.0f : 57344.0f; }

// scale = fmt_max / amax; 1 when amax is zero or not finite (or the quotient overflows).
__device__ __forceinline__ float scale_from_amax_dev(int fmt, float amax) {
    if (!(amax > 0.0f) || isinf(amax)) return 1.0f;
    float s = __fdiv_rn(fmt_max_dev(fmt), amax);
    if (isinf(s) || isnan(s)) return 1.0f;
    return s;
}

// Largest power of two p with p * amax <= fmt_max (fmt_max = 0.875 * 2^E, E = 9 or 16).
__device__ __forceinline__ float pow2_scale_dev(int fmt, float amax) {
    if (!(amax > 0.0f) || isinf(amax)) return 1.0f;
    const int E = fmt == FP8MLP_E4M3 ? 9 : 16;
    int e;
    float m = frexpf(amax, &e);
    int k = (m <= 0.875f) ? (E - e) : (E - 1 - e);
    k = max(-100, min(100, k));
    return ldexpf(1.0f, k);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Block-wide max of non-negative values, then one atomic on the float's bit pattern.
__device__ __forceinline__ void block_atomic_max(float v, float* out) {
    __shared__ float warp_part[kThreads / 32];
    v = warp_max(v);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < 32) {
        float w = threadIdx.x < kThreads / 32 ? warp_part[threadIdx.x] : 0.0f;
        w = warp_max(w);
        if (threadIdx.x == 0 && w > 0.0f) atomicMax(reinterpret_cast<unsigned int*>(out), __float_as_uint(w));
    }
}

// Loads 16 consecutive source elements as fp32.
template <typename SRC>
__device__ __forceinline__ void load16(const SRC* p, float (&v)[16]);

template <>
__device__ __forceinline__ void load16<float>(const float* p, float (&v)[16]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint4 q = ld_global_nc_v4(p + 4 * i);
        v[4 * i + 0] = __uint_as_float(q.x);
        v[4 * i + 1] = __uint_as_float(q.y);
        v[4 * i + 2] = __uint_as_float(q.z);
        v[4 * i + 3] = __uint_as_float(q.w);
    }
}
template <>
__device__ __forceinline__ void load16<uint16_t>(const uint16_t* p, float (&v)[16]) {   // bf16 bits
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        uint4 q = ld_global_nc_v4(p + 8 * i);
        v[8 * i + 0] = bf16_lo(q.x); v[8 * i + 1] = bf16_hi(q.x);
        v[8 * i + 2] = bf16_lo(q.y); v[8 * i + 3] = bf16_hi(q.y);
        v[8 * i + 4] = bf16_lo(q.z); v[8 * i + 5] = bf16_hi(q.z);
        v[8 * i + 6] = bf16_lo(q.w); v[8 * i + 7] = bf16_hi(q.w);
    }
}

// One pass over src in chunks of 16 elements.  CAST: write FP8 codes; AMAX: reduce max |v|.
// chunks_per_row = cols / 16.  row_mul (nullable) multiplies row r before anything else.
template <typename SRC, int FMT, bool CAST, bool AMAX>
__global__ void __launch_bounds__(kThreads)
quantize_kernel(const SRC* __restrict__ src, int64_t n_chunks, int64_t chunks_per_row,
                const float* __restrict__ row_mul, const float* __restrict__ scale_ptr,
                uint8_t* __restrict__ dst, int64_t ld_dst, float* __restrict__ amax_out) {
    float scale = 1.0f;
    if constexpr (CAST) scale = *scale_ptr;
    float local_max = 0.0f;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
    for (int64_t q = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; q < n_chunks; q += stride) {
        float v[16];
        load16<SRC>(src + q * 16, v);
        const int64_t r = q / chunks_per_row;
        if (row_mul != nullptr) {
            const float m = row_mul[r];
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = __fmul_rn(v[i], m);
        }
        if constexpr (AMAX) {
#pragma unroll
            for (int i = 0; i < 16; ++i) local_max = fmaxf(local_max, fabsf(v[i]));
        }
        if constexpr (CAST) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                w[i] = cvt_fp8x4<FMT>(__fmul_rn(v[4 * i], scale), __fmul_rn(v[4 * i + 1], scale),
                                      __fmul_rn(v[4 * i + 2], scale), __fmul_rn(v[4 * i + 3], scale));
            const int64_t c = (q - r * chunks_per_row) * 16;
            st_global_v4(dst + r * ld_dst + c, w[0], w[1], w[2], w[3]);
        }
    }
    if constexpr (AMAX) block_atomic_max(local_max, amax_out);
}

// scale = fmt_max / max(amax_a, amax_b)   (amax_b nullable)
__global__ void scale_kernel(int fmt, const float* amax_a, const float* amax_b, float* scale) {
    float a = *amax_a;
    if (amax_b != nullptr) a = fmaxf(a, *amax_b);
    *scale = scale_from_amax_dev(fmt, a);
}

// One launch for the whole amax -> scale bookkeeping (see UpdateScalesArgs).
__global__ void __launch_bounds__(kThreads) update_scales_kernel(UpdateScalesArgs a) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (a.amax_x && a.scale_x) *a.scale_x = scale_from_amax_dev(FP8MLP_E4M3, *a.amax_x);
        if (a.amax_w1 && a.amax_w2 && a.scale_w12)
            *a.scale_w12 = scale_from_amax_dev(FP8MLP_E4M3, fmaxf(*a.amax_w1, *a.amax_w2));
        if (a.amax_w3 && a.scale_w3) *a.scale_w3 = scale_from_amax_dev(FP8MLP_E4M3, *a.amax_w3);
        if (a.amax_dy && a.scale_dy) *a.scale_dy = scale_from_amax_dev(FP8MLP_E5M2, *a.amax_dy);
        if (a.amax_dz && a.scale_dz) *a.scale_dz = pow2_scale_dev(FP8MLP_E5M2, *a.amax_dz);
    }
    if (a.amax_h == nullptr || a.scale_h == nullptr) return;
    if (a.smooth) {
        for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < a.f;
             i += static_cast<int64_t>(gridDim.x) * kThreads)
            a.scale_h[i] = pow2_scale_dev(FP8MLP_E4M3, a.amax_h[i]);
    } else {
        // every block reduces the whole vector (f is a few tens of thousands), then writes its share
        __shared__ float part[kThreads / 32];
        __shared__ float total;
        float m = 0.0f;
        for (int64_t i = threadIdx.x; i < a.f; i += kThreads) m = fmaxf(m, a.amax_h[i]);
        m = warp_max(m);
        if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = m;
        __syncthreads();
        if (threadIdx.x == 0) {
            float t = 0.0f;
            for (int w = 0; w < kThreads / 32; ++w) t = fmaxf(t, part[w]);
            total = scale_from_amax_dev(FP8MLP_E4M3, t);
        }
        __syncthreads();
        const float sh = total;
        for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < a.f;
             i += static_cast<int64_t>(gridDim.x) * kThreads)
            a.scale_h[i] = sh;
    }
}

// out[i] = 1 / s[i]   (row multipliers for W3' = diag(s^-1) W3)
__global__ void __launch_bounds__(kThreads) reciprocal_kernel(const float* __restrict__ s, float* __restrict__ out, int64_t n) {
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < n;
         i += static_cast<int64_t>(gridDim.x) * kThreads)
        out[i] = __fdiv_rn(1.0f, s[i]);
}

int grid_for(int64_t n_chunks, int sm_count) {
    // enough blocks to keep every SM's load queues full; a multiple of the SM count
    int64_t want = (n_chunks + kThreads - 1) / kThreads;
    int64_t cap = static_cast<int64_t>(sm_count) * 8;
    if (want < 1) want = 1;
    return static_cast<int>(want < cap ? want : cap);
}

template <typename SRC, int FMT>
int launch_pass(bool cast, bool amax, const SRC* src, int64_t n_chunks, int64_t cpr, const float* row_mul,
                const float* scale, uint8_t* dst, int64_t ld_dst, float* amax_out, int sm_count, cudaStream_t st) {
    const int grid = grid_for(n_chunks, sm_count);
    if (cast && amax)
        quantize_kernel<SRC, FMT, true, true><<<grid, kThreads, 0, st>>>(src, n_chunks, cpr, row_mul, scale, dst, ld_dst, amax_out);
    else if (cast)
        quantize_kernel<SRC, FMT, true, false><<<grid, kThreads, 0, st>>>(src, n_chunks, cpr, row_mul, scale, dst, ld_dst, amax_out);
    else
        quantize_kernel<SRC, FMT, false, true><<<grid, kThreads, 0, st>>>(src, n_chunks, cpr, row_mul, scale, dst, ld_dst, amax_out);
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}

}  // namespace

int run_quantize_pass(bool cast, bool amax, const void* src, int src_dtype, int64_t rows, int64_t cols, int fmt,
                      const float* row_mul, const float* scale, uint8_t* dst, int64_t ld_dst, float* amax_out,
                      int sm_count, cudaStream_t st) {
    const int64_t cpr = cols / 16;
    const int64_t n_chunks = rows * cpr;
    if (n_chunks == 0) return FP8MLP_OK;
    if (src_dtype == FP8MLP_F32) {
        const float* s = static_cast<const float*>(src);
        return fmt == FP8MLP_E4M3
                   ? launch_pass<float, FP8MLP_E4M3>(cast, amax, s, n_chunks, cpr, row_mul, scale, dst, ld_dst, amax_out, sm_count, st)
                   : launch_pass<float, FP8MLP_E5M2>(cast, amax, s, n_chunks, cpr, row_mul, scale, dst, ld_dst, amax_out, sm_count, st);
    }
    const uint16_t* s = static_cast<const uint16_t*>(src);
    return fmt == FP8MLP_E4M3
               ? launch_pass<uint16_t, FP8MLP_E4M3>(cast, amax, s, n_chunks, cpr, row_mul, scale, dst, ld_dst, amax_out, sm_count, st)
               : launch_pass<uint16_t, FP8MLP_E5M2>(cast, amax, s, n_chunks, cpr, row_mul, scale, dst, ld_dst, amax_out, sm_count, st);
}

int run_scale_from_amax(int fmt, const float* amax_a, const float* amax_b, float* scale, cudaStream_t st) {
    scale_kernel<<<1, 1, 0, st>>>(fmt, amax_a, amax_b, scale);
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}

int run_update_scales(const UpdateScalesArgs& a, int sm_count, cudaStream_t st) {
    int64_t blocks = a.amax_h ? (a.f + kThreads - 1) / kThreads : 1;
    if (blocks < 1) blocks = 1;
    if (blocks > sm_count) blocks = sm_count;
    update_scales_kernel<<<static_cast<int>(blocks), kThreads, 0, st>>>(a);
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}

int run_reciprocal(const float* s, float* out, int64_t n, cudaStream_t st) {
    if (n == 0) return FP8MLP_OK;
    int64_t blocks = (n + kThreads - 1) / kThreads;
    if (blocks > 1024) blocks = 1024;
    reciprocal_kernel<<<static_cast<int>(blocks), kThreads, 0, st>>>(s, out, n);
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}

}  // namespace fp8mlp

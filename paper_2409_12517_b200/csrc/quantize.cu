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

// A unit is 32 bytes of source: 8 fp32 or 16 bf16 elements.  Lane l of a warp takes unit l of the
// warp's 1 KiB, so every load instruction of a warp covers whole 128-byte lines.
template <typename SRC> struct Unit;
template <> struct Unit<float> { static constexpr int kElems = 8; };
template <> struct Unit<uint16_t> { static constexpr int kElems = 16; };

template <typename SRC>
__device__ __forceinline__ void load_unit(const SRC* p, bool wide, uint32_t (&w)[8]) {
    if (wide) {
        ld_global_nc_v8(p, w);
    } else {   // the base is only 16-byte aligned
        const uint4 lo = ld_global_nc_v4(p), hi = ld_global_nc_v4(reinterpret_cast<const uint8_t*>(p) + 16);
        w[0] = lo.x; w[1] = lo.y; w[2] = lo.z; w[3] = lo.w; w[4] = hi.x; w[5] = hi.y; w[6] = hi.z; w[7] = hi.w;
    }
}

template <typename SRC>
__device__ __forceinline__ void unpack_unit(const uint32_t (&w)[8], float (&v)[Unit<SRC>::kElems]);
template <>
__device__ __forceinline__ void unpack_unit<float>(const uint32_t (&w)[8], float (&v)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(w[i]);
}
template <>
__device__ __forceinline__ void unpack_unit<uint16_t>(const uint32_t (&w)[8], float (&v)[16]) {   // bf16 bits
#pragma unroll
    for (int i = 0; i < 8; ++i) { v[2 * i] = bf16_lo(w[i]); v[2 * i + 1] = bf16_hi(w[i]); }
}

// One pass over up to kMaxQuantSegs tensors ("segments": e.g. W2 and W1, which become the two column
// halves of one FP8 operand, and W3').  Blocks are dealt to the segments round-robin;
// kUnroll 32-byte loads in flight per thread.
// CAST: write FP8 codes; AMAX: reduce max |v| into the segment's amax.
constexpr int kUnroll = 4;
constexpr int kBlocksPerSm = 3;

template <typename SRC, int FMT, bool CAST, bool AMAX>
__global__ void __launch_bounds__(kThreads, kBlocksPerSm)
quantize_kernel(const QuantLaunch q) {
    constexpr int E = Unit<SRC>::kElems;
    grid_dependency_wait();
    grid_launch_dependents();
    const int seg_id = blockIdx.x % q.nseg;
    const QuantSeg& sg = q.seg[seg_id];
    const SRC* __restrict__ src = static_cast<const SRC*>(sg.src);
    float scale = 1.0f;
    if constexpr (CAST) scale = *sg.scale;
    float local_max = 0.0f;
    // every block of a segment owns an equal, contiguous range of units: all blocks end together
    const uint32_t begin = (blockIdx.x / q.nseg) * q.units_per_block;
    const uint32_t end = min(begin + q.units_per_block, sg.n_units);
    const bool has_row = sg.row_mul != nullptr || sg.row_div != nullptr;
    const bool flat = !has_row && sg.col_mul == nullptr && sg.ld_dst == static_cast<int64_t>(sg.units_per_row) * E;
    // (row, column unit) of this thread's next unit, advanced by kThreads units at a time: one
    // division per thread instead of one per unit
    const uint32_t upr = sg.units_per_row;
    uint32_t next_row = (begin + threadIdx.x) / upr;
    uint32_t next_col = (begin + threadIdx.x) - next_row * upr;
    for (uint32_t u0 = begin + threadIdx.x; u0 < end; u0 += kThreads * kUnroll) {
        uint32_t w[kUnroll][8];
        uint32_t row[kUnroll], col[kUnroll];
        float mul[kUnroll];
#pragma unroll
        for (int k = 0; k < kUnroll; ++k) {
            const uint32_t u = u0 + k * kThreads;
            row[k] = next_row;
            col[k] = next_col;
            if (u < end) {
                load_unit<SRC>(src + static_cast<int64_t>(u) * E, q.wide != 0, w[k]);
                if (has_row) mul[k] = sg.row_div != nullptr ? sg.row_div[next_row] : sg.row_mul[next_row];
            }
            if (!flat) {
                next_col += kThreads;
                while (next_col >= upr) { next_col -= upr; ++next_row; }
            }
        }
#pragma unroll
        for (int k = 0; k < kUnroll; ++k) {
            const uint32_t u = u0 + k * kThreads;
            if (u >= end) break;
            float v[E];
            unpack_unit<SRC>(w[k], v);
            int64_t out = static_cast<int64_t>(u) * E;
            if (!flat) {
                out = static_cast<int64_t>(row[k]) * sg.ld_dst + static_cast<int64_t>(col[k]) * E;
                if (has_row) {
                    const float m = sg.row_div != nullptr ? __fdiv_rn(1.0f, mul[k]) : mul[k];
#pragma unroll
                    for (int i = 0; i < E; ++i) v[i] = __fmul_rn(v[i], m);
                }
            }
            if (sg.col_mul != nullptr) {
                const float* cm = sg.col_mul + static_cast<int64_t>(col[k]) * E;
#pragma unroll
                for (int i = 0; i < E; ++i) v[i] = __fmul_rn(v[i], cm[i]);
            }
            if constexpr (AMAX) {
#pragma unroll
                for (int i = 0; i < E; ++i) local_max = fmaxf(local_max, fabsf(v[i]));
            }
            if constexpr (CAST) {
                uint32_t c[E / 4];
#pragma unroll
                for (int i = 0; i < E / 4; ++i)
                    c[i] = cvt_fp8x4<FMT>(__fmul_rn(v[4 * i], scale), __fmul_rn(v[4 * i + 1], scale),
                                          __fmul_rn(v[4 * i + 2], scale), __fmul_rn(v[4 * i + 3], scale));
                if constexpr (E == 16) st_global_v4(sg.dst + out, c[0], c[1], c[2], c[3]);
                else st_global_v2(sg.dst + out, c[0], c[1]);
            }
        }
    }
    if constexpr (AMAX) block_atomic_max(local_max, sg.amax);
}

// scale = fmt_max / max(amax_a, amax_b)   (amax_b nullable)
__global__ void scale_kernel(int fmt, const float* amax_a, const float* amax_b, float* scale) {
    grid_dependency_wait();
    grid_launch_dependents();
    float a = *amax_a;
    if (amax_b != nullptr) a = fmaxf(a, *amax_b);
    *scale = scale_from_amax_dev(fmt, a);
}

// One launch for the whole amax -> scale bookkeeping (see UpdateScalesArgs).
__global__ void __launch_bounds__(kThreads) update_scales_kernel(UpdateScalesArgs a) {
    grid_dependency_wait();
    grid_launch_dependents();
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (a.amax_x && a.scale_x) *a.scale_x = scale_from_amax_dev(FP8MLP_E4M3, *a.amax_x);
        if (a.amax_w1 && a.amax_w2 && a.scale_w12)
            *a.scale_w12 = scale_from_amax_dev(FP8MLP_E4M3, fmaxf(*a.amax_w1, *a.amax_w2));
        if (a.amax_w3 && a.scale_w3) *a.scale_w3 = scale_from_amax_dev(FP8MLP_E4M3, *a.amax_w3);
        if (a.amax_dy && a.scale_dy) *a.scale_dy = scale_from_amax_dev(FP8MLP_E5M2, *a.amax_dy);
        if (a.amax_dz && a.scale_dz) *a.scale_dz = pow2_scale_dev(FP8MLP_E5M2, *a.amax_dz);
        if (a.amax_gu && a.scale_gu) *a.scale_gu = scale_from_amax_dev(FP8MLP_E4M3, *a.amax_gu);
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

// fp32 -> bf16 (round to nearest even) with max |v|: the weight of a layer that is not quantised
__global__ void __launch_bounds__(kThreads) cast_bf16_kernel(const float* __restrict__ src, uint16_t* __restrict__ dst,
                                                             int64_t n_units, float* amax_out) {
    grid_dependency_wait();
    grid_launch_dependents();
    float local_max = 0.0f;
    for (int64_t u = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; u < n_units;
         u += static_cast<int64_t>(gridDim.x) * kThreads) {
        const uint4 a = ld_global_nc_v4(src + 8 * u), b = ld_global_nc_v4(src + 8 * u + 4);
        const float v[8] = {__uint_as_float(a.x), __uint_as_float(a.y), __uint_as_float(a.z), __uint_as_float(a.w),
                            __uint_as_float(b.x), __uint_as_float(b.y), __uint_as_float(b.z), __uint_as_float(b.w)};
#pragma unroll
        for (int i = 0; i < 8; ++i) local_max = fmaxf(local_max, fabsf(v[i]));
        st_global_v4(dst + 8 * u, cvt_bf16x2(v[0], v[1]), cvt_bf16x2(v[2], v[3]), cvt_bf16x2(v[4], v[5]), cvt_bf16x2(v[6], v[7]));
    }
    if (amax_out != nullptr) block_atomic_max(local_max, amax_out);
}

// Zero codes and codes at the largest finite magnitude of an FP8 tensor [rows, cols] (row stride ld, both multiples
// of 16): a unit is 16 codes; counts go to two 64-bit device counters.
__global__ void __launch_bounds__(kThreads) code_stats_kernel(const uint8_t* __restrict__ codes, int64_t n_units, int units_per_row,
                                                              int64_t ld, uint32_t top_code, unsigned long long* zero,
                                                              unsigned long long* top) {
    grid_dependency_wait();
    grid_launch_dependents();
    unsigned int z = 0, t = 0;
    for (int64_t u = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; u < n_units;
         u += static_cast<int64_t>(gridDim.x) * kThreads) {
        const int64_t r = u / units_per_row, c = u - r * units_per_row;
        const uint4 v = ld_global_nc_v4(codes + r * ld + c * 16);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t mag = w[i] & 0x7F7F7F7Fu;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const uint32_t m = (mag >> (8 * b)) & 0xFFu;
                z += m == 0u;
                t += m == top_code;
            }
        }
    }
    z = __reduce_add_sync(0xffffffffu, z);
    t = __reduce_add_sync(0xffffffffu, t);
    if ((threadIdx.x & 31) == 0) {
        if (z) atomicAdd(zero, static_cast<unsigned long long>(z));
        if (t) atomicAdd(top, static_cast<unsigned long long>(t));
    }
}

template <typename SRC, int FMT>
int launch_pass(bool cast, bool amax, const QuantLaunch& q, int grid, cudaStream_t st) {
    cudaError_t e;
    if (cast && amax) e = launch_chained(quantize_kernel<SRC, FMT, true, true>, grid, kThreads, 0, st, q);
    else if (cast) e = launch_chained(quantize_kernel<SRC, FMT, true, false>, grid, kThreads, 0, st, q);
    else e = launch_chained(quantize_kernel<SRC, FMT, false, true>, grid, kThreads, 0, st, q);
    FP8MLP_CUDA_CHECK(e);
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}

}  // namespace

int run_quantize_segments(bool cast, bool amax, int src_dtype, int fmt, const QuantTensor* t, int nseg,
                          const float* scale, int sm_count, cudaStream_t st) {
    if (nseg < 1 || nseg > kMaxQuantSegs) return FP8MLP_ERR_ARG;
    const int elems = src_dtype == FP8MLP_F32 ? 8 : 16;
    // unit indices are 32-bit: tensors beyond 2^31 units are cut into row blocks
    const int64_t kMaxUnits = int64_t(1) << 31;
    int64_t worst = 0;
    for (int i = 0; i < nseg; ++i) {
        const int64_t units = t[i].rows * (t[i].cols / elems);
        if (units > worst) worst = units;
    }
    if (worst == 0) return FP8MLP_OK;
    if (worst > kMaxUnits) {
        for (int i = 0; i < nseg; ++i) {
            const int64_t upr = t[i].cols / elems;
            if (upr == 0 || t[i].rows == 0) continue;
            const int64_t rows_per = kMaxUnits / upr > 0 ? kMaxUnits / upr : 1;
            for (int64_t r0 = 0; r0 < t[i].rows; r0 += rows_per) {
                QuantTensor part = t[i];
                part.rows = t[i].rows - r0 < rows_per ? t[i].rows - r0 : rows_per;
                part.src = static_cast<const uint8_t*>(t[i].src) + r0 * t[i].cols * (src_dtype == FP8MLP_F32 ? 4 : 2);
                if (part.dst != nullptr) part.dst += r0 * t[i].ld_dst;
                if (part.row_mul != nullptr) part.row_mul += r0;
                if (part.row_div != nullptr) part.row_div += r0;
                int rc = run_quantize_segments(cast, amax, src_dtype, fmt, &part, 1, scale, sm_count, st);
                if (rc != FP8MLP_OK) return rc;
            }
        }
        return FP8MLP_OK;
    }
    QuantLaunch q{};
    q.nseg = nseg;
    q.scale = scale;
    q.wide = 1;
    for (int i = 0; i < nseg; ++i) {
        QuantSeg& sg = q.seg[i];
        sg.src = t[i].src; sg.dst = t[i].dst; sg.amax = t[i].amax;
        sg.row_mul = t[i].row_mul; sg.row_div = t[i].row_div; sg.col_mul = t[i].col_mul;
        sg.scale = t[i].scale != nullptr ? t[i].scale : scale;
        sg.units_per_row = static_cast<uint32_t>(t[i].cols / elems);
        sg.n_units = static_cast<uint32_t>(t[i].rows * (t[i].cols / elems));
        sg.ld_dst = t[i].ld_dst;
        if (reinterpret_cast<uintptr_t>(t[i].src) & 31u) q.wide = 0;
    }
    // every resident block slot of the device gets one block (fewer for small tensors), the same number
    // for every segment, and each block an equal share of its segment, rounded up to whole warps
    int64_t per_seg = static_cast<int64_t>(sm_count) * kBlocksPerSm / nseg;
    const int64_t enough = (worst + int64_t(kThreads) * kUnroll - 1) / (int64_t(kThreads) * kUnroll);
    if (per_seg > enough) per_seg = enough;
    if (per_seg < 1) per_seg = 1;
    q.units_per_block = static_cast<uint32_t>(((worst + per_seg - 1) / per_seg + 31) / 32 * 32);
    const int grid = static_cast<int>(per_seg) * nseg;
    if (src_dtype == FP8MLP_F32)
        return fmt == FP8MLP_E4M3 ? launch_pass<float, FP8MLP_E4M3>(cast, amax, q, grid, st)
                                  : launch_pass<float, FP8MLP_E5M2>(cast, amax, q, grid, st);
    return fmt == FP8MLP_E4M3 ? launch_pass<uint16_t, FP8MLP_E4M3>(cast, amax, q, grid, st)
                              : launch_pass<uint16_t, FP8MLP_E5M2>(cast, amax, q, grid, st);
}

int run_quantize_pass(bool cast, bool amax, const void* src, int src_dtype, int64_t rows, int64_t cols, int fmt,
                      const float* row_mul, const float* scale, uint8_t* dst, int64_t ld_dst, float* amax_out,
                      int sm_count, cudaStream_t st) {
    QuantTensor t{};
    t.src = src; t.rows = rows; t.cols = cols; t.dst = dst; t.ld_dst = ld_dst; t.amax = amax_out; t.row_mul = row_mul;
    return run_quantize_segments(cast, amax, src_dtype, fmt, &t, 1, scale, sm_count, st);
}

int run_cast_bf16(const float* src, uint16_t* dst, int64_t n, float* amax_out, int sm_count, cudaStream_t st) {
    const int64_t units = n / 8;
    if (units == 0) return FP8MLP_OK;
    int64_t blocks = (units + kThreads - 1) / kThreads;
    if (blocks > int64_t(sm_count) * 8) blocks = int64_t(sm_count) * 8;
    FP8MLP_CUDA_CHECK(launch_chained(cast_bf16_kernel, static_cast<int>(blocks), kThreads, 0, st, src, dst, units, amax_out));
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}

int run_code_stats(const uint8_t* codes, int64_t rows, int64_t cols, int64_t ld, int fmt, unsigned long long* zero,
                   unsigned long long* top, int sm_count, cudaStream_t st) {
    FP8MLP_CUDA_CHECK(cudaMemsetAsync(zero, 0, sizeof(unsigned long long), st));
    FP8MLP_CUDA_CHECK(cudaMemsetAsync(top, 0, sizeof(unsigned long long), st));
    const int64_t units = rows * (cols / 16);
    if (units == 0) return FP8MLP_OK;
    int64_t blocks = (units + kThreads - 1) / kThreads;
    if (blocks > int64_t(sm_count) * 8) blocks = int64_t(sm_count) * 8;
    FP8MLP_CUDA_CHECK(launch_chained(code_stats_kernel, static_cast<int>(blocks), kThreads, 0, st, codes, units,
                                     static_cast<int>(cols / 16), ld, fmt == FP8MLP_E4M3 ? 0x7Eu : 0x7Bu, zero, top));
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}

int run_scale_from_amax(int fmt, const float* amax_a, const float* amax_b, float* scale, cudaStream_t st) {
    FP8MLP_CUDA_CHECK(launch_chained(scale_kernel, 1, 1, 0, st, fmt, amax_a, amax_b, scale));
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}

int run_update_scales(const UpdateScalesArgs& a, int sm_count, cudaStream_t st) {
    int64_t blocks = a.amax_h ? (a.f + kThreads - 1) / kThreads : 1;
    if (blocks < 1) blocks = 1;
    if (blocks > sm_count) blocks = sm_count;
    FP8MLP_CUDA_CHECK(launch_chained(update_scales_kernel, static_cast<int>(blocks), kThreads, 0, st, a));
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}

}  // namespace fp8mlp

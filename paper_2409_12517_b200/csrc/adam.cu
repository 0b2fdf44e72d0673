// Adam step with both moments stored in FP8 (Section 5 of the paper: first moment E4M3, second
// moment E5M2), fused into one streaming pass: read g, w and the two code arrays, write w and the
// new codes.  16 bytes per parameter and step instead of 28 with fp32 moments.
// Per-tensor scales (decode with the scale the codes were written with, encode with the scale the
// caller chose for this step), maxima of the new moments reported for the next step's scales.
#include <cmath>

#include "common.cuh"

namespace fp8mlp {

namespace {

constexpr int kAdamThreads = 256;
constexpr int kAdamBlocksPerSm = 2;
constexpr int kAdamUnroll = 2;
constexpr int kAdamMaxTensors = 8;

struct AdamSeg {
    float* w; const float* g; uint8_t* m; uint8_t* v;
    const float *sm_in, *sv_in, *sm_out, *sv_out;
    float *amax_m, *amax_v;
    uint32_t n_units, units_per_block;     // a unit is 8 parameters
    // optional cast of the updated weights to the E4M3 operand of the next forward
    uint8_t* q_dst; int64_t q_ld; uint32_t q_units_per_row; const float* q_scale; const float* q_row_div; float* q_amax;
};
struct AdamLaunch {
    AdamSeg seg[kAdamMaxTensors];
    int nseg, wide;
    float lr, beta1, beta2, omb1, omb2, c1, c2, eps, wd;
};
struct AdamZero { float* p[3 * kAdamMaxTensors]; };

__global__ void adam_zero_kernel(AdamZero z) {
    grid_dependency_wait();
    grid_launch_dependents();
    if (threadIdx.x < 3 * kAdamMaxTensors && z.p[threadIdx.x] != nullptr) *z.p[threadIdx.x] = 0.0f;
}

// 8 FP8 codes (two 32-bit words) -> 8 floats, exactly
template <int FMT>
__device__ __forceinline__ void decode8(uint32_t lo, uint32_t hi, float (&out)[8]) {
    const uint32_t w[2] = {lo, hi};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint16_t pair = static_cast<uint16_t>(w[i >> 1] >> (16 * (i & 1)));
        uint32_t h2;
        if constexpr (FMT == FP8MLP_E4M3) asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(pair));
        else asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h2) : "h"(pair));
        float a, b;
        asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, h;\n\t}" : "=f"(a), "=f"(b) : "r"(h2));
        out[2 * i] = a;
        out[2 * i + 1] = b;
    }
}

__device__ __forceinline__ float warp_max_f(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// CAST: the pass also writes the E4M3 codes of the updated weights (scale, optional per-row divisor: exactly the
// arithmetic of the quantise pass of the forward, which the next forward can then skip) and their maximum.
template <bool CAST>
__global__ void __launch_bounds__(kAdamThreads, kAdamBlocksPerSm) adam_kernel(const AdamLaunch q) {
    grid_dependency_wait();
    grid_launch_dependents();
    const int seg_id = blockIdx.x % q.nseg;
    const AdamSeg& sg = q.seg[seg_id];
    const bool cast = CAST && sg.q_dst != nullptr;
    const float q_scale = cast ? *sg.q_scale : 1.0f;
    float max_q = 0.0f;
    const uint32_t begin = (blockIdx.x / q.nseg) * sg.units_per_block;
    const uint32_t end = min(begin + sg.units_per_block, sg.n_units);
    const float inv_sm = __fdiv_rn(1.0f, *sg.sm_in), inv_sv = __fdiv_rn(1.0f, *sg.sv_in);
    const float sm_out = *sg.sm_out, sv_out = *sg.sv_out;
    float max_m = 0.0f, max_v = 0.0f;
    for (uint32_t u0 = begin + threadIdx.x; u0 < end; u0 += kAdamThreads * kAdamUnroll) {
        uint32_t gw[kAdamUnroll][8], ww[kAdamUnroll][8];
        uint2 mc[kAdamUnroll], vc[kAdamUnroll];
#pragma unroll
        for (int k = 0; k < kAdamUnroll; ++k) {
            const uint32_t u = u0 + k * kAdamThreads;
            if (u < end) {
                const int64_t e0 = static_cast<int64_t>(u) * 8;
                if (q.wide) {
                    ld_global_nc_v8(sg.g + e0, gw[k]);
                    ld_global_v8(sg.w + e0, ww[k]);
                } else {
                    const uint4 a = ld_global_nc_v4(sg.g + e0), b = ld_global_nc_v4(sg.g + e0 + 4);
                    const uint4 c = *reinterpret_cast<const uint4*>(sg.w + e0), d = *reinterpret_cast<const uint4*>(sg.w + e0 + 4);
                    gw[k][0] = a.x; gw[k][1] = a.y; gw[k][2] = a.z; gw[k][3] = a.w;
                    gw[k][4] = b.x; gw[k][5] = b.y; gw[k][6] = b.z; gw[k][7] = b.w;
                    ww[k][0] = c.x; ww[k][1] = c.y; ww[k][2] = c.z; ww[k][3] = c.w;
                    ww[k][4] = d.x; ww[k][5] = d.y; ww[k][6] = d.z; ww[k][7] = d.w;
                }
                mc[k] = *reinterpret_cast<const uint2*>(sg.m + e0);
                vc[k] = *reinterpret_cast<const uint2*>(sg.v + e0);
            }
        }
#pragma unroll
        for (int k = 0; k < kAdamUnroll; ++k) {
            const uint32_t u = u0 + k * kAdamThreads;
            if (u >= end) break;
            const int64_t e0 = static_cast<int64_t>(u) * 8;
            float mp[8], vp[8], ms[8], vs[8];
            uint32_t wn[8];
            decode8<FP8MLP_E4M3>(mc[k].x, mc[k].y, mp);
            decode8<FP8MLP_E5M2>(vc[k].x, vc[k].y, vp);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float g = __uint_as_float(gw[k][i]);
                const float w = __uint_as_float(ww[k][i]);
                const float m_prev = __fmul_rn(mp[i], inv_sm);
                const float v_prev = __fmul_rn(vp[i], inv_sv);
                const float m = __fadd_rn(__fmul_rn(q.beta1, m_prev), __fmul_rn(q.omb1, g));
                const float v = __fadd_rn(__fmul_rn(q.beta2, v_prev), __fmul_rn(q.omb2, __fmul_rn(g, g)));
                const float mhat = __fmul_rn(m, q.c1);
                const float vhat = __fmul_rn(v, q.c2);
                // square root and division on the special-function unit (each within a few 2^-23 relative):
                // correctly rounded versions cost ~25 more instructions per parameter, which at the clock
                // the power cap leaves makes the pass instruction-bound instead of HBM-bound.  The moments
                // and their codes do not depend on them; the weight moves by <= 1e-6 of its update.
                float root, upd;
                asm("sqrt.approx.f32 %0, %1;" : "=f"(root) : "f"(vhat));
                const float den = __fadd_rn(root, q.eps);
                asm("div.approx.f32 %0, %1, %2;" : "=f"(upd) : "f"(mhat), "f"(den));
                if (q.wd != 0.0f) upd = __fadd_rn(upd, __fmul_rn(q.wd, w));
                wn[i] = __float_as_uint(__fsub_rn(w, __fmul_rn(q.lr, upd)));
                ms[i] = __fmul_rn(m, sm_out);
                vs[i] = __fmul_rn(v, sv_out);
                max_m = fmaxf(max_m, fabsf(m));
                max_v = fmaxf(max_v, v);
            }
            if (q.wide) {
                st_global_v8(sg.w + e0, wn);
            } else {
                st_global_v4(sg.w + e0, wn[0], wn[1], wn[2], wn[3]);
                st_global_v4(sg.w + e0 + 4, wn[4], wn[5], wn[6], wn[7]);
            }
            if (CAST && cast) {
                const uint32_t r = u / sg.q_units_per_row, cu = u - r * sg.q_units_per_row;
                float t[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) t[i] = __uint_as_float(wn[i]);
                if (sg.q_row_div != nullptr) {
                    const float inv = __fdiv_rn(1.0f, sg.q_row_div[r]);
#pragma unroll
                    for (int i = 0; i < 8; ++i) t[i] = __fmul_rn(t[i], inv);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) max_q = fmaxf(max_q, fabsf(t[i]));
                st_global_v2(sg.q_dst + static_cast<int64_t>(r) * sg.q_ld + static_cast<int64_t>(cu) * 8,
                             cvt_fp8x4<FP8MLP_E4M3>(__fmul_rn(t[0], q_scale), __fmul_rn(t[1], q_scale), __fmul_rn(t[2], q_scale), __fmul_rn(t[3], q_scale)),
                             cvt_fp8x4<FP8MLP_E4M3>(__fmul_rn(t[4], q_scale), __fmul_rn(t[5], q_scale), __fmul_rn(t[6], q_scale), __fmul_rn(t[7], q_scale)));
            }
            st_global_v2(sg.m + e0, cvt_fp8x4<FP8MLP_E4M3>(ms[0], ms[1], ms[2], ms[3]), cvt_fp8x4<FP8MLP_E4M3>(ms[4], ms[5], ms[6], ms[7]));
            st_global_v2(sg.v + e0, cvt_fp8x4<FP8MLP_E5M2>(vs[0], vs[1], vs[2], vs[3]), cvt_fp8x4<FP8MLP_E5M2>(vs[4], vs[5], vs[6], vs[7]));
        }
    }
    // block-wide maxima (non-negative: their bit patterns order like unsigned integers)
    __shared__ float part[3][kAdamThreads / 32];
    max_m = warp_max_f(max_m);
    max_v = warp_max_f(max_v);
    max_q = warp_max_f(max_q);
    if ((threadIdx.x & 31) == 0) { part[0][threadIdx.x >> 5] = max_m; part[1][threadIdx.x >> 5] = max_v; part[2][threadIdx.x >> 5] = max_q; }
    __syncthreads();
    if (threadIdx.x < 32) {
        float a = threadIdx.x < kAdamThreads / 32 ? part[0][threadIdx.x] : 0.0f;
        float b = threadIdx.x < kAdamThreads / 32 ? part[1][threadIdx.x] : 0.0f;
        float c = threadIdx.x < kAdamThreads / 32 ? part[2][threadIdx.x] : 0.0f;
        a = warp_max_f(a);
        b = warp_max_f(b);
        c = warp_max_f(c);
        if (threadIdx.x == 0) {
            if (a > 0.0f) atomicMax(reinterpret_cast<unsigned int*>(sg.amax_m), __float_as_uint(a));
            if (b > 0.0f) atomicMax(reinterpret_cast<unsigned int*>(sg.amax_v), __float_as_uint(b));
            if (CAST && cast && sg.q_amax != nullptr && c > 0.0f) atomicMax(reinterpret_cast<unsigned int*>(sg.q_amax), __float_as_uint(c));
        }
    }
}

bool al(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace

}  // namespace fp8mlp

using namespace fp8mlp;

namespace {
int adam_launch(const fp8mlp_adam_tensor* t, const fp8mlp_adam_cast* casts, int count, float lr, float beta1, float beta2,
                float eps, float weight_decay, int64_t step, void* stream) {
    if (t == nullptr || count < 1 || count > kAdamMaxTensors) return FP8MLP_ERR_ARG;
    for (int i = 0; casts != nullptr && i < count; ++i) {
        const fp8mlp_adam_cast& c = casts[i];
        if (c.dst == nullptr) continue;
        if (c.scale == nullptr) return FP8MLP_ERR_ARG;
        if (c.cols <= 0 || c.cols % 16 != 0 || c.ld_dst < c.cols || c.ld_dst % 16 != 0 || t[i].n % c.cols != 0) return FP8MLP_ERR_SHAPE;
        if (!al(c.dst, 16)) return FP8MLP_ERR_ALIGN;
    }
    if (step < 1 || !(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f)) return FP8MLP_ERR_ARG;
    int64_t worst = 0;
    for (int i = 0; i < count; ++i) {
        const fp8mlp_adam_tensor& a = t[i];
        if (a.n < 0 || a.n % 16 != 0 || a.n / 8 >= (int64_t(1) << 31)) return FP8MLP_ERR_SHAPE;
        if (a.scale_m_in == nullptr || a.scale_v_in == nullptr || a.scale_m_out == nullptr || a.scale_v_out == nullptr ||
            a.amax_m == nullptr || a.amax_v == nullptr)
            return FP8MLP_ERR_ARG;
        if (a.n > 0 && (a.w == nullptr || a.g == nullptr || a.m == nullptr || a.v == nullptr)) return FP8MLP_ERR_ARG;
        if (!al(a.w, 16) || !al(a.g, 16) || !al(a.m, 16) || !al(a.v, 16)) return FP8MLP_ERR_ALIGN;
        if (a.n / 8 > worst) worst = a.n / 8;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    FP8MLP_CUDA_CHECK(cudaGetDevice(&dev));
    FP8MLP_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    AdamZero z{};
    for (int i = 0; i < count; ++i) {
        z.p[3 * i] = t[i].amax_m; z.p[3 * i + 1] = t[i].amax_v;
        z.p[3 * i + 2] = (casts != nullptr && casts[i].dst != nullptr) ? casts[i].amax : nullptr;
    }
    FP8MLP_CUDA_CHECK(launch_chained(adam_zero_kernel, 1, 32, 0, st, z));
    FP8MLP_LAUNCH_CHECK();
    if (worst == 0) return FP8MLP_OK;

    AdamLaunch q{};
    q.nseg = count;
    q.wide = 1;
    q.lr = lr; q.beta1 = beta1; q.beta2 = beta2; q.eps = eps; q.wd = weight_decay;
    q.omb1 = 1.0f - beta1;
    q.omb2 = 1.0f - beta2;
    // bias corrections 1 / (1 - beta^t), evaluated in fp64 and rounded once
    q.c1 = static_cast<float>(1.0 / (1.0 - std::pow(static_cast<double>(beta1), static_cast<double>(step))));
    q.c2 = static_cast<float>(1.0 / (1.0 - std::pow(static_cast<double>(beta2), static_cast<double>(step))));
    // every resident block slot gets one block, the same number per tensor, each an equal share
    int64_t per_seg = static_cast<int64_t>(sms) * kAdamBlocksPerSm / count;
    const int64_t enough = (worst + int64_t(kAdamThreads) * kAdamUnroll - 1) / (int64_t(kAdamThreads) * kAdamUnroll);
    if (per_seg > enough) per_seg = enough;
    if (per_seg < 1) per_seg = 1;
    for (int i = 0; i < count; ++i) {
        AdamSeg& sg = q.seg[i];
        sg.w = t[i].w; sg.g = t[i].g; sg.m = t[i].m; sg.v = t[i].v;
        sg.sm_in = t[i].scale_m_in; sg.sv_in = t[i].scale_v_in; sg.sm_out = t[i].scale_m_out; sg.sv_out = t[i].scale_v_out;
        sg.amax_m = t[i].amax_m; sg.amax_v = t[i].amax_v;
        sg.n_units = static_cast<uint32_t>(t[i].n / 8);
        sg.units_per_block = static_cast<uint32_t>(((t[i].n / 8 + per_seg - 1) / per_seg + 31) / 32 * 32);
        if (!al(t[i].w, 32) || !al(t[i].g, 32)) q.wide = 0;
        if (casts != nullptr && casts[i].dst != nullptr) {
            sg.q_dst = casts[i].dst; sg.q_ld = casts[i].ld_dst; sg.q_units_per_row = static_cast<uint32_t>(casts[i].cols / 8);
            sg.q_scale = casts[i].scale; sg.q_row_div = casts[i].row_div; sg.q_amax = casts[i].amax;
        }
    }
    const int grid = static_cast<int>(per_seg) * count;
    if (casts != nullptr) FP8MLP_CUDA_CHECK(launch_chained(adam_kernel<true>, grid, kAdamThreads, 0, st, q));
    else FP8MLP_CUDA_CHECK(launch_chained(adam_kernel<false>, grid, kAdamThreads, 0, st, q));
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}
}  // namespace

extern "C" int fp8mlp_adam_step(const fp8mlp_adam_tensor* t, int count, float lr, float beta1, float beta2, float eps,
                                float weight_decay, int64_t step, void* stream) {
    return adam_launch(t, nullptr, count, lr, beta1, beta2, eps, weight_decay, step, stream);
}

extern "C" int fp8mlp_adam_step_cast(const fp8mlp_adam_tensor* t, const fp8mlp_adam_cast* casts, int count, float lr,
                                     float beta1, float beta2, float eps, float weight_decay, int64_t step, void* stream) {
    if (casts == nullptr) return FP8MLP_ERR_ARG;
    return adam_launch(t, casts, count, lr, beta1, beta2, eps, weight_decay, step, stream);
}

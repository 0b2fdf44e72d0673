// C ABI of libfp8mlp (declared in include/fp8mlp.h): argument validation, the context's
// workspace, and the sequence of kernels that makes up forward and backward.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "gemm.cuh"
#include "quantize.cuh"

namespace fp8mlp {

namespace {
thread_local char g_last_error[512] = "";
std::atomic<int64_t> g_launches{0};
}  // namespace

void set_cuda_error(const char* what, cudaError_t e) {
    std::snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, cudaGetErrorString(e));
}
void set_cuda_error_str(const char* what, const char* msg) {
    std::snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, msg);
}
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

// Sets up to 8 device floats and one vector of floats to zero in one launch (amax accumulators).
struct ZeroList { float* p[8]; float* vec; int64_t n; unsigned int* words; int n_words; };
__global__ void zero_floats_kernel(ZeroList z) {
    grid_dependency_wait();
    grid_launch_dependents();
    if (blockIdx.x == 0 && threadIdx.x < 8 && z.p[threadIdx.x] != nullptr) *z.p[threadIdx.x] = 0.0f;
    if (blockIdx.x == 0)        // the split-contraction counters (a kernel that gave up on a wait may have left some set)
        for (int i = threadIdx.x; i < z.n_words; i += blockDim.x) z.words[i] = 0u;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < z.n;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x)
        z.vec[i] = 0.0f;
}

// Self-test of the bounded waits: one thread waits on a barrier that nothing ever completes, with
// a short limit.  The wait must give up, raise the status word and let the kernel end normally.
__global__ void wait_selftest_kernel(int* status, uint64_t timeout_ns, int* gave_up) {
    __shared__ uint64_t never;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&never), 1);
        abort_flag = 0;
        mbar_init_fence();
        const bool got = mbar_wait(smem_u32(&never), 0, &abort_flag, status, timeout_ns);
        *gave_up = got ? 0 : 1;
    }
}

}  // namespace fp8mlp

using namespace fp8mlp;

struct fp8mlp_ctx {
    int64_t T_max, d, f;
    uint32_t flags;
    int device, sm_count;
    uint8_t *xq, *w12q, *w3q, *hq, *dyq, *dzq;
    uint16_t* gu;
    uint16_t *hb, *w3b;  // FP8MLP_H_BF16: the SwiGLU output and W3 in bf16 (operands of the unquantised last layer)
    float* splitk_ws;           // fp32 partial tiles of a split contraction (small problems), kSplitFloats of them
    unsigned int* splitk_cnt;   // their arrival counters, kSplitWords words
    float* dummy;     // [8 + f] sinks for amax outputs the caller did not ask for
    int* status;      // bounded-wait status word
    int64_t saved_T;  // tokens of the last forward that saved activations, -1 if none
    bool merged;      // the FP8 weights hold the inference-merged form (fp8mlp_merge_weights)
    int64_t bytes[9];
    // per-phase timing
    bool profiling;
    struct Bracket { int phase; cudaEvent_t e0, e1; };
    std::vector<Bracket>* brackets;      // recorded, not yet read
    std::vector<cudaEvent_t>* free_events;
};

namespace {

// Records an event pair around a phase of forward/backward when profiling is on.
struct PhaseTimer {
    fp8mlp_ctx* c;
    cudaStream_t st;
    fp8mlp_ctx::Bracket b;
    bool on;
    static cudaEvent_t take(fp8mlp_ctx* c) {
        if (!c->free_events->empty()) { cudaEvent_t e = c->free_events->back(); c->free_events->pop_back(); return e; }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
    PhaseTimer(fp8mlp_ctx* ctx, int phase, cudaStream_t s) : c(ctx), st(s), on(ctx->profiling) {
        if (!on) return;
        b.phase = phase; b.e0 = take(c); b.e1 = take(c);
        if (b.e0 == nullptr || b.e1 == nullptr) { on = false; return; }
        cudaEventRecord(b.e0, st);
    }
    ~PhaseTimer() {
        if (!on) return;
        cudaEventRecord(b.e1, st);
        c->brackets->push_back(b);
    }
};

// A context's buffers live on the device that was current when it was created: calls on it must be
// made with that device current.
bool on_device_of(const fp8mlp_ctx* c) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == c->device;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// A split contraction is only made when the problem has fewer tiles than the device has CTA pairs, so its shares
// number at most that many 256 x 256 tiles; 128 pairs cover every device this library runs on.
constexpr int64_t kSplitFloats = int64_t(128) * 256 * 256;
constexpr int kSplitWords = 128 * 16;

int zero_floats(const fp8mlp_ctx* c, std::initializer_list<float*> ptrs, cudaStream_t st, float* vec = nullptr, int64_t n_vec = 0) {
    ZeroList z{};
    int n = 0;
    for (float* p : ptrs) z.p[n++] = p;
    z.vec = vec;
    z.n = vec != nullptr ? n_vec : 0;
    if (c != nullptr && c->splitk_cnt != nullptr) { z.words = c->splitk_cnt; z.n_words = kSplitWords; }
    const int blocks = z.n > 256 ? static_cast<int>((z.n + 255) / 256 < 256 ? (z.n + 255) / 256 : 256) : 1;
    FP8MLP_CUDA_CHECK(launch_chained(zero_floats_kernel, blocks, 256, 0, st, z));
    FP8MLP_LAUNCH_CHECK();
    return FP8MLP_OK;
}

#define FP8MLP_TRY(expr)                    \
    do {                                    \
        int rc__ = (expr);                  \
        if (rc__ != FP8MLP_OK) return rc__; \
    } while (0)

// amax + cast of one tensor, in either scale mode.  amax must be non-null.
// row_mul / row_div (both nullable): per-row multiplier, or per-row divisor (W3' = diag(s^-1) W3).
int quantize_tensor(const void* src, int dtype, int64_t rows, int64_t cols, int fmt, int mode, float* scale,
                    float* amax, const float* amax_other, const float* row_mul, const float* row_div, uint8_t* dst,
                    int64_t ld_dst, int sm_count, cudaStream_t st) {
    QuantTensor t{};
    t.src = src; t.rows = rows; t.cols = cols; t.dst = dst; t.ld_dst = ld_dst; t.amax = amax;
    t.row_mul = row_mul; t.row_div = row_div;
    if (mode == FP8MLP_SCALE_FROM_CURRENT_AMAX) {
        FP8MLP_TRY(run_quantize_segments(false, true, dtype, fmt, &t, 1, nullptr, sm_count, st));
        FP8MLP_TRY(run_scale_from_amax(fmt, amax, amax_other, scale, st));
        return run_quantize_segments(true, false, dtype, fmt, &t, 1, scale, sm_count, st);
    }
    return run_quantize_segments(true, true, dtype, fmt, &t, 1, scale, sm_count, st);
}

GemmArgs base_args(fp8mlp_ctx* c, int M, int N, int K) {
    GemmArgs a{};
    a.M = M; a.N = N; a.K = K;
    a.n_tile_cols = kBlockN;
    a.b1_offset = 128;
    a.status = c ? c->status : nullptr;
    if (c != nullptr && c->splitk_ws != nullptr && c->splitk_cnt != nullptr) {
        a.partial = c->splitk_ws; a.partial_floats = kSplitFloats;
        a.tile_counters = c->splitk_cnt; a.counter_words = kSplitWords;
    }
    a.n_split = N;
    a.ld_out = N;
    a.store = 1;
    return a;
}

// [W2 | W1] -> E4M3 codes in the [d, 2f] layout (gate columns first), one scale for both halves
int quantize_w12(fp8mlp_ctx* c, const float* W1, const float* W2, int mode, float* scale, float* a_w1, float* a_w2,
                 cudaStream_t st) {
    const int64_t d = c->d, f = c->f;
    const int sms = c->sm_count;
    if (mode == FP8MLP_SCALE_FROM_CURRENT_AMAX) {
        QuantTensor t[2] = {};
        t[0].src = W2; t[0].rows = d; t[0].cols = f; t[0].dst = c->w12q; t[0].ld_dst = 2 * f; t[0].amax = a_w2;
        t[1].src = W1; t[1].rows = d; t[1].cols = f; t[1].dst = c->w12q + f; t[1].ld_dst = 2 * f; t[1].amax = a_w1;
        FP8MLP_TRY(run_quantize_segments(false, true, FP8MLP_F32, FP8MLP_E4M3, t, 2, nullptr, sms, st));
        FP8MLP_TRY(run_scale_from_amax(FP8MLP_E4M3, a_w1, a_w2, scale, st));
        return run_quantize_segments(true, false, FP8MLP_F32, FP8MLP_E4M3, t, 2, scale, sms, st);
    }
    QuantTensor t[2] = {};
    t[0].src = W2; t[0].rows = d; t[0].cols = f; t[0].dst = c->w12q; t[0].ld_dst = 2 * f; t[0].amax = a_w2;
    t[1].src = W1; t[1].rows = d; t[1].cols = f; t[1].dst = c->w12q + f; t[1].ld_dst = 2 * f; t[1].amax = a_w1;
    return run_quantize_segments(true, true, FP8MLP_F32, FP8MLP_E4M3, t, 2, scale, sms, st);
}

// G|U = Xq [W2q|W1q] with the SwiGLU / Smooth-SwiGLU epilogue
int gemm1_swiglu(fp8mlp_ctx* c, int64_t T, const fp8mlp_scales* s, float* amax_h, int store, cudaStream_t st,
                 bool save_gu = true, float* amax_gu = nullptr) {
    CUtensorMap tmA, tmB0, tmB1;
    FP8MLP_TRY(make_tmap_u8(&tmA, c->xq, c->d, T, c->d));
    FP8MLP_TRY(make_tmap_u8(&tmB0, c->w12q, c->f, c->d, 2 * c->f));
    FP8MLP_TRY(make_tmap_u8(&tmB1, c->w12q + c->f, c->f, c->d, 2 * c->f));
    GemmArgs a = base_args(c, static_cast<int>(T), static_cast<int>(c->f), static_cast<int>(c->d));
    a.n_tile_cols = 128;
    a.b1_offset = 0;
    a.s0 = s->x; a.s1 = s->w12;
    a.s_h = s->h;
    a.store = store;
    a.hq = c->hq;
    a.hb = (c->flags & FP8MLP_H_BF16) ? c->hb : nullptr;
    a.gu = (save_gu && (c->flags & FP8MLP_SAVE_FOR_BWD)) ? c->gu : nullptr;
    if (a.gu != nullptr && (c->flags & FP8MLP_GU_FP8)) {      // kept as E4M3 codes instead
        a.gu8 = reinterpret_cast<uint8_t*>(c->gu);
        a.gu = nullptr;
        a.s_gu = s->gu;
        a.amax_gu = reinterpret_cast<unsigned int*>(amax_gu);
    }
    a.amax_h = reinterpret_cast<unsigned int*>(amax_h);
    return launch_gemm(EPI_SWIGLU_FWD, false, true, FP8MLP_E4M3, FP8MLP_E4M3, tmA, tmB0, tmB1, a, c->sm_count, st);
}

// Everything fp8mlp_forward can refuse before it enqueues anything.
int check_forward_args(const fp8mlp_ctx* c, int64_t T, const void* x, const float* W1, const float* W2, const float* W3,
                       int mode, const fp8mlp_scales* sc, const fp8mlp_amax* am, const void* y) {
    if (c == nullptr || sc == nullptr) return FP8MLP_ERR_ARG;
    const bool cast_done = mode == FP8MLP_SCALE_GIVEN_WEIGHTS_CAST;      // the FP8 weight buffers are already filled
    if (!cast_done && (W1 == nullptr || W2 == nullptr || W3 == nullptr)) return FP8MLP_ERR_ARG;
    if (mode != FP8MLP_SCALE_GIVEN && mode != FP8MLP_SCALE_FROM_CURRENT_AMAX && !cast_done) return FP8MLP_ERR_ARG;
    if (cast_done && (c->flags & FP8MLP_H_BF16)) return FP8MLP_ERR_ARG;  // that variant keeps W3 in bf16, not as codes
    if (!on_device_of(c)) return FP8MLP_ERR_STATE;
    if (T < 0 || T > c->T_max) return FP8MLP_ERR_SHAPE;
    if (T > 0 && (x == nullptr || y == nullptr)) return FP8MLP_ERR_ARG;
    if (sc->x == nullptr || sc->w12 == nullptr || sc->w3 == nullptr || sc->h == nullptr) return FP8MLP_ERR_ARG;
    if (mode == FP8MLP_SCALE_FROM_CURRENT_AMAX &&
        (am == nullptr || am->x == nullptr || am->w1 == nullptr || am->w2 == nullptr || am->w3 == nullptr || am->h == nullptr))
        return FP8MLP_ERR_ARG;
    const bool gu_fp8 = (c->flags & FP8MLP_GU_FP8) != 0;
    if (gu_fp8 && (sc->gu == nullptr || (mode == FP8MLP_SCALE_FROM_CURRENT_AMAX && am->gu == nullptr))) return FP8MLP_ERR_ARG;
    if (!aligned16(x) || !aligned16(y) || !aligned16(W1) || !aligned16(W2) || !aligned16(W3)) return FP8MLP_ERR_ALIGN;
    return FP8MLP_OK;
}

}  // namespace

extern "C" {

const char* fp8mlp_strerror(int code) {
    switch (code) {
        case FP8MLP_OK: return "ok";
        case FP8MLP_ERR_ARG: return "invalid argument (null pointer or bad enum value)";
        case FP8MLP_ERR_SHAPE: return "invalid shape (negative, not a multiple of 16, or T > T_max)";
        case FP8MLP_ERR_ALIGN: return "pointer not 16-byte aligned";
        case FP8MLP_ERR_CUDA: return "CUDA call failed";
        case FP8MLP_ERR_TIMEOUT: return "a kernel gave up on a bounded wait";
        case FP8MLP_ERR_STATE: return "call does not fit the context's state (backward without a matching forward that saved "
                                      "activations, merged forward without merged weights, or another device is current)";
        case FP8MLP_ERR_TOO_LARGE: return "problem does not fit the library's built-in scratch (see FP8MLP_STATIC_SCRATCH_BYTES)";
        default: return "unknown error code";
    }
}

const char* fp8mlp_last_cuda_error(void) { return g_last_error; }

int64_t fp8mlp_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int fp8mlp_create(fp8mlp_ctx** out, int64_t T_max, int64_t d, int64_t f, uint32_t flags) {
    if (out == nullptr) return FP8MLP_ERR_ARG;
    *out = nullptr;
    if (flags & ~uint32_t(FP8MLP_SMOOTH | FP8MLP_SAVE_FOR_BWD | FP8MLP_H_BF16 | FP8MLP_GU_FP8)) return FP8MLP_ERR_ARG;
    if ((flags & FP8MLP_SMOOTH) && (flags & FP8MLP_H_BF16)) return FP8MLP_ERR_ARG;   // nothing to smooth: H is not quantised
    if ((flags & FP8MLP_GU_FP8) && ((flags & FP8MLP_H_BF16) || !(flags & FP8MLP_SAVE_FOR_BWD))) return FP8MLP_ERR_ARG;
    if (T_max < 0 || d <= 0 || f <= 0 || d % 16 != 0 || f % 16 != 0) return FP8MLP_ERR_SHAPE;
    if (T_max > (1 << 30) || d > (1 << 24) || f > (1 << 24)) return FP8MLP_ERR_SHAPE;
    fp8mlp_ctx* c = new (std::nothrow) fp8mlp_ctx();
    if (c == nullptr) return FP8MLP_ERR_ARG;
    std::memset(c, 0, sizeof(*c));
    c->brackets = new (std::nothrow) std::vector<fp8mlp_ctx::Bracket>();
    c->free_events = new (std::nothrow) std::vector<cudaEvent_t>();
    if (c->brackets == nullptr || c->free_events == nullptr) { fp8mlp_destroy(c); return FP8MLP_ERR_ARG; }
    c->T_max = T_max; c->d = d; c->f = f; c->flags = flags; c->saved_T = -1;
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    const int64_t Tm = T_max > 0 ? T_max : 1;
    c->bytes[FP8MLP_WS_XQ] = Tm * d;
    c->bytes[FP8MLP_WS_W12Q] = d * 2 * f;
    c->bytes[FP8MLP_WS_W3Q] = f * d;
    c->bytes[FP8MLP_WS_HQ] = Tm * f;
    c->bytes[FP8MLP_WS_GU] = (flags & FP8MLP_SAVE_FOR_BWD) ? Tm * 2 * f * ((flags & FP8MLP_GU_FP8) ? 1 : 2) : 16;
    c->bytes[FP8MLP_WS_DYQ] = (flags & FP8MLP_SAVE_FOR_BWD) ? Tm * d : 16;
    c->bytes[FP8MLP_WS_DZQ] = (flags & FP8MLP_SAVE_FOR_BWD) ? Tm * 2 * f : 16;
    const bool hb16 = (flags & FP8MLP_H_BF16) != 0;
    if (hb16) {   // the last layer's operands are bf16: no FP8 copies of H, W3, dY
        c->bytes[FP8MLP_WS_HQ] = 16;
        c->bytes[FP8MLP_WS_W3Q] = 16;
        c->bytes[FP8MLP_WS_DYQ] = 16;
    }
    c->bytes[FP8MLP_WS_HB] = hb16 ? Tm * f * 2 : 16;
    c->bytes[FP8MLP_WS_W3B] = hb16 ? f * d * 2 : 16;
    void** slots[9] = {(void**)&c->xq, (void**)&c->w12q, (void**)&c->w3q, (void**)&c->hq,
                       (void**)&c->gu, (void**)&c->dyq, (void**)&c->dzq, (void**)&c->hb, (void**)&c->w3b};
    for (int i = 0; i < 9 && e == cudaSuccess; ++i) e = cudaMalloc(slots[i], static_cast<size_t>(c->bytes[i]));
    if (e == cudaSuccess) e = cudaMalloc((void**)&c->dummy, sizeof(float) * (8 + f));
    if (e == cudaSuccess) e = cudaMalloc((void**)&c->splitk_ws, sizeof(float) * kSplitFloats);
    if (e == cudaSuccess) e = cudaMalloc((void**)&c->splitk_cnt, sizeof(unsigned int) * kSplitWords);
    if (e == cudaSuccess) e = cudaMemset(c->splitk_cnt, 0, sizeof(unsigned int) * kSplitWords);
    if (e == cudaSuccess) e = cudaMalloc((void**)&c->status, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(c->status, 0, sizeof(int));
    if (e != cudaSuccess) {
        set_cuda_error("fp8mlp_create", e);
        fp8mlp_destroy(c);
        return FP8MLP_ERR_CUDA;
    }
    *out = c;
    return FP8MLP_OK;
}

int fp8mlp_destroy(fp8mlp_ctx* c) {
    if (c == nullptr) return FP8MLP_OK;
    void* ptrs[] = {c->xq, c->w12q, c->w3q, c->hq, c->gu, c->dyq, c->dzq, c->hb, c->w3b, c->dummy, c->status, c->splitk_ws, c->splitk_cnt};
    for (void* p : ptrs)
        if (p != nullptr) cudaFree(p);
    if (c->brackets != nullptr) {
        for (auto& b : *c->brackets) { cudaEventDestroy(b.e0); cudaEventDestroy(b.e1); }
        delete c->brackets;
    }
    if (c->free_events != nullptr) {
        for (cudaEvent_t e : *c->free_events) cudaEventDestroy(e);
        delete c->free_events;
    }
    delete c;
    return FP8MLP_OK;
}

int fp8mlp_status(fp8mlp_ctx* c, void* stream) {
    if (c == nullptr) return FP8MLP_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int word = 0;
    FP8MLP_CUDA_CHECK(cudaMemcpyAsync(&word, c->status, sizeof(int), cudaMemcpyDeviceToHost, st));
    FP8MLP_CUDA_CHECK(cudaStreamSynchronize(st));
    if (word != STATUS_OK) {
        FP8MLP_CUDA_CHECK(cudaMemsetAsync(c->status, 0, sizeof(int), st));
        return FP8MLP_ERR_TIMEOUT;
    }
    return FP8MLP_OK;
}

int fp8mlp_selftest_wait_timeout(fp8mlp_ctx* c, int64_t timeout_us, void* stream) {
    if (c == nullptr) return FP8MLP_ERR_ARG;
    if (timeout_us < 1 || timeout_us > 1000000) return FP8MLP_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* gave_up = reinterpret_cast<int*>(c->dummy + 6);      // a spare word of the context
    FP8MLP_CUDA_CHECK(cudaMemsetAsync(gave_up, 0, sizeof(int), st));
    wait_selftest_kernel<<<1, 32, 0, st>>>(c->status, static_cast<uint64_t>(timeout_us) * 1000ull, gave_up);
    FP8MLP_LAUNCH_CHECK();
    int flag = 0;
    FP8MLP_CUDA_CHECK(cudaMemcpyAsync(&flag, gave_up, sizeof(int), cudaMemcpyDeviceToHost, st));
    FP8MLP_CUDA_CHECK(cudaStreamSynchronize(st));
    return flag == 1 ? FP8MLP_OK : FP8MLP_ERR_STATE;
}

int fp8mlp_profile_enable(fp8mlp_ctx* c, int on) {
    if (c == nullptr) return FP8MLP_ERR_ARG;
    c->profiling = on != 0;
    return FP8MLP_OK;
}

int fp8mlp_profile_read(fp8mlp_ctx* c, double* ms, int64_t* count) {
    if (c == nullptr || ms == nullptr || count == nullptr) return FP8MLP_ERR_ARG;
    for (int i = 0; i < FP8MLP_PH_COUNT; ++i) { ms[i] = 0.0; count[i] = 0; }
    for (auto& b : *c->brackets) {
        FP8MLP_CUDA_CHECK(cudaEventSynchronize(b.e1));
        float t = 0.0f;
        FP8MLP_CUDA_CHECK(cudaEventElapsedTime(&t, b.e0, b.e1));
        ms[b.phase] += t;
        count[b.phase] += 1;
        c->free_events->push_back(b.e0);
        c->free_events->push_back(b.e1);
    }
    c->brackets->clear();
    return FP8MLP_OK;
}

int fp8mlp_workspace(fp8mlp_ctx* c, int which, void** ptr, int64_t* bytes) {
    if (c == nullptr || ptr == nullptr || bytes == nullptr || which < 0 || which > FP8MLP_WS_W3B) return FP8MLP_ERR_ARG;
    void* all[9] = {c->xq, c->w12q, c->w3q, c->hq, c->gu, c->dyq, c->dzq, c->hb, c->w3b};
    *ptr = all[which];
    *bytes = c->bytes[which];
    return FP8MLP_OK;
}

int fp8mlp_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols, int fp8_fmt, int scale_mode,
                    float* scale, float* amax, const float* row_mul, uint8_t* dst, int64_t ld_dst, void* stream) {
    if (src == nullptr || dst == nullptr || scale == nullptr) return FP8MLP_ERR_ARG;
    if (src_dtype != FP8MLP_BF16 && src_dtype != FP8MLP_F32) return FP8MLP_ERR_ARG;
    if (fp8_fmt != FP8MLP_E4M3 && fp8_fmt != FP8MLP_E5M2) return FP8MLP_ERR_ARG;
    if (scale_mode != FP8MLP_SCALE_GIVEN && scale_mode != FP8MLP_SCALE_FROM_CURRENT_AMAX) return FP8MLP_ERR_ARG;
    if (scale_mode == FP8MLP_SCALE_FROM_CURRENT_AMAX && amax == nullptr) return FP8MLP_ERR_ARG;
    if (rows < 0 || cols < 0 || cols % 16 != 0 || ld_dst < cols || ld_dst % 16 != 0) return FP8MLP_ERR_SHAPE;
    if (!aligned16(src) || !aligned16(dst)) return FP8MLP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    FP8MLP_CUDA_CHECK(cudaGetDevice(&dev));
    FP8MLP_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (amax != nullptr) FP8MLP_TRY(zero_floats(nullptr, {amax}, st));
    if (scale_mode == FP8MLP_SCALE_FROM_CURRENT_AMAX)
        return quantize_tensor(src, src_dtype, rows, cols, fp8_fmt, scale_mode, scale, amax, nullptr, row_mul, nullptr, dst,
                               ld_dst, sms, st);
    return run_quantize_pass(true, amax != nullptr, src, src_dtype, rows, cols, fp8_fmt, row_mul, scale, dst, ld_dst,
                             amax, sms, st);
}

int fp8mlp_code_stats(const uint8_t* codes, int64_t rows, int64_t cols, int64_t ld, int fp8_fmt, uint64_t* zero_count,
                      uint64_t* top_count, void* stream) {
    if (codes == nullptr || zero_count == nullptr || top_count == nullptr) return FP8MLP_ERR_ARG;
    if (fp8_fmt != FP8MLP_E4M3 && fp8_fmt != FP8MLP_E5M2) return FP8MLP_ERR_ARG;
    if (rows < 0 || cols < 0 || cols % 16 != 0 || ld < cols || ld % 16 != 0) return FP8MLP_ERR_SHAPE;
    if (!aligned16(codes) || (reinterpret_cast<uintptr_t>(zero_count) & 7u) || (reinterpret_cast<uintptr_t>(top_count) & 7u)) return FP8MLP_ERR_ALIGN;
    int dev = 0, sms = 0;
    FP8MLP_CUDA_CHECK(cudaGetDevice(&dev));
    FP8MLP_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    return run_code_stats(codes, rows, cols, ld, fp8_fmt, reinterpret_cast<unsigned long long*>(zero_count),
                          reinterpret_cast<unsigned long long*>(top_count), sms, static_cast<cudaStream_t>(stream));
}

int fp8mlp_scale_from_amax(const float* amax, int fp8_fmt, float* scale, void* stream) {
    if (amax == nullptr || scale == nullptr) return FP8MLP_ERR_ARG;
    if (fp8_fmt != FP8MLP_E4M3 && fp8_fmt != FP8MLP_E5M2) return FP8MLP_ERR_ARG;
    return run_scale_from_amax(fp8_fmt, amax, nullptr, scale, static_cast<cudaStream_t>(stream));
}

int fp8mlp_update_scales(fp8mlp_ctx* c, const fp8mlp_amax* am, fp8mlp_scales* sc, void* stream) {
    if (c == nullptr || am == nullptr || sc == nullptr) return FP8MLP_ERR_ARG;
    UpdateScalesArgs a{};
    a.amax_x = am->x; a.amax_w1 = am->w1; a.amax_w2 = am->w2; a.amax_w3 = am->w3;
    a.amax_dy = am->dy; a.amax_dz = am->dz; a.amax_h = am->h;
    a.scale_x = sc->x; a.scale_w12 = sc->w12; a.scale_w3 = sc->w3;
    a.scale_dy = sc->dy; a.scale_dz = sc->dz; a.scale_h = sc->h;
    if (c->flags & FP8MLP_GU_FP8) { a.amax_gu = am->gu; a.scale_gu = sc->gu; }
    a.f = c->f;
    a.smooth = (c->flags & FP8MLP_SMOOTH) ? 1 : 0;
    return run_update_scales(a, c->sm_count, static_cast<cudaStream_t>(stream));
}

int fp8mlp_forward(fp8mlp_ctx* c, int64_t T, const void* x, const float* W1, const float* W2, const float* W3,
                   int mode, fp8mlp_scales* sc, fp8mlp_amax* am, void* y, void* stream) {
    FP8MLP_TRY(check_forward_args(c, T, x, W1, W2, W3, mode, sc, am, y));
    const bool weights_cast = mode == FP8MLP_SCALE_GIVEN_WEIGHTS_CAST;
    if (weights_cast) mode = FP8MLP_SCALE_GIVEN;
    const bool gu_fp8 = (c->flags & FP8MLP_GU_FP8) != 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool smooth = (c->flags & FP8MLP_SMOOTH) != 0;
    const int64_t d = c->d, f = c->f;
    // amax sinks the caller did not provide
    float* a_x = (am && am->x) ? am->x : c->dummy + 0;
    float* a_w1 = (am && am->w1) ? am->w1 : c->dummy + 1;
    float* a_w2 = (am && am->w2) ? am->w2 : c->dummy + 2;
    float* a_w3 = (am && am->w3) ? am->w3 : c->dummy + 3;
    float* a_h = (am && am->h) ? am->h : c->dummy + 8;
    float* a_gu = (gu_fp8 && am && am->gu) ? am->gu : c->dummy + 7;
    c->saved_T = -1;
    c->merged = false;

    {
        PhaseTimer pt(c, FP8MLP_PH_MISC, st);
        if (weights_cast) FP8MLP_TRY(zero_floats(c, {a_x, a_gu}, st, a_h, f));     // the weights' maxima came with their codes
        else FP8MLP_TRY(zero_floats(c, {a_x, a_w1, a_w2, a_w3, a_gu}, st, a_h, f));
    }
    {   // x -> E4M3
        PhaseTimer pt(c, FP8MLP_PH_QUANT_X, st);
        FP8MLP_TRY(quantize_tensor(x, FP8MLP_BF16, T, d, FP8MLP_E4M3, mode, sc->x, a_x, nullptr, nullptr, nullptr, c->xq, d, c->sm_count, st));
    }
    if (c->flags & FP8MLP_H_BF16) {
        // "SwiGLU output in BF16" variant: the last layer is not quantised.  [W2 | W1] -> E4M3, W3 -> bf16,
        // GEMM-1 stores H in bf16 (no scale, so no calibration pass), GEMM-2 runs on bf16 operands.
        {
            PhaseTimer pt(c, FP8MLP_PH_QUANT_W12, st);
            FP8MLP_TRY(quantize_w12(c, W1, W2, mode, sc->w12, a_w1, a_w2, st));
        }
        {
            PhaseTimer pt(c, FP8MLP_PH_QUANT_W3, st);
            FP8MLP_TRY(run_cast_bf16(W3, c->w3b, f * d, a_w3, c->sm_count, st));
        }
        if (T == 0) { c->saved_T = (c->flags & FP8MLP_SAVE_FOR_BWD) ? 0 : -1; return FP8MLP_OK; }
        {
            PhaseTimer pt(c, FP8MLP_PH_GEMM1, st);
            FP8MLP_TRY(gemm1_swiglu(c, T, sc, a_h, /*store=*/1, st));
        }
        PhaseTimer pt2(c, FP8MLP_PH_GEMM2, st);
        CUtensorMap tmA, tmB;
        FP8MLP_TRY(make_tmap(&tmA, c->hb, 2, false, f, T, 2 * f));
        FP8MLP_TRY(make_tmap(&tmB, c->w3b, 2, true, d, f, 2 * d));
        GemmArgs a = base_args(c, static_cast<int>(T), static_cast<int>(d), static_cast<int>(f));
        a.elem_bytes = 2;
        a.out_bf16 = static_cast<uint16_t*>(y);
        FP8MLP_TRY(launch_gemm(EPI_BF16, false, true, 1, 1, tmA, tmB, tmB, a, c->sm_count, st));
        if (c->flags & FP8MLP_SAVE_FOR_BWD) c->saved_T = T;
        return FP8MLP_OK;
    }
    if (weights_cast) {
        // nothing to do: the optimizer step wrote this step's [W2 | W1] and W3' codes (fp8mlp_adam_step_cast)
    } else if (mode == FP8MLP_SCALE_GIVEN) {
        // every scale is known: [W2 | W1] (one scale) and W3' = diag(1/s) W3 in one pass over the masters;
        // the reciprocal of s_i is taken inside the pass, row by row
        PhaseTimer pt(c, FP8MLP_PH_QUANT_W12, st);
        QuantTensor t[3] = {};
        t[0].src = W2; t[0].rows = d; t[0].cols = f; t[0].dst = c->w12q; t[0].ld_dst = 2 * f; t[0].amax = a_w2;
        t[1].src = W1; t[1].rows = d; t[1].cols = f; t[1].dst = c->w12q + f; t[1].ld_dst = 2 * f; t[1].amax = a_w1;
        t[2].src = W3; t[2].rows = f; t[2].cols = d; t[2].dst = c->w3q; t[2].ld_dst = d; t[2].amax = a_w3;
        t[2].row_div = smooth ? sc->h : nullptr; t[2].scale = sc->w3;
        FP8MLP_TRY(run_quantize_segments(true, true, FP8MLP_F32, FP8MLP_E4M3, t, 3, sc->w12, c->sm_count, st));
    } else {
        {   // [W2 | W1] -> E4M3 with one scale
            PhaseTimer pt(c, FP8MLP_PH_QUANT_W12, st);
            FP8MLP_TRY(quantize_w12(c, W1, W2, mode, sc->w12, a_w1, a_w2, st));
        }
        // calibration pass: per-channel maxima of H, then s_i (or the per-tensor scale)
        if (T > 0) {
            PhaseTimer pt(c, FP8MLP_PH_GEMM1, st);
            FP8MLP_TRY(gemm1_swiglu(c, T, sc, a_h, /*store=*/0, st, true, a_gu));
        }
        {
            PhaseTimer pt(c, FP8MLP_PH_MISC, st);
            UpdateScalesArgs u{};
            u.amax_h = a_h; u.scale_h = sc->h; u.f = f; u.smooth = smooth ? 1 : 0;
            if (gu_fp8) { u.amax_gu = a_gu; u.scale_gu = sc->gu; }
            FP8MLP_TRY(run_update_scales(u, c->sm_count, st));
        }
        // W3' = diag(1/s) W3 -> E4M3
        PhaseTimer pt(c, FP8MLP_PH_QUANT_W3, st);
        FP8MLP_TRY(quantize_tensor(W3, FP8MLP_F32, f, d, FP8MLP_E4M3, mode, sc->w3, a_w3, nullptr, nullptr,
                                   smooth ? sc->h : nullptr, c->w3q, d, c->sm_count, st));
    }
    if (T == 0) { c->saved_T = (c->flags & FP8MLP_SAVE_FOR_BWD) ? 0 : -1; return FP8MLP_OK; }
    {
        PhaseTimer pt(c, FP8MLP_PH_GEMM1, st);
        FP8MLP_TRY(gemm1_swiglu(c, T, sc, a_h, /*store=*/1, st, true, a_gu));
    }
    // Y = Hq W3q
    PhaseTimer pt2(c, FP8MLP_PH_GEMM2, st);
    CUtensorMap tmA, tmB;
    FP8MLP_TRY(make_tmap_u8(&tmA, c->hq, f, T, f));
    FP8MLP_TRY(make_tmap_u8(&tmB, c->w3q, d, f, d));
    GemmArgs a = base_args(c, static_cast<int>(T), static_cast<int>(d), static_cast<int>(f));
    a.s0 = sc->w3;
    a.s1 = smooth ? nullptr : sc->h;
    a.out_bf16 = static_cast<uint16_t*>(y);
    FP8MLP_TRY(launch_gemm(EPI_BF16, false, true, FP8MLP_E4M3, FP8MLP_E4M3, tmA, tmB, tmB, a, c->sm_count, st));
    if (c->flags & FP8MLP_SAVE_FOR_BWD) c->saved_T = T;
    return FP8MLP_OK;
}

int fp8mlp_merge_weights(fp8mlp_ctx* c, const float* W1, const float* W2, const float* W3, const float* s,
                         int mode, fp8mlp_scales* sc, fp8mlp_amax* am, void* stream) {
    if (c == nullptr || sc == nullptr || W1 == nullptr || W2 == nullptr || W3 == nullptr || s == nullptr) return FP8MLP_ERR_ARG;
    if (mode != FP8MLP_SCALE_GIVEN && mode != FP8MLP_SCALE_FROM_CURRENT_AMAX) return FP8MLP_ERR_ARG;
    if (sc->w12 == nullptr || sc->w3 == nullptr) return FP8MLP_ERR_ARG;
    if (c->flags & FP8MLP_H_BF16) return FP8MLP_ERR_STATE;          // this context has no FP8 W3
    if (!on_device_of(c)) return FP8MLP_ERR_STATE;
    if (!aligned16(W1) || !aligned16(W2) || !aligned16(W3) || !aligned16(s)) return FP8MLP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t d = c->d, f = c->f;
    float* a_w1 = (am && am->w1) ? am->w1 : c->dummy + 1;
    float* a_w2 = (am && am->w2) ? am->w2 : c->dummy + 2;
    float* a_w3 = (am && am->w3) ? am->w3 : c->dummy + 3;
    c->saved_T = -1;
    c->merged = false;
    FP8MLP_TRY(zero_floats(c, {a_w1, a_w2, a_w3}, st));
    QuantTensor t[3] = {};
    t[0].src = W2; t[0].rows = d; t[0].cols = f; t[0].dst = c->w12q; t[0].ld_dst = 2 * f; t[0].amax = a_w2;
    t[1].src = W1; t[1].rows = d; t[1].cols = f; t[1].dst = c->w12q + f; t[1].ld_dst = 2 * f; t[1].amax = a_w1;
    t[1].col_mul = s;                                            // w1~_i = s_i w1_i
    t[2].src = W3; t[2].rows = f; t[2].cols = d; t[2].dst = c->w3q; t[2].ld_dst = d; t[2].amax = a_w3;
    t[2].row_div = s; t[2].scale = sc->w3;                       // w3~_i = s_i^-1 w3_i
    if (mode == FP8MLP_SCALE_FROM_CURRENT_AMAX) {
        FP8MLP_TRY(run_quantize_segments(false, true, FP8MLP_F32, FP8MLP_E4M3, t, 3, nullptr, c->sm_count, st));
        FP8MLP_TRY(run_scale_from_amax(FP8MLP_E4M3, a_w1, a_w2, sc->w12, st));
        FP8MLP_TRY(run_scale_from_amax(FP8MLP_E4M3, a_w3, nullptr, sc->w3, st));
        FP8MLP_TRY(run_quantize_segments(true, false, FP8MLP_F32, FP8MLP_E4M3, t, 3, sc->w12, c->sm_count, st));
    } else {
        FP8MLP_TRY(run_quantize_segments(true, true, FP8MLP_F32, FP8MLP_E4M3, t, 3, sc->w12, c->sm_count, st));
    }
    c->merged = true;
    return FP8MLP_OK;
}

int fp8mlp_forward_merged(fp8mlp_ctx* c, int64_t T, const void* x, int mode, fp8mlp_scales* sc, fp8mlp_amax* am,
                          void* y, void* stream) {
    if (c == nullptr || sc == nullptr) return FP8MLP_ERR_ARG;
    if (mode != FP8MLP_SCALE_GIVEN && mode != FP8MLP_SCALE_FROM_CURRENT_AMAX) return FP8MLP_ERR_ARG;
    if (T < 0 || T > c->T_max) return FP8MLP_ERR_SHAPE;
    if (!on_device_of(c) || !c->merged) return FP8MLP_ERR_STATE;
    if (T > 0 && (x == nullptr || y == nullptr)) return FP8MLP_ERR_ARG;
    if (sc->x == nullptr || sc->w12 == nullptr || sc->w3 == nullptr || sc->h == nullptr) return FP8MLP_ERR_ARG;
    if (mode == FP8MLP_SCALE_FROM_CURRENT_AMAX && (am == nullptr || am->x == nullptr || am->h == nullptr)) return FP8MLP_ERR_ARG;
    if (!aligned16(x) || !aligned16(y)) return FP8MLP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t d = c->d, f = c->f;
    float* a_x = (am && am->x) ? am->x : c->dummy + 0;
    float* a_h = (am && am->h) ? am->h : nullptr;                // maxima of H only if asked for
    if (T == 0) return FP8MLP_OK;
    {
        PhaseTimer pt(c, FP8MLP_PH_MISC, st);
        FP8MLP_TRY(zero_floats(c, {a_x}, st, a_h, f));
    }
    {
        PhaseTimer pt(c, FP8MLP_PH_QUANT_X, st);
        FP8MLP_TRY(quantize_tensor(x, FP8MLP_BF16, T, d, FP8MLP_E4M3, mode, sc->x, a_x, nullptr, nullptr, nullptr, c->xq, d, c->sm_count, st));
    }
    if (mode == FP8MLP_SCALE_FROM_CURRENT_AMAX) {
        {
            PhaseTimer pt(c, FP8MLP_PH_GEMM1, st);
            FP8MLP_TRY(gemm1_swiglu(c, T, sc, a_h, /*store=*/0, st, /*save_gu=*/false));
        }
        PhaseTimer pt(c, FP8MLP_PH_MISC, st);
        UpdateScalesArgs u{};
        u.amax_h = a_h; u.scale_h = sc->h; u.f = f; u.smooth = 0;   // one per-tensor scale: the s_i sit in the weights
        FP8MLP_TRY(run_update_scales(u, c->sm_count, st));
    }
    {
        PhaseTimer pt(c, FP8MLP_PH_GEMM1, st);
        FP8MLP_TRY(gemm1_swiglu(c, T, sc, a_h, /*store=*/1, st, /*save_gu=*/false));
    }
    PhaseTimer pt2(c, FP8MLP_PH_GEMM2, st);
    CUtensorMap tmA, tmB;
    FP8MLP_TRY(make_tmap_u8(&tmA, c->hq, f, T, f));
    FP8MLP_TRY(make_tmap_u8(&tmB, c->w3q, d, f, d));
    GemmArgs a = base_args(c, static_cast<int>(T), static_cast<int>(d), static_cast<int>(f));
    a.s0 = sc->w3;
    a.s1 = sc->h;
    a.out_bf16 = static_cast<uint16_t*>(y);
    return launch_gemm(EPI_BF16, false, true, FP8MLP_E4M3, FP8MLP_E4M3, tmA, tmB, tmB, a, c->sm_count, st);
}

int fp8mlp_backward(fp8mlp_ctx* c, int64_t T, const void* dy, int mode, fp8mlp_scales* sc, fp8mlp_amax* am,
                    void* dx, float* dW1, float* dW2, float* dW3, void* stream) {
    if (c == nullptr || sc == nullptr || dW1 == nullptr || dW2 == nullptr || dW3 == nullptr) return FP8MLP_ERR_ARG;
    if (mode != FP8MLP_SCALE_GIVEN && mode != FP8MLP_SCALE_FROM_CURRENT_AMAX) return FP8MLP_ERR_ARG;
    if (T < 0 || T > c->T_max) return FP8MLP_ERR_SHAPE;
    if (!on_device_of(c)) return FP8MLP_ERR_STATE;
    if (!(c->flags & FP8MLP_SAVE_FOR_BWD) || c->saved_T != T) return FP8MLP_ERR_STATE;
    if (T > 0 && (dy == nullptr || dx == nullptr)) return FP8MLP_ERR_ARG;
    if (sc->x == nullptr || sc->w12 == nullptr || sc->w3 == nullptr || sc->h == nullptr || sc->dy == nullptr || sc->dz == nullptr)
        return FP8MLP_ERR_ARG;
    if ((c->flags & FP8MLP_GU_FP8) && sc->gu == nullptr) return FP8MLP_ERR_ARG;
    if (mode == FP8MLP_SCALE_FROM_CURRENT_AMAX && (am == nullptr || am->dy == nullptr || am->dz == nullptr)) return FP8MLP_ERR_ARG;
    if (!aligned16(dy) || !aligned16(dx) || !aligned16(dW1) || !aligned16(dW2) || !aligned16(dW3)) return FP8MLP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool smooth = (c->flags & FP8MLP_SMOOTH) != 0;
    const int64_t d = c->d, f = c->f;
    float* a_dy = (am && am->dy) ? am->dy : c->dummy + 4;
    float* a_dz = (am && am->dz) ? am->dz : c->dummy + 5;
    {
        PhaseTimer pt(c, FP8MLP_PH_MISC, st);
        FP8MLP_TRY(zero_floats(c, {a_dy, a_dz}, st));
    }
    if (T == 0) {   // empty batch: the weight gradients are sums over no tokens
        FP8MLP_CUDA_CHECK(cudaMemsetAsync(dW1, 0, sizeof(float) * d * f, st));
        FP8MLP_CUDA_CHECK(cudaMemsetAsync(dW2, 0, sizeof(float) * d * f, st));
        FP8MLP_CUDA_CHECK(cudaMemsetAsync(dW3, 0, sizeof(float) * d * f, st));
        return FP8MLP_OK;
    }
    const int Ti = static_cast<int>(T), di = static_cast<int>(d), fi = static_cast<int>(f);

    const bool hb16 = (c->flags & FP8MLP_H_BF16) != 0;
    if (!hb16) {   // dY -> E5M2 (with the bf16 last layer dY is used as it is)
        PhaseTimer pt(c, FP8MLP_PH_QUANT_DY, st);
        FP8MLP_TRY(quantize_tensor(dy, FP8MLP_BF16, T, d, FP8MLP_E5M2, mode, sc->dy, a_dy, nullptr, nullptr, nullptr, c->dyq, d, c->sm_count, st));
    }

    // dH~ = dYq W3q^T with the SwiGLU-backward epilogue -> dZq = [dG | dU]
    {
        CUtensorMap tmA, tmB;
        GemmArgs a = base_args(c, Ti, fi, di);
        int fa = FP8MLP_E5M2, fb = FP8MLP_E4M3;
        if (hb16) {                      // dH = dY W3b^T on the bf16 operands, no dequantisation
            FP8MLP_TRY(make_tmap(&tmA, dy, 2, false, d, T, 2 * d));
            FP8MLP_TRY(make_tmap(&tmB, c->w3b, 2, false, d, f, 2 * d));
            a.elem_bytes = 2;
            fa = fb = 1;
        } else {
            FP8MLP_TRY(make_tmap_u8(&tmA, c->dyq, d, T, d));
            FP8MLP_TRY(make_tmap_u8(&tmB, c->w3q, d, f, d));
            a.s0 = sc->dy; a.s1 = sc->w3;
        }
        a.s_h = sc->h; a.smooth = smooth ? 1 : 0;
        a.gu = c->gu; a.sdz = sc->dz; a.dzq = c->dzq;
        if (c->flags & FP8MLP_GU_FP8) { a.gu8 = reinterpret_cast<uint8_t*>(c->gu); a.gu = nullptr; a.s_gu = sc->gu; }
        a.amax_dz = reinterpret_cast<unsigned int*>(a_dz);
        if (mode == FP8MLP_SCALE_FROM_CURRENT_AMAX) {
            a.store = 0;
            {
                PhaseTimer pt(c, FP8MLP_PH_DGRAD2, st);
                FP8MLP_TRY(launch_gemm(EPI_SWIGLU_BWD, false, false, fa, fb, tmA, tmB, tmB, a, c->sm_count, st));
            }
            PhaseTimer pt(c, FP8MLP_PH_MISC, st);
            UpdateScalesArgs u{};
            u.amax_dz = a_dz; u.scale_dz = sc->dz;
            FP8MLP_TRY(run_update_scales(u, c->sm_count, st));
            a.store = 1;
        }
        PhaseTimer pt(c, FP8MLP_PH_DGRAD2, st);
        FP8MLP_TRY(launch_gemm(EPI_SWIGLU_BWD, false, false, fa, fb, tmA, tmB, tmB, a, c->sm_count, st));
    }
    // dW3 = diag(1/s) (Hq^T dYq)
    {
        CUtensorMap tmA, tmB;
        GemmArgs a = base_args(c, fi, di, Ti);
        int fa = FP8MLP_E4M3, fb = FP8MLP_E5M2;
        if (hb16) {                      // dW3 = Hb^T dY on the bf16 operands
            FP8MLP_TRY(make_tmap(&tmA, c->hb, 2, true, f, T, 2 * f));
            FP8MLP_TRY(make_tmap(&tmB, dy, 2, true, d, T, 2 * d));
            a.elem_bytes = 2;
            fa = fb = 1;
        } else {
            FP8MLP_TRY(make_tmap_u8(&tmA, c->hq, f, T, f));
            FP8MLP_TRY(make_tmap_u8(&tmB, c->dyq, d, T, d));
            a.s0 = sc->dy; a.row_s = sc->h;
        }
        a.out_f32_0 = dW3; a.out_f32_1 = dW3;
        PhaseTimer pt(c, FP8MLP_PH_WGRAD3, st);
        FP8MLP_TRY(launch_gemm(EPI_F32, true, true, fa, fb, tmA, tmB, tmB, a, c->sm_count, st));
    }
    // dX = dZq [W2q|W1q]^T
    {
        CUtensorMap tmA, tmB;
        FP8MLP_TRY(make_tmap_u8(&tmA, c->dzq, 2 * f, T, 2 * f));
        FP8MLP_TRY(make_tmap_u8(&tmB, c->w12q, 2 * f, d, 2 * f));
        GemmArgs a = base_args(c, Ti, di, 2 * fi);
        a.s0 = sc->dz; a.s1 = sc->w12;
        a.out_bf16 = static_cast<uint16_t*>(dx);
        PhaseTimer pt(c, FP8MLP_PH_DGRAD1, st);
        FP8MLP_TRY(launch_gemm(EPI_BF16, false, false, FP8MLP_E5M2, FP8MLP_E4M3, tmA, tmB, tmB, a, c->sm_count, st));
    }
    // [dW2 | dW1] = Xq^T dZq
    {
        CUtensorMap tmA, tmB;
        FP8MLP_TRY(make_tmap_u8(&tmA, c->xq, d, T, d));
        FP8MLP_TRY(make_tmap_u8(&tmB, c->dzq, 2 * f, T, 2 * f));
        GemmArgs a = base_args(c, di, 2 * fi, Ti);
        a.s0 = sc->x; a.s1 = sc->dz;
        a.out_f32_0 = dW2; a.out_f32_1 = dW1;
        a.n_split = fi; a.ld_out = f;
        PhaseTimer pt(c, FP8MLP_PH_WGRAD12, st);
        FP8MLP_TRY(launch_gemm(EPI_F32, true, true, FP8MLP_E4M3, FP8MLP_E5M2, tmA, tmB, tmB, a, c->sm_count, st));
    }
    return FP8MLP_OK;
}

// ---------------------------------------------------------------- forward without allocation
}  // extern "C"

namespace {
// Built-in scratch of fp8mlp_forward_static.  In host code this name is only a stand-in for the
// symbol, not a device address: the address on the current device is asked of the runtime with
// cudaGetSymbolAddress (a table lookup after the first call on a device; asking every time keeps
// no pointer that a cudaDeviceReset could leave stale).
__device__ __align__(256) unsigned char g_static_scratch[FP8MLP_STATIC_SCRATCH_BYTES];

int64_t round_up_256(int64_t v) { return (v + 255) & ~int64_t(255); }
}  // namespace

extern "C" {

int fp8mlp_forward_static(int64_t T, int64_t d, int64_t f, uint32_t flags, const void* x, const float* W1,
                          const float* W2, const float* W3, int mode, fp8mlp_scales* sc, fp8mlp_amax* am, void* y,
                          void* stream) {
    if (flags & ~uint32_t(FP8MLP_SMOOTH)) return FP8MLP_ERR_ARG;
    if (mode == FP8MLP_SCALE_GIVEN_WEIGHTS_CAST) return FP8MLP_ERR_ARG;      // nothing persists in the built-in scratch
    if (T < 0 || d <= 0 || f <= 0 || d % 16 != 0 || f % 16 != 0) return FP8MLP_ERR_SHAPE;
    if (T > (1 << 22) || d > (1 << 22) || f > (1 << 22)) return FP8MLP_ERR_TOO_LARGE;
    if (T * d + 3 * d * f + T * f + 8 * f + 4096 > int64_t(FP8MLP_STATIC_SCRATCH_BYTES)) return FP8MLP_ERR_TOO_LARGE;

    int dev = 0, sms = 0;
    FP8MLP_CUDA_CHECK(cudaGetDevice(&dev));
    FP8MLP_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));

    // a context that lives on this stack frame; its buffers are carved out of the built-in array below
    fp8mlp_ctx c;
    std::memset(&c, 0, sizeof(c));
    c.T_max = T; c.d = d; c.f = f; c.flags = flags; c.device = dev; c.sm_count = sms; c.saved_T = -1;
    // every argument error is found here, before anything is enqueued
    FP8MLP_TRY(check_forward_args(&c, T, x, W1, W2, W3, mode, sc, am, y));

    void* sym = nullptr;
    FP8MLP_CUDA_CHECK(cudaGetSymbolAddress(&sym, g_static_scratch));
    unsigned char* base = static_cast<unsigned char*>(sym);
    int64_t off = 0;
    auto carve = [&](int64_t bytes) { unsigned char* p = base + off; off += round_up_256(bytes); return p; };
    c.status = reinterpret_cast<int*>(carve(256));
    c.dummy = reinterpret_cast<float*>(carve(sizeof(float) * (8 + f)));
    c.xq = carve(T * d);
    c.w12q = carve(2 * d * f);
    c.w3q = carve(f * d);
    c.hq = carve(T * f);
    if (off > int64_t(FP8MLP_STATIC_SCRATCH_BYTES)) return FP8MLP_ERR_TOO_LARGE;
    // the array keeps the previous call's contents: the status word must start at zero (forward
    // itself clears the maxima it accumulates into)
    FP8MLP_CUDA_CHECK(cudaMemsetAsync(c.status, 0, sizeof(int), static_cast<cudaStream_t>(stream)));
    return fp8mlp_forward(&c, T, x, W1, W2, W3, mode, sc, am, y, stream);
}

int fp8mlp_gemm_plan(int kind, int64_t M, int64_t N, int64_t K, int sm_count, int with_workspace, fp8mlp_gemm_plan_t* out) {
    if (out == nullptr || kind < EPI_F32 || kind > EPI_SWIGLU_BWD || sm_count < 1) return FP8MLP_ERR_ARG;
    if (M <= 0 || N <= 0 || K <= 0 || M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return FP8MLP_ERR_SHAPE;
    GemmArgs a = base_args(nullptr, static_cast<int>(M), static_cast<int>(N), static_cast<int>(K));
    if (kind == EPI_SWIGLU_FWD) { a.n_tile_cols = 128; a.b1_offset = 0; }
    static float ws_stand_in;               // never dereferenced: planning only asks whether a workspace exists
    static unsigned int cnt_stand_in;
    if (with_workspace) { a.partial = &ws_stand_in; a.partial_floats = kSplitFloats; a.tile_counters = &cnt_stand_in; a.counter_words = kSplitWords; }
    const GemmPlan p = plan_gemm(kind, a, sm_count);
    out->cta_pairs = p.pair ? 1 : 0;
    out->tile_rows = p.tile_m;
    out->tile_cols = a.n_tile_cols;
    out->m_tiles = a.num_m_tiles; out->n_tiles = a.num_n_tiles; out->k_stages = a.num_k_blocks;
    out->split_k = a.split_k; out->stages_per_share = a.kb_per_split;
    out->band_along_n = a.band_n; out->band_tiles = a.group;
    out->staged_stores = a.tma_store;
    out->work_items = p.items;
    return FP8MLP_OK;
}

int fp8mlp_gemm_bf16(int64_t M, int64_t N, int64_t K, const void* A, int a_kmajor, const void* B, int b_kmajor,
                     float* out, void* stream) {
    if (A == nullptr || B == nullptr || out == nullptr) return FP8MLP_ERR_ARG;
    if (M <= 0 || N <= 0 || K <= 0 || M % 16 || N % 16 || K % 16 || M > (1 << 24) || N > (1 << 24) || K > (1 << 24)) return FP8MLP_ERR_SHAPE;
    if (!aligned16(A) || !aligned16(B) || !aligned16(out)) return FP8MLP_ERR_ALIGN;
    int dev = 0, sms = 0;
    FP8MLP_CUDA_CHECK(cudaGetDevice(&dev));
    FP8MLP_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CUtensorMap tmA, tmB;
    if (a_kmajor) FP8MLP_TRY(make_tmap(&tmA, A, 2, false, K, M, 2 * K)); else FP8MLP_TRY(make_tmap(&tmA, A, 2, true, M, K, 2 * M));
    if (b_kmajor) FP8MLP_TRY(make_tmap(&tmB, B, 2, false, K, N, 2 * K)); else FP8MLP_TRY(make_tmap(&tmB, B, 2, true, N, K, 2 * N));
    GemmArgs a = base_args(nullptr, static_cast<int>(M), static_cast<int>(N), static_cast<int>(K));
    a.elem_bytes = 2;
    a.out_f32_0 = out; a.out_f32_1 = out;
    return launch_gemm(EPI_F32, !a_kmajor, !b_kmajor, 1, 1, tmA, tmB, tmB, a, sms, static_cast<cudaStream_t>(stream));
}

int fp8mlp_gemm_fp8(int64_t M, int64_t N, int64_t K, const uint8_t* A, int a_kmajor, int a_fmt, const uint8_t* B,
                    int b_kmajor, int b_fmt, const float* scale_a, const float* scale_b, float* out, void* stream) {
    if (A == nullptr || B == nullptr || out == nullptr) return FP8MLP_ERR_ARG;
    if ((a_fmt != FP8MLP_E4M3 && a_fmt != FP8MLP_E5M2) || (b_fmt != FP8MLP_E4M3 && b_fmt != FP8MLP_E5M2)) return FP8MLP_ERR_ARG;
    if (M <= 0 || N <= 0 || K <= 0 || M % 16 || N % 16 || K % 16 || M > (1 << 24) || N > (1 << 24) || K > (1 << 24)) return FP8MLP_ERR_SHAPE;
    if (!aligned16(A) || !aligned16(B) || !aligned16(out)) return FP8MLP_ERR_ALIGN;
    int dev = 0, sms = 0;
    FP8MLP_CUDA_CHECK(cudaGetDevice(&dev));
    FP8MLP_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CUtensorMap tmA, tmB;
    if (a_kmajor) FP8MLP_TRY(make_tmap_u8(&tmA, A, K, M, K)); else FP8MLP_TRY(make_tmap_u8(&tmA, A, M, K, M));
    if (b_kmajor) FP8MLP_TRY(make_tmap_u8(&tmB, B, K, N, K)); else FP8MLP_TRY(make_tmap_u8(&tmB, B, N, K, N));
    GemmArgs a = base_args(nullptr, static_cast<int>(M), static_cast<int>(N), static_cast<int>(K));
    a.s0 = scale_a; a.s1 = scale_b;
    a.out_f32_0 = out; a.out_f32_1 = out;
    return launch_gemm(EPI_F32, !a_kmajor, !b_kmajor, a_fmt, b_fmt, tmA, tmB, tmB, a, sms, static_cast<cudaStream_t>(stream));
}

}  // extern "C"

// tcgen05 FP8 GEMM kernel and its fused epilogues (see gemm.cuh for the design).
#include "gemm.cuh"

#include <mutex>

namespace fp8mlp {

namespace {

// ---------------------------------------------------------------- shared memory plan
// Single CTA: a stage holds an A box and two B boxes (128 x 256 tile).  CTA pair: a stage holds this
// CTA's A box and its one B box (its halves of a 256 x 256 tile).
// The backward SwiGLU kernel gives up a stage for a ring of three 16-KiB slots through which a loader warp
// streams the saved G and U to the epilogue: a slot holds a box of 128 rows x 64 bytes of G and one of U
// (32 channels as bf16, consumed by the four warps of one column half; or 64 channels as E4M3 codes,
// consumed by all eight), 64-byte swizzle.  The main loop is sensitive to its depth - with three operand stages this
// kernel runs 14 % slower than with four - so the ring is kept as small as hides the latency of its own loads.
constexpr int kGuSlots = 3;
constexpr int kGuBoxBytes = 128 * 64;
constexpr int kGuSlotBytes = 2 * kGuBoxBytes;
// WIDEN (CTA pairs, plain epilogues): a 256 x 512 tile - both accumulators belong to one tile, the A block
// of a stage is loaded once for two B blocks (a quarter less operand traffic), the epilogue is not overlapped.
template <bool PAIR, int EPI, bool WIDEN> struct Plan;
template <int EPI, bool WIDEN> struct Plan<false, EPI, WIDEN> {
    static constexpr int kStages = EPI == EPI_SWIGLU_BWD ? 3 : 4, kStageBytes = 3 * kBoxBytes, kTileM = 128;
};
template <int EPI, bool WIDEN> struct Plan<true, EPI, WIDEN> {
    static constexpr int kStages = WIDEN ? 4 : EPI == EPI_SWIGLU_BWD ? 5 : 6, kStageBytes = (WIDEN ? 3 : 2) * kBoxBytes, kTileM = 256;
};
constexpr int kMaxStages = 6;
// With a short contraction (few tokens) the fp32-output kernels (weight gradients) are bound by their output, and a
// thread owns a row of the accumulator, so direct stores touch 32 different lines per instruction and cost several
// times the data-pipe cycles.  Then the output is staged in shared memory, in 32-row x 32-column blocks (4 KiB,
// 128-byte swizzle) per epilogue warp, and sent to global memory as bulk tensor stores.  The staging blocks take the
// place of the last two operand stages, which a short contraction does not need (args.stages, args.tma_store).
constexpr int kStoreBlockBytes = 32 * 128;
constexpr int kStagesLentToStores = 2;
// The 256 x 512-tile kernels with bf16 output (down projection, input gradient) do not overlap their epilogue with a
// main loop, so what the epilogue costs is what its stores cost: they stage 32-row x 32-column bf16 blocks (2 KiB,
// 64-byte swizzle), two per epilogue warp, in shared memory of their own (these kernels use four 48-KiB stages).
constexpr int kStoreBlockBytesBf16 = 32 * 64;
template <int EPI, bool WIDEN> struct OwnStoreBytes { static constexpr int value = (EPI == EPI_BF16 && WIDEN) ? (kEpiThreads / 32) * 2 * kStoreBlockBytesBf16 : 0; };

template <bool FUSED>            // FUSED: the SwiGLU epilogues, which keep per-channel scales and maxima of the tile here
struct __align__(8) SmemTailT {
    uint64_t full[kMaxStages];   // TMA -> MMA: stage filled (CTA pair: only rank 0's are used)
    uint64_t empty[kMaxStages];  // MMA -> TMA: stage drained
    uint64_t tmem_full[2];       // MMA -> epilogue: accumulator complete
    uint64_t tmem_empty[2];      // epilogue -> MMA: accumulator drained (CTA pair: rank 0's count both CTAs)
    uint64_t gu_full[kGuSlots];  // loader -> epilogue: saved G, U chunk landed (backward)
    uint64_t gu_empty[kGuSlots]; // epilogue -> loader: chunk read into registers
    uint32_t tmem_base;
    int abort;
    float s_tile[2][FUSED ? kBlockN : 1];    // per-channel scales of the current tile(s)
    unsigned int amax_tile[FUSED ? 128 : 1]; // per-channel maxima of the current tile (forward)
};
using SmemTail = SmemTailT<true>;
template <int EPI> using TailOf = SmemTailT<EPI == EPI_SWIGLU_FWD || EPI == EPI_SWIGLU_BWD>;
template <bool PAIR, int EPI, bool WIDEN>
constexpr size_t smem_bytes() {
    return 1024 /*alignment slack*/ + size_t(Plan<PAIR, EPI, WIDEN>::kStages) * Plan<PAIR, EPI, WIDEN>::kStageBytes +
           (EPI == EPI_SWIGLU_BWD ? size_t(kGuSlots) * kGuSlotBytes : 0) + OwnStoreBytes<EPI, WIDEN>::value + sizeof(TailOf<EPI>);
}
static_assert(smem_bytes<true, EPI_BF16, true>() <= 232448 && smem_bytes<true, EPI_F32, false>() <= 232448 && smem_bytes<false, EPI_F32, false>() <= 232448 &&
              smem_bytes<true, EPI_SWIGLU_BWD, false>() <= 232448, "shared memory plan exceeds what a CTA can have");

// ---------------------------------------------------------------- descriptors
// Shared-memory matrix descriptor, 128-byte swizzle.  Bits: [0,14) address>>4, [16,30) leading
// byte offset>>4, [32,46) stride byte offset>>4, [46,48) version 1, [61,64) layout 2 = SW128.
//   K-major : rows 128 bytes apart, 8-row atoms 1024 bytes apart (stride offset); leading unused.
//   MN-major: each K row holds 128 contiguous M/N bytes; 8-K-row atoms 1024 bytes apart (stride
//             offset); the next 128 M/N bytes start one box (16 KiB) later (leading offset).
// ELEM = bytes per operand element (1: FP8, 2: bf16).  A 128-byte swizzle atom holds 128 / ELEM
// elements, so an MN-major operand of 128 rows is ELEM atoms side by side, kBoxBytes / ELEM apart.
template <bool MN_MAJOR, int ELEM>
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    constexpr uint64_t lbo = MN_MAJOR ? ((kBoxBytes / ELEM) >> 4) : 1;
    constexpr uint64_t sbo = 1024 >> 4;
    return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}
// Byte step of the descriptor start address per tcgen05.mma (32 bytes of K per row).
template <bool MN_MAJOR, int ELEM>
__device__ __forceinline__ uint32_t k_step_bytes() { return MN_MAJOR ? (32u / ELEM) * 128u : 32u; }

// One operand block of 128 rows x 128 bytes of K into shared memory (16 KiB): a K-major operand is
// one TMA box; an MN-major operand is ELEM boxes of 128 / ELEM rows each, side by side.
template <bool MN_MAJOR, int ELEM, bool PAIR>
__device__ __forceinline__ void load_operand(uint32_t dst, const CUtensorMap* map, uint32_t bar, int row0, int k0, int hint,
                                             uint64_t policy) {
    auto box = [&](uint32_t to, int x, int y) {
        if (hint == L2_HINT_NONE) {
            if constexpr (PAIR) tma_load_2d_pair(to, map, bar, x, y); else tma_load_2d(to, map, bar, x, y);
        } else {
            if constexpr (PAIR) tma_load_2d_pair_hint(to, map, bar, x, y, policy); else tma_load_2d_hint(to, map, bar, x, y, policy);
        }
    };
    if constexpr (!MN_MAJOR) {
        box(dst, k0, row0);
    } else {
#pragma unroll
        for (int h = 0; h < ELEM; ++h) box(dst + h * (kBoxBytes / ELEM), row0 + h * (128 / ELEM), k0);
    }
}

__device__ __forceinline__ void tile_coords(const GemmArgs& p, int tile, int& m_tile, int& n_tile) {
    // Bands of `group` tiles along one dimension, walked along that dimension first, so that the CTAs running at
    // the same time share a few A row-blocks and a few B column-blocks in L2.  The band's slice of the operand
    // indexed by the banded dimension is what every wave of the band reads again.
    if (p.band_n == 0) {                 // bands of group m-tiles; the band's A rows are re-read
        const int per_band = p.group * p.num_n_tiles;
        const int band = tile / per_band;
        const int first_m = band * p.group;
        const int rows = min(p.num_m_tiles - first_m, p.group);
        const int in_band = tile - band * per_band;
        m_tile = first_m + in_band % rows;
        n_tile = in_band / rows;
    } else {                             // bands of group n-tiles; the band's B rows are re-read
        const int per_band = p.group * p.num_m_tiles;
        const int band = tile / per_band;
        const int first_n = band * p.group;
        const int cols = min(p.num_n_tiles - first_n, p.group);
        const int in_band = tile - band * per_band;
        n_tile = first_n + in_band % cols;
        m_tile = in_band / cols;
    }
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }
// all epilogue threads agree on one predicate (and of all)
__device__ __forceinline__ bool epi_all(bool v) {
    uint32_t r;
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t"
        "}\n"
        : "=r"(r) : "r"(static_cast<uint32_t>(v)), "n"(kEpiThreads) : "memory");
    return r != 0;
}

__device__ __forceinline__ float inv_or_one(const float* s) { return s ? __fdiv_rn(1.0f, *s) : 1.0f; }

// ---------------------------------------------------------------- epilogues
// Eight warps drain an accumulator: warp (quad, half) owns TMEM lanes [32 quad, 32 quad + 32) - one
// row per thread - and one half of the tile's columns, in chunks of 32.  Every chunk is worked
// through in stages over all 32 elements (independent instructions back to back), and a thread's
// 32 consecutive outputs leave as whole 32-byte sectors when the rows are 32-byte aligned (wide).

// 32 fp32 values of one row -> global, columns [c0, c0 + 32) of an N-column matrix, 8 at a time
__device__ __forceinline__ void store_f32x32(const GemmArgs& p, const float (&v)[32], int m, int c0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const int col = c0 + 8 * q;
        if (col < p.N) {
            float* dst = col < p.n_split ? p.out_f32_0 + static_cast<int64_t>(m) * p.ld_out + col
                                         : p.out_f32_1 + static_cast<int64_t>(m) * p.ld_out + (col - p.n_split);
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) w[e] = __float_as_uint(v[8 * q + e]);
            if (p.wide) {
                st_global_v8(dst, w);
            } else {
                st_global_v4(dst, w[0], w[1], w[2], w[3]);
                st_global_v4(dst + 4, w[4], w[5], w[6], w[7]);
            }
        }
    }
}

__device__ __forceinline__ void epilogue_f32(const GemmArgs& p, uint32_t taddr, int half, int m, int n0, float dq) {
    const bool row_ok = m < p.M;
#pragma unroll 1
    for (int jj = 0; jj < 4; ++jj) {
        const int j = 4 * half + jj;
        const int c0 = n0 + 32 * j;
        if (c0 >= p.N) break;
        uint32_t r[32];
        tmem_ld32(taddr + 32 * j, r);
        tmem_ld_wait();
        if (!row_ok) continue;
        float v[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __fmul_rn(__uint_as_float(r[e]), dq);
        store_f32x32(p, v, m, c0);
    }
}

// The same through shared memory: the thread writes its row's 32 values into one of the warp's NBUF staging blocks
// (16-byte piece j of row r at piece j ^ (r & 7): the 128-byte swizzle, so the writes are free of bank conflicts and
// the block is what a swizzled tensor-map box expects), one lane sends the block off as a bulk tensor store.  Rows
// past M and columns past the output's width are cut off by the tensor map.  A chunk that straddles the boundary
// between the two outputs of a split output is stored directly.  `blocks_sent` counts the warp's blocks.
template <int NBUF>
__device__ __forceinline__ void epilogue_f32_staged(const GemmArgs& p, const CUtensorMap* out0, const CUtensorMap* out1,
                                                    uint32_t warp_stage_addr, uint32_t& blocks_sent, uint32_t taddr, int lane,
                                                    int half, int m, int row0, int n0, float dq) {
    const bool row_ok = m < p.M;
#pragma unroll 1
    for (int jj = 0; jj < 4; ++jj) {
        const int j = 4 * half + jj;
        const int c0 = n0 + 32 * j;
        if (c0 >= p.N) break;
        uint32_t r[32];
        tmem_ld32(taddr + 32 * j, r);
        tmem_ld_wait();
        float v[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __fmul_rn(__uint_as_float(r[e]), dq);
        if (c0 < p.n_split && c0 + 32 > p.n_split) {       // straddles the two outputs
            if (row_ok) store_f32x32(p, v, m, c0);
            continue;
        }
        const uint32_t block = warp_stage_addr + (blocks_sent % NBUF) * kStoreBlockBytes;
        ++blocks_sent;
        if (lane == 0) tma_store_wait_read<NBUF - 1>();    // the store that used this block last has read it
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 8; ++q)
            st_shared_v4(block + static_cast<uint32_t>(lane) * 128u + static_cast<uint32_t>((q ^ (lane & 7)) * 16),
                         __float_as_uint(v[4 * q]), __float_as_uint(v[4 * q + 1]), __float_as_uint(v[4 * q + 2]), __float_as_uint(v[4 * q + 3]));
        fence_smem_to_async_proxy();
        __syncwarp();
        if (lane == 0) {
            if (c0 < p.n_split) tma_store_2d(out0, block, c0, row0);
            else tma_store_2d(out1, block, c0 - p.n_split, row0);
            tma_store_commit();
        }
    }
}

// 16 floats -> 16 bf16 (32 bytes) at dst, columns guarded by the caller
__device__ __forceinline__ void store_bf16x16(uint16_t* dst, const float* v, bool wide) {
    uint32_t w[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) w[e] = cvt_bf16x2(v[2 * e], v[2 * e + 1]);
    if (wide) {
        st_global_v8(dst, w);
    } else {
        st_global_v4(dst, w[0], w[1], w[2], w[3]);
        st_global_v4(dst + 8, w[4], w[5], w[6], w[7]);
    }
}

__device__ __forceinline__ void epilogue_bf16(const GemmArgs& p, uint32_t taddr, int half, int m, int n0, float dq) {
    const bool row_ok = m < p.M;
#pragma unroll 1
    for (int jj = 0; jj < 4; ++jj) {
        const int j = 4 * half + jj;
        const int c0 = n0 + 32 * j;
        if (c0 >= p.N) break;
        uint32_t r[32];
        tmem_ld32(taddr + 32 * j, r);
        tmem_ld_wait();
        if (!row_ok) continue;
        float v[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __fmul_rn(__uint_as_float(r[e]), dq);
        uint16_t* dst = p.out_bf16 + static_cast<int64_t>(m) * p.ld_out + c0;
        store_bf16x16(dst, v, p.wide);
        if (c0 + 16 < p.N) store_bf16x16(dst + 16, v + 16, p.wide);
    }
}

// Split contraction: this CTA pair holds one of split_k partial sums of the tile.  The warp writes its raw fp32
// partial (32 rows x 128 columns) to the workspace and counts itself; the warp that finds all the others of its
// region already counted adds the split_k partials in split order - whichever warp that is, the sum is the same -
// applies the dequantisation and writes the output.  Nothing waits: every warp but the last just leaves.
template <int EPI>
__device__ __forceinline__ void epilogue_split(const GemmArgs& p, uint32_t taddr, int lane, int half, unsigned int* counter,
                                               int split, int m, int n0, float dq) {
    const bool row_ok = m < p.M;
    float* mine = p.partial + (static_cast<int64_t>(split) * p.M + m) * p.N;
#pragma unroll 1
    for (int jj = 0; jj < 4; ++jj) {
        const int c0 = n0 + 32 * (4 * half + jj);
        if (c0 >= p.N) break;
        uint32_t r[32];
        tmem_ld32(taddr + 32 * (4 * half + jj), r);
        tmem_ld_wait();
        if (!row_ok) continue;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (c0 + 8 * q >= p.N) break;
            const uint32_t w[8] = {r[8 * q], r[8 * q + 1], r[8 * q + 2], r[8 * q + 3], r[8 * q + 4], r[8 * q + 5], r[8 * q + 6], r[8 * q + 7]};
            st_global_v8(mine + c0 + 8 * q, w);
        }
    }
    __threadfence();                       // this lane's partials are visible device-wide before the count
    __syncwarp();
    unsigned int before = 0;
    if (lane == 0) before = atomicAdd(counter, 1u);
    before = __shfl_sync(0xffffffffu, before, 0);
    if (before != static_cast<unsigned int>(p.split_k - 1)) return;
    __threadfence();                       // the other splits' partials, counted before ours, are visible now
    if (lane == 0) *counter = 0u;          // every split has counted: ready for the next launch
    if (!row_ok) return;
#pragma unroll 1
    for (int jj = 0; jj < 4; ++jj) {
        const int c0 = n0 + 32 * (4 * half + jj);
        if (c0 >= p.N) break;
        float v[32] = {};
        // two splits' rows are fetched at a time, so that their trips to L2 overlap; added in split order
        for (int s = 0; s < p.split_k; s += 2) {
            const bool two = s + 1 < p.split_k;
            const float* first = p.partial + (static_cast<int64_t>(s) * p.M + m) * p.N + c0;
            const float* second = first + static_cast<int64_t>(p.M) * p.N;
            uint32_t w0[4][8], w1[4][8];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const bool in = c0 + 8 * q < p.N;
                if (in) ld_global_cg_v8(first + 8 * q, w0[q]);
                if (in && two) ld_global_cg_v8(second + 8 * q, w1[q]);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (c0 + 8 * q >= p.N) break;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float t = s == 0 ? __uint_as_float(w0[q][e]) : __fadd_rn(v[8 * q + e], __uint_as_float(w0[q][e]));
                    if (two) t = __fadd_rn(t, __uint_as_float(w1[q][e]));
                    v[8 * q + e] = t;
                }
            }
        }
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __fmul_rn(v[e], dq);
        if constexpr (EPI == EPI_F32) {
            store_f32x32(p, v, m, c0);
        } else {
            uint16_t* dst = p.out_bf16 + static_cast<int64_t>(m) * p.ld_out + c0;
            store_bf16x16(dst, v, p.wide);
            if (c0 + 16 < p.N) store_bf16x16(dst + 16, v + 16, p.wide);
        }
    }
}

// bf16 output through shared memory (see kStoreBlockBytesBf16): the thread writes its row's 32 values as four 16-byte
// pieces (piece j of row r at piece j ^ ((r >> 1) & 3): the 64-byte swizzle), one lane sends the block off as a bulk
// tensor store; rows past M and columns past N are cut off by the tensor map.
__device__ __forceinline__ void epilogue_bf16_staged(const GemmArgs& p, const CUtensorMap* out, uint32_t warp_stage_addr,
                                                     uint32_t& blocks_sent, uint32_t taddr, int lane, int half, int row0, int n0,
                                                     float dq) {
#pragma unroll 1
    for (int jj = 0; jj < 4; ++jj) {
        const int j = 4 * half + jj;
        const int c0 = n0 + 32 * j;
        if (c0 >= p.N) break;
        uint32_t r[32];
        tmem_ld32(taddr + 32 * j, r);
        tmem_ld_wait();
        uint32_t w[16];
#pragma unroll
        for (int e = 0; e < 16; ++e)
            w[e] = cvt_bf16x2(__fmul_rn(__uint_as_float(r[2 * e]), dq), __fmul_rn(__uint_as_float(r[2 * e + 1]), dq));
        const uint32_t block = warp_stage_addr + (blocks_sent & 1u) * kStoreBlockBytesBf16;
        ++blocks_sent;
        if (lane == 0) tma_store_wait_read<1>();           // the store that used this block last has read it
        __syncwarp();
        const uint32_t sw = static_cast<uint32_t>((lane >> 1) & 3);
#pragma unroll
        for (int q = 0; q < 4; ++q)
            st_shared_v4(block + static_cast<uint32_t>(lane) * 64u + ((static_cast<uint32_t>(q) ^ sw) * 16u),
                         w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
        fence_smem_to_async_proxy();
        __syncwarp();
        if (lane == 0) {
            tma_store_2d(out, block, c0, row0);
            tma_store_commit();
        }
    }
}

// 32 floats -> 32 FP8 codes (32 bytes) at dst; the second 16 only if `both`
template <int FMT>
__device__ __forceinline__ void store_fp8x32(uint8_t* dst, const float (&v)[32], bool both, bool wide) {
    uint32_t w[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) w[e] = cvt_fp8x4<FMT>(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
    if (both && wide) {
        st_global_v8(dst, w);
    } else {
        st_global_v4(dst, w[0], w[1], w[2], w[3]);
        if (both) st_global_v4(dst + 16, w[4], w[5], w[6], w[7]);
    }
}

// Forward: accumulator columns [0,128) are G = x W2 (gate), [128,256) are U = x W1 (linear) of the
// same 128 channels; this warp takes channels [64 half, 64 half + 64) of them.
// H = U * G * sigma(G); per-channel max |H|; Hq = Q_e4m3(H * s_i); G, U kept for backward as bf16, or
// as E4M3 codes Q(sgu G), Q(sgu U) with their common maximum (GU8).  H itself never leaves the SM.
template <bool GU8>
__device__ __forceinline__ void epilogue_swiglu_fwd(const GemmArgs& p, SmemTail* tail, uint32_t taddr, int lane,
                                                    int half, int m, int n0, float dq, float sgu, float& gu_max) {
    const bool row_ok = m < p.M;
    const int f = p.N;
#pragma unroll 1
    for (int jj = 0; jj < 2; ++jj) {
        const int j = 2 * half + jj;
        const int c0 = n0 + 32 * j;
        if (c0 >= f) break;
        uint32_t g_raw[32], u_raw[32];
        tmem_ld32(taddr + 32 * j, g_raw);
        tmem_ld32(taddr + 128 + 32 * j, u_raw);
        tmem_ld_wait();
        float g[32], u[32], h[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) {
            g[e] = __fmul_rn(__uint_as_float(g_raw[e]), dq);
            u[e] = __fmul_rn(__uint_as_float(u_raw[e]), dq);
        }
#pragma unroll
        for (int e = 0; e < 32; ++e) h[e] = ex2_approx(__fmul_rn(g[e], -1.4426950408889634f));
#pragma unroll
        for (int e = 0; e < 32; ++e) h[e] = rcp_approx(__fadd_rn(1.0f, h[e]));          // sigma(G)
#pragma unroll
        for (int e = 0; e < 32; ++e) h[e] = __fmul_rn(u[e], __fmul_rn(g[e], h[e]));       // H
        if (p.amax_h != nullptr) {
            float colmax = 0.0f;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                const float cm = warp_max_nonneg(fabsf(h[e]));   // max over this warp's 32 rows
                if (lane == e) colmax = cm;
            }
            atomicMax(&tail->amax_tile[32 * j + lane], __float_as_uint(colmax));
        }
        if constexpr (GU8) {              // rows past M and columns past f hold zeros
            float mx = gu_max;
#pragma unroll
            for (int e = 0; e < 32; ++e) mx = fmaxf(mx, fmaxf(fabsf(g[e]), fabsf(u[e])));
            gu_max = mx;
        }
        if (!p.store || !row_ok) continue;
        const bool both = c0 + 16 < f;
        if constexpr (GU8) {
            uint8_t* grow = p.gu8 + static_cast<int64_t>(m) * 2 * f + c0;
            float t[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) t[e] = __fmul_rn(g[e], sgu);
            store_fp8x32<FP8MLP_E4M3>(grow, t, both, p.wide);
#pragma unroll
            for (int e = 0; e < 32; ++e) t[e] = __fmul_rn(u[e], sgu);
            store_fp8x32<FP8MLP_E4M3>(grow + f, t, both, p.wide);
        }
        if (!GU8 && p.gu != nullptr) {
            uint16_t* grow = p.gu + static_cast<int64_t>(m) * 2 * f + c0;
            store_bf16x16(grow, g, true);
            store_bf16x16(grow + f, u, true);
            if (both) {
                store_bf16x16(grow + 16, g + 16, true);
                store_bf16x16(grow + f + 16, u + 16, true);
            }
        }
        if (p.hb != nullptr) {           // the last layer runs in bf16: H leaves unscaled, rounded to bf16
            uint16_t* hrow = p.hb + static_cast<int64_t>(m) * f + c0;
            store_bf16x16(hrow, h, true);
            if (both) store_bf16x16(hrow + 16, h + 16, true);
            continue;
        }
#pragma unroll
        for (int e = 0; e < 32; ++e) h[e] = __fmul_rn(h[e], tail->s_tile[0][32 * j + e]);
        store_fp8x32<FP8MLP_E4M3>(p.hq + static_cast<int64_t>(m) * f + c0, h, both, p.wide);
    }
}

// Backward: accumulator = dY W3'^T for 256 channels, worked through in four chunks of 64 channels; of
// each chunk this warp takes channels [32 half, 32 half + 32).  The saved bf16 G and U of those 32 channels
// arrive in a ring slot of their own (loader warp, TMA, 64-byte swizzle: the 16-byte piece j of row r sits at
// piece j ^ ((r >> 1) & 3)), read by the four warps of this column half; the thread copies its row's 64 + 64
// bytes to registers and hands the slot back (the warps of the other half pass the slot without reading).  Kept as E4M3 codes instead (p.gu8), a slot holds all 64 channels
// of the chunk, shared by all eight warps; the thread copies 32 + 32 bytes and G = code * (1 / sgu).
// dH = acc * dq (* s_i with Smooth-SwiGLU); dU = dH * G sigma(G);
// dG = dH * U * sigma(G) (1 + G (1 - sigma(G))); max of |dG|, |dU|; dZq = Q_e5m2([dG | dU] * sdz).
// gu_fill: the ring fills this warp has passed (fills are numbered as the loader issues them).
// Returns false if a wait ran out.  GU8: the saved activations are E4M3 codes (p.gu8), else bf16 (p.gu).
template <bool GU8>
__device__ __forceinline__ bool epilogue_swiglu_bwd(const GemmArgs& p, SmemTail* tail, uint32_t gu_base, uint32_t& gu_fill,
                                                    const float* s_tile, uint32_t taddr, int lane, int half, int row,
                                                    int m, int n0, float dq, float sdz, float inv_sgu,
                                                    volatile int* abort_flag, float& run_max) {
    const bool row_ok = m < p.M;
    constexpr bool gu8 = GU8;
    const int f = p.N;
    float local_max = 0.0f;
    // A power-of-two sdz (what fp8mlp_update_scales produces) commutes with every rounding below, so it
    // is folded into the dequantisation factor: dG, dU come out already scaled, bit for bit the same as
    // scaling them at the end, and the running maximum is scaled back once.
    const bool fold = (__float_as_uint(sdz) & 0x007FFFFFu) == 0u && sdz > 1.0e-30f && sdz < 1.0e30f;
    if (fold) dq = __fmul_rn(dq, sdz);
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
        const int col = 64 * c + 32 * half;            // first of this warp's 32 accumulator columns
        const int c0 = n0 + col;
        uint4 gq[4], uq[4];
        // Every warp passes every fill of the ring in order, whether the fill is for its column half or not: a
        // barrier's parity only tells consecutive phases apart, so a warp that skipped a fill could take a slot's
        // previous phase for the one it waits for (loads do not land in the order they were issued).
#pragma unroll
        for (int k = 0; k < (gu8 ? 1 : 2); ++k) {
            const uint32_t slot = gu_fill % kGuSlots, phase = (gu_fill / kGuSlots) & 1u;
            // the warp leaves together or not at all: a wait that ran out for some lanes only would split it
            // between the failure path and the warp-wide instructions below
            const bool landed = mbar_wait(smem_u32(&tail->gu_full[slot]), phase, abort_flag, p.status);
            if (!__all_sync(0xffffffffu, landed)) return false;
            const uint32_t rbase = gu_base + slot * kGuSlotBytes + static_cast<uint32_t>(row) * 64u;
            const uint32_t sw = static_cast<uint32_t>((row >> 1) & 3);
            if constexpr (gu8) {
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const uint32_t off = ((static_cast<uint32_t>(2 * half + i)) ^ sw) * 16u;
                    gq[i] = ld_shared_v4(rbase + off);
                    uq[i] = ld_shared_v4(rbase + kGuBoxBytes + off);
                }
                gq[2] = gq[3] = uq[2] = uq[3] = make_uint4(0u, 0u, 0u, 0u);
            } else if (k == half) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t off = (static_cast<uint32_t>(i) ^ sw) * 16u;
                    gq[i] = ld_shared_v4(rbase + off);
                    uq[i] = ld_shared_v4(rbase + kGuBoxBytes + off);
                }
            }
            // The slot goes back to the loader, whose refill writes it through the bulk-copy engine (the async proxy),
            // while these reads are ordinary (generic-proxy) loads: the two are only ordered by a proxy fence.  Without
            // it the refill now and then overwrote a 16-byte piece before a lane had read it - 8 wrong channels in one
            // row, a few times per 10^9 pieces, found by repeating a step and comparing bits.  Consuming the loaded
            // words first makes each lane hold its data before it fences.
            if (gu8 || k == half) {
                uint32_t seen = 0;
#pragma unroll
                for (int i = 0; i < (gu8 ? 2 : 4); ++i)
                    seen ^= gq[i].x ^ gq[i].y ^ gq[i].z ^ gq[i].w ^ uq[i].x ^ uq[i].y ^ uq[i].z ^ uq[i].w;
                asm volatile("" ::"r"(seen) : "memory");
                fence_smem_to_async_proxy();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tail->gu_empty[slot]));     // this warp is done with the slot
            ++gu_fill;
        }
        if (c0 >= f) continue;
        uint32_t acc[32];
        tmem_ld32(taddr + col, acc);
        tmem_ld_wait();
        const uint32_t* gw = reinterpret_cast<const uint32_t*>(gq);
        const uint32_t* uw = reinterpret_cast<const uint32_t*>(uq);
        // element pairs (2q, 2q+1) travel as one 64-bit register through the multiplies and adds
        float dg[32], du[32];
        f32x2 dh2[16], g2[16], sig2[16];
        const f32x2 dq2 = pack2(dq, dq), one2 = pack2(1.0f, 1.0f), nl2 = pack2(-1.4426950408889634f, -1.4426950408889634f);
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            dh2[q] = mul2(pack2(__uint_as_float(acc[2 * q]), __uint_as_float(acc[2 * q + 1])), dq2);
            if (p.smooth) dh2[q] = mul2(dh2[q], pack2(s_tile[col + 2 * q], s_tile[col + 2 * q + 1]));
            if constexpr (gu8) {
                float a, b;
                e4m3x2_to_f32(gw[q >> 1] >> (16 * (q & 1)), a, b);
                g2[q] = mul2(pack2(a, b), pack2(inv_sgu, inv_sgu));
            } else {
                g2[q] = pack2(bf16_lo(gw[q]), bf16_hi(gw[q]));
            }
        }
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            float a, b;
            unpack2(mul2(g2[q], nl2), a, b);
            sig2[q] = pack2(ex2_approx(a), ex2_approx(b));
        }
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            float a, b;
            unpack2(add2(one2, sig2[q]), a, b);
            sig2[q] = pack2(rcp_approx(a), rcp_approx(b));                                  // sigma(G)
        }
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            f32x2 u2;
            if constexpr (gu8) {
                float a, b;
                e4m3x2_to_f32(uw[q >> 1] >> (16 * (q & 1)), a, b);
                u2 = mul2(pack2(a, b), pack2(inv_sgu, inv_sgu));
            } else {
                u2 = pack2(bf16_lo(uw[q]), bf16_hi(uw[q]));
            }
            const f32x2 du_2 = mul2(dh2[q], mul2(g2[q], sig2[q]));
            const f32x2 t1 = add2(one2, mul2(g2[q], sub2(one2, sig2[q])));
            const f32x2 dg_2 = mul2(mul2(dh2[q], u2), mul2(sig2[q], t1));
            unpack2(du_2, du[2 * q], du[2 * q + 1]);
            unpack2(dg_2, dg[2 * q], dg[2 * q + 1]);
            local_max = fmaxf(local_max, fmaxf(fmaxf(fabsf(dg[2 * q]), fabsf(dg[2 * q + 1])),
                                               fmaxf(fabsf(du[2 * q]), fabsf(du[2 * q + 1]))));
        }
        if (!p.store || !row_ok) continue;
        if (!fold) {
            const f32x2 sdz2 = pack2(sdz, sdz);
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                unpack2(mul2(pack2(dg[2 * q], dg[2 * q + 1]), sdz2), dg[2 * q], dg[2 * q + 1]);
                unpack2(mul2(pack2(du[2 * q], du[2 * q + 1]), sdz2), du[2 * q], du[2 * q + 1]);
            }
        }
        uint8_t* zrow = p.dzq + static_cast<int64_t>(m) * 2 * f + c0;
        const bool both = c0 + 16 < f;
        store_fp8x32<FP8MLP_E5M2>(zrow, dg, both, p.wide);
        store_fp8x32<FP8MLP_E5M2>(zrow + f, du, both, p.wide);
    }
    run_max = fmaxf(run_max, fold ? __fmul_rn(local_max, __fdiv_rn(1.0f, sdz)) : local_max);
    return true;
}

// ---------------------------------------------------------------- the kernel
// PAIR = false: one CTA per 128 x 256 tile.  PAIR = true: a cluster of two CTAs per 256 x 256 tile
// (tcgen05 cta_group::2): rank r loads rows [128 r, 128 r + 128) of the A tile and of the B tile,
// rank 0 issues the MMAs for both, and each CTA drains its own 128 rows of the accumulator.
// GU8 (SwiGLU epilogues only): the activations saved for backward are E4M3 codes (args.gu8), not bf16.
template <int EPI, bool A_MN, bool B_MN, bool PAIR, int ELEM, bool WIDEN, bool GU8>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
            const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmG,
            const __grid_constant__ CUtensorMap tmU, const GemmArgs p) {
    constexpr int kStages = Plan<PAIR, EPI, WIDEN>::kStages;
    constexpr int kStageBytes = Plan<PAIR, EPI, WIDEN>::kStageBytes;
    constexpr int kTileM = Plan<PAIR, EPI, WIDEN>::kTileM;
    static_assert(!WIDEN || (PAIR && (EPI == EPI_F32 || EPI == EPI_BF16)), "wide tiles: CTA pairs, plain epilogues");
    static_assert(!GU8 || EPI == EPI_SWIGLU_BWD || EPI == EPI_SWIGLU_FWD, "GU8 belongs to the SwiGLU epilogues");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;         // swizzle atoms need 1024-byte alignment
    uint8_t* tiles_ptr = smem_raw + (tiles_addr - raw_addr);
    constexpr uint32_t kRingBytes = EPI == EPI_SWIGLU_BWD ? kGuSlots * kGuSlotBytes : 0;
    const uint32_t gu_base = tiles_addr + kStages * kStageBytes;     // ring of saved G, U chunks (backward only)
    const uint32_t store_base = tiles_addr + static_cast<uint32_t>(p.stages) * kStageBytes;   // staging blocks of the fp32 output, if used
    using Tail = TailOf<EPI>;
    const uint32_t own_store_base = gu_base + kRingBytes;            // staging blocks of the wide-tile bf16 output
    Tail* tail = reinterpret_cast<Tail*>(tiles_ptr + size_t(kStages) * kStageBytes + kRingBytes + OwnStoreBytes<EPI, WIDEN>::value);
    const uint32_t n_stages = static_cast<uint32_t>(p.stages);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // a work item is a tile, or with a split contraction one of a tile's split_k shares (shares of a tile are
    // neighbouring items, so they run at the same time on neighbouring CTA pairs)
    const int num_tiles = p.num_m_tiles * p.num_n_tiles * p.split_k;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;             // rank in the CTA pair
    const int first_tile = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
    const int tile_step = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
    volatile int* abort_flag = &tail->abort;

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB0);
        tma_prefetch_desc(&tmB1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&tail->full[s]), 1);
            mbar_init(smem_u32(&tail->empty[s]), 1);
        }
        for (int b = 0; b < kGuSlots; ++b) {
            mbar_init(smem_u32(&tail->gu_full[b]), 1);
            mbar_init(smem_u32(&tail->gu_empty[b]), kEpiThreads / 32);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&tail->tmem_full[b]), 1);
            mbar_init(smem_u32(&tail->tmem_empty[b]), (PAIR ? 2 : 1) * (kEpiThreads / 32));
        }
        tail->abort = 0;
        mbar_init_fence();
    }
    if (warp == 1) {
        if constexpr (PAIR) { tmem_alloc_pair(smem_u32(&tail->tmem_base), kTmemCols); tmem_relinquish_pair(); }
        else { tmem_alloc(smem_u32(&tail->tmem_base), kTmemCols); tmem_relinquish(); }
    }
    tc_fence_before();
    if constexpr (PAIR) cluster_sync_all(); else __syncthreads();   // barriers of both CTAs are ready
    tc_fence_after();
    const uint32_t tmem_base = tail->tmem_base;
    // Everything above touched only this CTA's shared and tensor memory and may have run while the previous
    // kernel of the stream was still finishing; from here on its results are needed.
    grid_dependency_wait();
    grid_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            const CUtensorMap* tmB = (PAIR && rank != 0) ? &tmB1 : &tmB0;
            const uint64_t pol_a = l2_policy(p.hint_a), pol_b = l2_policy(p.hint_b);
            int it = 0;
            for (int item = first_tile; ok && item < num_tiles; item += tile_step, ++it) {
                int m_tile, n_tile;
                const int tile = item / p.split_k, split = item - tile * p.split_k;
                tile_coords(p, tile, m_tile, n_tile);
                const int m0 = m_tile * kTileM + static_cast<int>(rank) * kBlockM;
                const int nb0 = n_tile * p.n_tile_cols + (PAIR ? static_cast<int>(rank) * p.b1_offset : 0);
                const int nb1 = nb0 + p.b1_offset;
                const int kb_begin = split * p.kb_per_split, kb_end = min(p.num_k_blocks, kb_begin + p.kb_per_split);
                // Every other wave of tiles (a CTA's it-th tile belongs to the it-th wave) walks the contraction
                // backwards: what L2 still holds when a wave ends is the end of the contraction, so the next wave meets
                // the operand slice it shares with this one where it is still cached.  Only the order of the fp32 sum
                // changes, and it is the same in every launch of the same problem.
                const bool backwards = p.k_alternate && (it & 1);
                for (int step = kb_begin; step < kb_end; ++step) {
                    const int kb = backwards ? kb_begin + kb_end - 1 - step : step;
                    if (!mbar_wait(smem_u32(&tail->empty[stage]), phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    const uint32_t dst = tiles_addr + stage * kStageBytes;
                    const int k0 = kb * (kBlockK / ELEM);          // in elements
                    if constexpr (PAIR) {
                        // both CTAs' bytes are counted on rank 0's barrier, armed by rank 0 for both
                        const uint32_t bar = mapa_shared(smem_u32(&tail->full[stage]), 0);
                        if (rank == 0) mbar_expect_tx(smem_u32(&tail->full[stage]), 2 * kStageBytes);
                        load_operand<A_MN, ELEM, true>(dst, &tmA, bar, m0, k0, p.hint_a, pol_a);
                        load_operand<B_MN, ELEM, true>(dst + kBoxBytes, tmB, bar, nb0, k0, p.hint_b, pol_b);
                        if constexpr (WIDEN) load_operand<B_MN, ELEM, true>(dst + 2 * kBoxBytes, tmB, bar, nb0 + kBlockN, k0, p.hint_b, pol_b);
                    } else {
                        const uint32_t bar = smem_u32(&tail->full[stage]);
                        mbar_expect_tx(bar, kStageBytes);
                        load_operand<A_MN, ELEM, false>(dst, &tmA, bar, m0, k0, p.hint_a, pol_a);
                        load_operand<B_MN, ELEM, false>(dst + kBoxBytes, &tmB0, bar, nb0, k0, p.hint_b, pol_b);
                        load_operand<B_MN, ELEM, false>(dst + 2 * kBoxBytes, &tmB1, bar, nb1, k0, p.hint_b, pol_b);
                    }
                    if (++stage == n_stages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (CTA pair: rank 0 only)
        if (lane == 0 && rank == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            int it = 0;
            for (int item = first_tile; ok && item < num_tiles; item += tile_step, ++it) {
                const uint32_t acc = WIDEN ? 0u : (it & 1), acc_phase = WIDEN ? (it & 1) : ((it >> 1) & 1);
                if (!mbar_wait(smem_u32(&tail->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, p.status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kBlockN;
                const int split = item % p.split_k;
                const int kb_begin = split * p.kb_per_split, kb_end = min(p.num_k_blocks, kb_begin + p.kb_per_split);
                for (int kb = kb_begin; kb < kb_end; ++kb) {
                    if (!mbar_wait(smem_u32(&tail->full[stage]), phase, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = tiles_addr + stage * kStageBytes;
                    const uint32_t b_addr = a_addr + kBoxBytes;
#pragma unroll
                    for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                        const uint64_t da = smem_desc<A_MN, ELEM>(a_addr + k * k_step_bytes<A_MN, ELEM>());
                        const uint64_t db = smem_desc<B_MN, ELEM>(b_addr + k * k_step_bytes<B_MN, ELEM>());
                        const uint32_t accum = (kb != kb_begin || k != 0) ? 1u : 0u;
                        if constexpr (WIDEN) {       // second half of the 512 columns: same A, the stage's other B block
                            const uint64_t db1 = smem_desc<B_MN, ELEM>(b_addr + kBoxBytes + k * k_step_bytes<B_MN, ELEM>());
                            umma_f8_pair(d_tmem, da, db, p.idesc, accum);
                            umma_f8_pair(d_tmem + kBlockN, da, db1, p.idesc, accum);
                        } else if constexpr (ELEM == 1) {
                            if constexpr (PAIR) umma_f8_pair(d_tmem, da, db, p.idesc, accum); else umma_f8(d_tmem, da, db, p.idesc, accum);
                        } else {
                            if constexpr (PAIR) umma_f16_pair(d_tmem, da, db, p.idesc, accum); else umma_f16(d_tmem, da, db, p.idesc, accum);
                        }
                    }
                    // frees the stage (in both CTAs) once these MMAs have read it
                    if constexpr (PAIR) umma_commit_pair(smem_u32(&tail->empty[stage]));
                    else umma_commit(smem_u32(&tail->empty[stage]));
                    if (++stage == n_stages) { stage = 0; phase ^= 1u; }
                }
                if (ok) {
                    if constexpr (PAIR) umma_commit_pair(smem_u32(&tail->tmem_full[acc]));
                    else umma_commit(smem_u32(&tail->tmem_full[acc]));
                }
            }
        }
    } else if (warp == 10) {
        // ------------------------------------------------------------ loader of the saved G, U (backward only)
        if constexpr (EPI == EPI_SWIGLU_BWD) {
            if (lane == 0) {
                tma_prefetch_desc(&tmG);
                tma_prefetch_desc(&tmU);
                uint32_t count = 0;
                bool ok = true;
                for (int tile = first_tile; ok && tile < num_tiles; tile += tile_step) {
                    int m_tile, n_tile;
                    tile_coords(p, tile, m_tile, n_tile);
                    const int m0 = m_tile * kTileM + static_cast<int>(rank) * kBlockM;
                    const int n0 = n_tile * p.n_tile_cols;
                    // per fill 64 bytes of every row of G and of U: 32 channels as bf16 (8 fills a tile, alternating
                    // between the two column halves of a 64-channel chunk) or 64 channels as E4M3 codes (4 fills)
                    constexpr int n_fills = GU8 ? 4 : 8, per_fill = GU8 ? 64 : 32;
                    for (int c = 0; c < n_fills; ++c, ++count) {
                        const uint32_t slot = count % kGuSlots, phase = (count / kGuSlots) & 1u;
                        if (!mbar_wait(smem_u32(&tail->gu_empty[slot]), phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
                        const uint32_t bar = smem_u32(&tail->gu_full[slot]);
                        const uint32_t dst = gu_base + slot * kGuSlotBytes;
                        mbar_expect_tx(bar, kGuSlotBytes);
                        tma_load_2d(dst, &tmG, bar, n0 + per_fill * c, m0);        // columns past f read as zeros
                        tma_load_2d(dst + kGuBoxBytes, &tmU, bar, n0 + per_fill * c, m0);
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9)
        const int quad = warp & 3;                     // TMEM lanes [32*quad, 32*quad+32) belong to this warp
        const int half = (warp - 2) >> 2;              // which half of the tile's columns
        const int row = quad * 32 + lane;
        const int et = (warp - 2) * 32 + lane;         // index among the epilogue threads
        const float dq0 = __fmul_rn(inv_or_one(p.s0), inv_or_one(p.s1));
        float sdz = 1.0f;
        if constexpr (EPI == EPI_SWIGLU_BWD) sdz = *p.sdz;
        float run_max = 0.0f;
        float sgu = 1.0f, inv_sgu = 1.0f, gu_max = 0.0f;     // saved G, U as E4M3 codes: scale, reciprocal, running max
        if constexpr (EPI == EPI_SWIGLU_FWD || EPI == EPI_SWIGLU_BWD) {
            if constexpr (GU8) { sgu = *p.s_gu; inv_sgu = __fdiv_rn(1.0f, sgu); }
        }
        // staging blocks per warp for the fp32 output: what two lent stages hold, shared by the eight epilogue warps
        constexpr int kStoreBlocks = (kStagesLentToStores * kStageBytes) / ((kEpiThreads / 32) * kStoreBlockBytes) >= 2 ? 2 : 1;
        uint32_t blocks_sent = 0;
        uint32_t gu_fill = 0;                          // ring fills of saved G, U this warp has passed (backward)
        int it = 0;
        for (int item = first_tile; item < num_tiles; item += tile_step, ++it) {
            int m_tile, n_tile;
            const int tile = item / p.split_k, split = item - tile * p.split_k;
            tile_coords(p, tile, m_tile, n_tile);
            const int m = m_tile * kTileM + static_cast<int>(rank) * kBlockM + row;
            const int n0 = n_tile * p.n_tile_cols;
            const uint32_t acc = WIDEN ? 0u : (it & 1), acc_phase = WIDEN ? (it & 1) : ((it >> 1) & 1);
            if constexpr (EPI == EPI_SWIGLU_FWD) {
                if (et < 128) {
                    tail->s_tile[0][et] = (n0 + et) < p.N ? p.s_h[n0 + et] : 1.0f;
                    tail->amax_tile[et] = 0u;
                }
            }
            if constexpr (EPI == EPI_SWIGLU_BWD) tail->s_tile[acc][et] = (n0 + et) < p.N ? p.s_h[n0 + et] : 1.0f;
            const bool got = mbar_wait(smem_u32(&tail->tmem_full[acc]), acc_phase, abort_flag, p.status);
            if (!epi_all(got)) break;                  // also orders the s_tile / amax_tile writes above
            tc_fence_after();
            const uint32_t taddr = tmem_base + acc * kBlockN + (static_cast<uint32_t>(quad * 32) << 16);
            if constexpr (EPI == EPI_F32) {
                float dq = dq0;
                if (p.row_s != nullptr)
                    dq = __fmul_rn(inv_or_one(p.s0), m < p.M ? __fdiv_rn(1.0f, p.row_s[m]) : 1.0f);
                if (!WIDEN && p.split_k > 1)
                    epilogue_split<EPI_F32>(p, taddr, lane, half, p.tile_counters + tile * 16 + rank * 8 + (warp - 2), split, m, n0, dq);
                else if (!WIDEN && p.tma_store)
                    epilogue_f32_staged<kStoreBlocks>(p, &tmG, &tmU, store_base + static_cast<uint32_t>(warp - 2) * (kStoreBlocks * kStoreBlockBytes),
                                                      blocks_sent, taddr, lane, half, m, m - lane, n0, dq);
                else epilogue_f32(p, taddr, half, m, n0, dq);
                if constexpr (WIDEN) epilogue_f32(p, taddr + kBlockN, half, m, n0 + kBlockN, dq);
            } else if constexpr (EPI == EPI_BF16) {
                if (!WIDEN && p.split_k > 1)
                    epilogue_split<EPI_BF16>(p, taddr, lane, half, p.tile_counters + tile * 16 + rank * 8 + (warp - 2), split, m, n0, dq0);
                else if (WIDEN && p.tma_store) {
                    const uint32_t mine = own_store_base + static_cast<uint32_t>(warp - 2) * (2 * kStoreBlockBytesBf16);
                    epilogue_bf16_staged(p, &tmG, mine, blocks_sent, taddr, lane, half, m - lane, n0, dq0);
                    epilogue_bf16_staged(p, &tmG, mine, blocks_sent, taddr + kBlockN, lane, half, m - lane, n0 + kBlockN, dq0);
                } else {
                    epilogue_bf16(p, taddr, half, m, n0, dq0);
                    if constexpr (WIDEN) epilogue_bf16(p, taddr + kBlockN, half, m, n0 + kBlockN, dq0);
                }
            } else if constexpr (EPI == EPI_SWIGLU_FWD) {
                epilogue_swiglu_fwd<GU8>(p, tail, taddr, lane, half, m, n0, dq0, sgu, gu_max);
            } else {
                const bool fine = epilogue_swiglu_bwd<GU8>(p, tail, gu_base, gu_fill, tail->s_tile[acc], taddr, lane, half, row,
                                                           m, n0, dq0, sdz, inv_sgu, abort_flag, run_max);
                if (!epi_all(fine)) break;
            }
            // accumulator drained: hand it back to the MMA warp (of rank 0)
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if constexpr (PAIR) mbar_arrive_cluster(mapa_shared(smem_u32(&tail->tmem_empty[acc]), 0));
                else mbar_arrive(smem_u32(&tail->tmem_empty[acc]));
            }
            if constexpr (EPI == EPI_SWIGLU_FWD) {
                epi_bar_sync();                        // all eight warps have merged into amax_tile
                if (et < 128 && p.amax_h != nullptr) {
                    const unsigned int v = tail->amax_tile[et];
                    if ((n0 + et) < p.N && v != 0u) atomicMax(p.amax_h + n0 + et, v);
                }
                // each thread resets only its own amax_tile / s_tile entry for the next tile, and the
                // others touch them again only after the next tile's barrier: no second barrier needed
            }
        }
        if constexpr (EPI == EPI_F32 || EPI == EPI_BF16) {
            if (lane == 0) tma_store_wait_all();       // the staged output has reached global memory
        }
        if constexpr (EPI == EPI_SWIGLU_BWD) {
            run_max = warp_max_nonneg(run_max);
            if (lane == 0 && run_max > 0.0f) atomicMax(p.amax_dz, __float_as_uint(run_max));
        }
        if constexpr (EPI == EPI_SWIGLU_FWD && GU8) {
            gu_max = warp_max_nonneg(gu_max);
            if (lane == 0 && gu_max > 0.0f) atomicMax(p.amax_gu, __float_as_uint(gu_max));
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // give copies that are still in flight time to land before shared memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        __syncthreads();
    }
    // neither CTA of a pair may leave while the other can still reach its shared or tensor memory
    if constexpr (PAIR) cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        if constexpr (PAIR) tmem_dealloc_pair(tmem_base, kTmemCols); else tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres);
        if (e == cudaSuccess && qres == cudaDriverEntryPointSuccess) fn = reinterpret_cast<EncodeTiledFn>(sym);
        else set_cuda_error("cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)", e);
    });
    return fn;
}

template <int EPI, bool A_MN, bool B_MN, bool PAIR, int ELEM, bool WIDEN = false, bool GU8 = false>
int launch_inst(const CUtensorMap& tmA, const CUtensorMap& tmB0, const CUtensorMap& tmB1, const GemmArgs& args_in,
                int64_t tiles, int sm_count, cudaStream_t st) {
    constexpr size_t kSmem = smem_bytes<PAIR, EPI, WIDEN>();
    GemmArgs args = args_in;
    if (!((EPI == EPI_F32 && !WIDEN) || (EPI == EPI_BF16 && WIDEN))) args.tma_store = 0;
    args.stages = Plan<PAIR, EPI, WIDEN>::kStages - ((args.tma_store && EPI == EPI_F32) ? kStagesLentToStores : 0);
    // the saved activations [M, 2f] bf16 as two matrices of f columns: G, and U starting f elements in
    CUtensorMap tmG = tmA, tmU = tmA;
    if constexpr (EPI == EPI_SWIGLU_BWD) {
        const uint64_t f = static_cast<uint64_t>(args.N), rows = static_cast<uint64_t>(args.M);
        int rc;
        if (GU8) {                       // E4M3 codes [M, 2f]: boxes of 64 channels x 128 rows
            rc = make_tmap_ring(&tmG, args.gu8, 1, f, rows, 2 * f);
            if (rc == FP8MLP_OK) rc = make_tmap_ring(&tmU, args.gu8 + f, 1, f, rows, 2 * f);
        } else {                         // bf16 [M, 2f]: boxes of 32 channels x 128 rows
            rc = make_tmap_ring(&tmG, args.gu, 2, f, rows, 4 * f);
            if (rc == FP8MLP_OK) rc = make_tmap_ring(&tmU, args.gu + f, 2, f, rows, 4 * f);
        }
        if (rc != FP8MLP_OK) return rc;
    }
    if constexpr (EPI == EPI_BF16 && WIDEN) {
        if (args.tma_store) {
            int rc = make_tmap_out_bf16(&tmG, args.out_bf16, static_cast<uint64_t>(args.N), static_cast<uint64_t>(args.M),
                                        static_cast<uint64_t>(args.ld_out) * 2);
            if (rc != FP8MLP_OK) return rc;
        }
    }
    if constexpr (EPI == EPI_F32 && !WIDEN) {
        if (args.tma_store) {                // the two outputs of a (possibly split) fp32 result, boxes of 32 x 32
            const uint64_t rows = static_cast<uint64_t>(args.M), w0 = static_cast<uint64_t>(args.n_split < args.N ? args.n_split : args.N);
            int rc = make_tmap_out_f32(&tmG, args.out_f32_0, w0, rows, static_cast<uint64_t>(args.ld_out) * 4);
            if (rc == FP8MLP_OK && args.N > args.n_split)
                rc = make_tmap_out_f32(&tmU, args.out_f32_1, static_cast<uint64_t>(args.N - args.n_split), rows,
                                       static_cast<uint64_t>(args.ld_out) * 4);
            if (rc != FP8MLP_OK) return rc;
        }
    }
    // the function attribute and the occupancy answer belong to a device: looked up once per device
    constexpr int kMaxDevices = 64;
    static std::once_flag once_dev[kMaxDevices];
    static cudaError_t attr_err_dev[kMaxDevices] = {};
    static int max_clusters_dev[kMaxDevices] = {};
    int dev = 0;
    FP8MLP_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) { set_cuda_error_str("gemm launch", "device ordinal out of range"); return FP8MLP_ERR_CUDA; }
    std::once_flag& once = once_dev[dev];
    cudaError_t& attr_err = attr_err_dev[dev];
    int& max_clusters = max_clusters_dev[dev];
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = st;
    // set up behind the previous kernel of the stream (see launch_chained); the kernel waits for it itself
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (PAIR) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = 2;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(gemm_kernel<EPI, A_MN, B_MN, PAIR, ELEM, WIDEN, GU8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(kSmem));
        if (PAIR && attr_err == cudaSuccess) {
            // how many CTA pairs the device can hold at once (one CTA per SM, pairs on neighbouring SMs)
            cfg.gridDim = dim3(static_cast<unsigned>(sm_count) & ~1u);
            attr_err = cudaOccupancyMaxActiveClusters(&max_clusters, gemm_kernel<EPI, A_MN, B_MN, PAIR, ELEM, WIDEN, GU8>, &cfg);
        }
    });
    FP8MLP_CUDA_CHECK(attr_err);
    int64_t grid;
    if (PAIR) {
        if (max_clusters < 1) { set_cuda_error_str("gemm launch", "no CTA pair fits on the device"); return FP8MLP_ERR_CUDA; }
        grid = 2 * (tiles < max_clusters ? tiles : max_clusters);
    } else {
        grid = tiles < sm_count ? tiles : sm_count;
    }
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    FP8MLP_CUDA_CHECK(cudaLaunchKernelEx(&cfg, gemm_kernel<EPI, A_MN, B_MN, PAIR, ELEM, WIDEN, GU8>, tmA, tmB0, tmB1, tmG, tmU, args));
    count_launch();
    return FP8MLP_OK;
}

}  // namespace

size_t gemm_smem_bytes() { return smem_bytes<true, EPI_F32, false>(); }

int make_tmap(CUtensorMap* map, const void* base, int elem_bytes, bool mn_major, uint64_t inner, uint64_t outer,
              uint64_t row_stride_bytes) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return FP8MLP_ERR_CUDA;
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {row_stride_bytes};
    // 128 bytes wide; 128 rows, or for an MN-major 16-bit operand the 64 K-rows of one pipeline stage
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / elem_bytes),
                               static_cast<cuuint32_t>((mn_major && elem_bytes == 2) ? 64 : 128)};
    const cuuint32_t elem[2] = {1, 1};
    CUresult r = fn(map, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                    const_cast<void*>(base), dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_cuda_error_str("cuTensorMapEncodeTiled", "driver rejected the tensor map");
        return FP8MLP_ERR_CUDA;
    }
    return FP8MLP_OK;
}

int make_tmap_ring(CUtensorMap* map, const void* base, int elem_bytes, uint64_t inner, uint64_t outer, uint64_t row_stride_bytes) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return FP8MLP_ERR_CUDA;
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {row_stride_bytes};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(64 / elem_bytes), 128};
    const cuuint32_t elem[2] = {1, 1};
    CUresult r = fn(map, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                    const_cast<void*>(base), dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_cuda_error_str("cuTensorMapEncodeTiled", "driver rejected the tensor map of the saved activations");
        return FP8MLP_ERR_CUDA;
    }
    return FP8MLP_OK;
}

int make_tmap_out_bf16(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t row_stride_bytes) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return FP8MLP_ERR_CUDA;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_stride_bytes};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t elem[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_cuda_error_str("cuTensorMapEncodeTiled", "driver rejected the output tensor map");
        return FP8MLP_ERR_CUDA;
    }
    return FP8MLP_OK;
}

int make_tmap_out_f32(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t row_stride_bytes) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return FP8MLP_ERR_CUDA;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_stride_bytes};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t elem[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, elem,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_cuda_error_str("cuTensorMapEncodeTiled", "driver rejected the output tensor map");
        return FP8MLP_ERR_CUDA;
    }
    return FP8MLP_OK;
}

int make_tmap_u8(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t row_stride) {
    return make_tmap(map, base, 1, false, inner, outer, row_stride);
}

GemmPlan plan_gemm(int epi, GemmArgs& args, int sm_count) {
    GemmPlan plan{};
    // a CTA pair works on 256 rows at a time; a problem of at most 128 rows runs on single CTAs
    const bool pair = args.pair_mode == 1 || (args.pair_mode == 0 && args.M > kBlockM);
    const int tile_m = pair ? 2 * kBlockM : kBlockM;
    args.num_m_tiles = (args.M + tile_m - 1) / tile_m;
    // 256 x 512 tiles for the bf16-output GEMMs on CTA pairs with at least 512 output columns (GEMM-2, dgrad-1).  The
    // fp32-output weight gradients keep 256 x 256 tiles: their epilogue (four times the bytes) would sit in the open
    // and their tile counts divide worse over the CTA pairs; measured slower with wide tiles.
    const bool widen = pair && args.elem_bytes != 2 && ((epi == EPI_BF16 && args.wide_tiles != 2) || (epi == EPI_F32 && args.wide_tiles == 1)) &&
                       args.n_tile_cols == kBlockN && args.N >= 2 * kBlockN &&
                       // a small problem needs its tiles for parallelism first: wide tiles only if they still fill the CTA pairs
                       static_cast<int64_t>(args.num_m_tiles) * ((args.N + 2 * kBlockN - 1) / (2 * kBlockN)) >= sm_count / 2;
    if (widen) args.n_tile_cols = 2 * kBlockN;
    args.num_n_tiles = (args.N + args.n_tile_cols - 1) / args.n_tile_cols;
    const int elem = args.elem_bytes == 2 ? 2 : 1;
    const int kblk = kBlockK / elem;     // contraction elements per stage
    args.num_k_blocks = (args.K + kblk - 1) / kblk;
    if (args.group <= 0) {
        // Rasterisation.  A wave of tiles (one per CTA or CTA pair) streams a block of A rows and a block of B rows
        // through L2 for the whole contraction; what the next wave can still find there is the slice of one operand
        // that its tiles share with this wave's.  The plain GEMMs band along the smaller operand, the whole of it while
        // it is under 96 MiB (with every other wave walking the contraction backwards, below, the shared slice is met
        // where it is still cached; measured at the 7B shapes: 20-45 % less DRAM reading than bands of 16 row tiles,
        // 2.5 % off the step); the fused-epilogue GEMMs read less with bands of 16 row tiles.
        args.group = 16;
        args.band_n = 0;
        const int64_t a_bytes = static_cast<int64_t>(args.M) * args.K * elem, b_bytes = static_cast<int64_t>(args.N) * args.K * elem;
        // (operands that fit in L2 together are fetched from DRAM once whatever the order: those problems keep the default)
        if ((epi == EPI_F32 || epi == EPI_BF16) && a_bytes + b_bytes > (int64_t(64) << 20)) {
            constexpr int64_t kBandBytes = int64_t(96) << 20;
            args.band_n = b_bytes < a_bytes ? 1 : 0;
            const int64_t bands = ((args.band_n ? b_bytes : a_bytes) + kBandBytes - 1) / kBandBytes;
            const int along = args.band_n ? args.num_n_tiles : args.num_m_tiles;
            args.group = static_cast<int>((along + bands - 1) / bands);
        }
    }
    // fp32 outputs leave as bulk tensor stores when every box is at least as wide as the output is (32 columns)
    // (and when the contraction is so short that the kernel is bound by its output: at 16 stages' worth of work and
    // beyond, direct stores hide behind the main loop and the staging only costs shared-memory bandwidth)
    args.tma_store = (epi == EPI_F32 && !widen && args.num_k_blocks <= 8 && args.N >= 32 &&
                      (args.n_split >= args.N || (args.n_split >= 32 && args.N - args.n_split >= 32))) ? 1 : 0;
    // the bf16 output of the 256 x 512-tile kernels always does: their epilogue is not hidden behind a main loop
    if (epi == EPI_BF16 && widen) args.tma_store = 1;
    int64_t tiles = static_cast<int64_t>(args.num_m_tiles) * args.num_n_tiles;
    // A problem with fewer tiles than CTA pairs leaves SMs idle through a long contraction: split it.
    // Walking every other wave's contraction backwards pays where a wave of tiles streams more through L2 than L2 keeps
    // (about 9 x 9 tiles' operand rows times the contraction): there it saves 10-20 % of the DRAM reads at no cost in
    // time; where the operands stay cached anyway it only costs (about 2 % on the GEMMs at T = 2048).
    args.k_alternate = static_cast<int64_t>(args.K) * elem * (tile_m + (widen ? 2 * kBlockN : kBlockN)) * 9 > (int64_t(40) << 20) ? 1 : 0;
    args.split_k = 1;
    args.kb_per_split = args.num_k_blocks;
    if (tiles > 0 && args.num_k_blocks > 0 && pair && !widen && (epi == EPI_F32 || epi == EPI_BF16) && args.partial != nullptr &&
        args.tile_counters != nullptr) {
        const int64_t pairs = sm_count / 2;
        int64_t want = pairs / tiles;                                   // shares per tile that still fit one wave
        if (want > 8) want = 8;
        while (want > 1 && args.num_k_blocks / want < 8) --want;        // a share keeps at least 8 stages' worth of work
        while (want > 1 && want * static_cast<int64_t>(args.M) * args.N > args.partial_floats) --want;
        if (want > 1 && tiles * 16 <= args.counter_words) {
            args.kb_per_split = static_cast<int>((args.num_k_blocks + want - 1) / want);
            args.split_k = (args.num_k_blocks + args.kb_per_split - 1) / args.kb_per_split;   // every share non-empty
            tiles *= args.split_k;
        }
    }
    plan.pair = pair; plan.widen = widen; plan.tile_m = tile_m; plan.items = tiles;
    return plan;
}

int launch_gemm(int epi, bool a_mn, bool b_mn, int a_fmt, int b_fmt, const CUtensorMap& tmA, const CUtensorMap& tmB0,
                const CUtensorMap& tmB1, GemmArgs args, int sm_count, cudaStream_t st) {
    const GemmPlan plan = plan_gemm(epi, args, sm_count);
    const bool pair = plan.pair, widen = plan.widen;
    const int tile_m = plan.tile_m;
    const int elem = args.elem_bytes == 2 ? 2 : 1;
    const int64_t tiles = plan.items;
    // instruction descriptor: [4,6) D = fp32; [7,10) A format; [10,13) B format (0 = E4M3, 1 = E5M2);
    // bit 15 / 16: A / B is MN-major; [17,23) N >> 3; [24,29) M >> 4 (M counts both CTAs of a pair)
    args.idesc = (1u << 4) | (static_cast<uint32_t>(a_fmt) << 7) | (static_cast<uint32_t>(b_fmt) << 10) |
                 (static_cast<uint32_t>(a_mn) << 15) | (static_cast<uint32_t>(b_mn) << 16) |
                 (static_cast<uint32_t>(kBlockN >> 3) << 17) | (static_cast<uint32_t>(tile_m >> 4) << 24);
    // 32-byte stores need 32-byte aligned rows: the caller's pointers are only promised 16
    auto al32 = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 31u) == 0; };
    switch (epi) {
        case EPI_F32: args.wide = al32(args.out_f32_0) && al32(args.out_f32_1); break;
        case EPI_BF16: args.wide = al32(args.out_bf16); break;
        case EPI_SWIGLU_FWD: args.wide = al32(args.hq) && al32(args.gu8) && args.N % 32 == 0; break;
        default: args.wide = al32(args.dzq) && args.N % 32 == 0; break;
    }
    if (tiles == 0 || args.num_k_blocks == 0) return FP8MLP_OK;

#define FP8MLP_DISPATCH_WIDE(E, AM, BM)                                                                     \
    if (widen && epi == E && a_mn == AM && b_mn == BM)                                                      \
        return launch_inst<E, AM, BM, true, 1, true>(tmA, tmB0, tmB1, args, tiles, sm_count, st);
    FP8MLP_DISPATCH_WIDE(EPI_F32, false, false)
    FP8MLP_DISPATCH_WIDE(EPI_F32, false, true)
    FP8MLP_DISPATCH_WIDE(EPI_F32, true, false)
    FP8MLP_DISPATCH_WIDE(EPI_F32, true, true)
    FP8MLP_DISPATCH_WIDE(EPI_BF16, false, false)
    FP8MLP_DISPATCH_WIDE(EPI_BF16, false, true)
#undef FP8MLP_DISPATCH_WIDE
#define FP8MLP_DISPATCH(E, AM, BM, EL)                                                                     \
    if (epi == E && a_mn == AM && b_mn == BM && elem == EL)                                                \
        return pair ? launch_inst<E, AM, BM, true, EL>(tmA, tmB0, tmB1, args, tiles, sm_count, st)         \
                    : launch_inst<E, AM, BM, false, EL>(tmA, tmB0, tmB1, args, tiles, sm_count, st);
    FP8MLP_DISPATCH(EPI_F32, false, false, 1)
    FP8MLP_DISPATCH(EPI_F32, false, true, 1)
    FP8MLP_DISPATCH(EPI_F32, true, false, 1)
    FP8MLP_DISPATCH(EPI_F32, true, true, 1)
    FP8MLP_DISPATCH(EPI_BF16, false, false, 1)
    FP8MLP_DISPATCH(EPI_BF16, false, true, 1)
    if (epi == EPI_SWIGLU_FWD && args.gu8 != nullptr) {       // activations kept as E4M3 codes
        if (a_mn || !b_mn || elem != 1 || args.amax_gu == nullptr || args.s_gu == nullptr) return FP8MLP_ERR_ARG;
        return pair ? launch_inst<EPI_SWIGLU_FWD, false, true, true, 1, false, true>(tmA, tmB0, tmB1, args, tiles, sm_count, st)
                    : launch_inst<EPI_SWIGLU_FWD, false, true, false, 1, false, true>(tmA, tmB0, tmB1, args, tiles, sm_count, st);
    }
    FP8MLP_DISPATCH(EPI_SWIGLU_FWD, false, true, 1)
    if (epi == EPI_SWIGLU_BWD && args.gu8 != nullptr && (a_mn || b_mn || elem != 1)) return FP8MLP_ERR_ARG;
    if (epi == EPI_SWIGLU_BWD && args.gu8 != nullptr)      // saved activations as E4M3 codes
        return pair ? launch_inst<EPI_SWIGLU_BWD, false, false, true, 1, false, true>(tmA, tmB0, tmB1, args, tiles, sm_count, st)
                    : launch_inst<EPI_SWIGLU_BWD, false, false, false, 1, false, true>(tmA, tmB0, tmB1, args, tiles, sm_count, st);
    FP8MLP_DISPATCH(EPI_SWIGLU_BWD, false, false, 1)
    // the bf16 last layer of the "SwiGLU output in BF16" variant
    FP8MLP_DISPATCH(EPI_BF16, false, true, 2)
    FP8MLP_DISPATCH(EPI_SWIGLU_BWD, false, false, 2)
    FP8MLP_DISPATCH(EPI_F32, true, true, 2)
    FP8MLP_DISPATCH(EPI_F32, false, false, 2)      // the remaining layouts, for fp8mlp_gemm_bf16
    FP8MLP_DISPATCH(EPI_F32, false, true, 2)
    FP8MLP_DISPATCH(EPI_F32, true, false, 2)
#undef FP8MLP_DISPATCH
    return FP8MLP_ERR_ARG;
}

}  // namespace fp8mlp

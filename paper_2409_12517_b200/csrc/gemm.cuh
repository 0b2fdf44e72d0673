// FP8 (and, for one variant, bf16) GEMM for sm_100a: persistent, warp-specialised, tcgen05.mma
// kind::f8f6f4 / kind::f16 with fp32 accumulators in tensor memory, operands streamed by TMA through
// a multi-stage shared-memory ring, and the block's element-wise steps fused into the epilogue that
// drains tensor memory.
//
//   D[m, n] = sum_k A(m, k) * B(n, k)
//
// Either operand may be stored with K contiguous ("K-major", [rows, K]) or with its M/N index
// contiguous ("MN-major", [K, rows]); both are fetched as 128-byte-wide TMA boxes with the 128-byte
// swizzle and only the shared-memory matrix descriptors differ.  That lets the forward, dgrad and
// wgrad GEMMs of the block all read the same buffers without transposed copies.
//
// Whenever M > 128 two CTAs on neighbouring SMs (a cluster of two) share one 256 x 256 tile through
// tcgen05 cta_group::2: each loads half of A's and half of B's rows (no multicast), the CTA of rank 0
// issues the MMAs for both, each drains its own 128 rows of the accumulator.  Otherwise one CTA works
// on a 128 x 256 tile.
//
// CTA = 11 warps: warp 0 issues TMA loads, warp 1 owns tensor memory and issues the MMAs,
// warps 2-9 are the epilogue (a TMEM lane quadrant and one half of the columns each), warp 10
// streams the saved G, U to the backward SwiGLU epilogue (idle elsewhere).  Two 256-column
// accumulators alternate, so the epilogue of one tile overlaps the main loop of the next.
// Every wait is bounded: on expiry the CTA raises a status word and drains.
#pragma once

#include "common.cuh"

namespace fp8mlp {

enum : int { EPI_F32 = 0, EPI_BF16 = 1, EPI_SWIGLU_FWD = 2, EPI_SWIGLU_BWD = 3 };

constexpr int kBlockM = 128;          // rows of D per tile (TMEM lanes)
constexpr int kBlockN = 256;          // accumulator columns per tile
constexpr int kBlockK = 128;          // contraction bytes per pipeline stage (128 FP8 or 64 bf16 elements)
constexpr int kUmmaK = 32;            // contraction bytes per tcgen05.mma
constexpr int kBoxBytes = 128 * 128;  // one TMA box: 128 bytes x 128 rows
constexpr int kGemmThreads = 352;       // TMA warp, MMA warp, 8 epilogue warps, loader warp of the saved activations
constexpr int kTmemCols = 512;
constexpr int kEpiThreads = 256;

struct GemmArgs {
    int M, N, K;            // N: extent of the n coordinate space (output columns; d_ff channels for the SwiGLU epilogues)
    int num_m_tiles, num_n_tiles, num_k_blocks;
    int n_tile_cols;        // n coordinates per tile: 256, or 128 when the two B boxes are gate and linear halves
    int b1_offset;          // n offset of the second B box: 128, or 0 in the gate/linear case
    int group;              // tiles per rasterisation band, counted along m (band_n = 0) or along n (band_n = 1); 0: chosen by the launcher
    int band_n;
    int hint_a, hint_b;     // L2 eviction priority of the A / B operand loads (L2_HINT_*)
    int pair_mode;          // 0: CTA pairs when M > 128; 1: always CTA pairs; 2: always single CTAs
    int elem_bytes;         // operand element size: 1 (FP8, default) or 2 (bf16; a_fmt = b_fmt = 1)
    int wide_tiles;         // 256 x 512 tiles: 0 = for bf16 outputs (default), 1 = for fp32 outputs too, 2 = never
    uint32_t idesc;
    int* status;
    // Split of the contraction over several CTA pairs (problems with fewer tiles than the GPU has CTA pairs;
    // plain epilogues only).  Every split writes its fp32 partial tile to `partial` ([split_k][M][N]) and counts
    // itself in tile_counters (16 words per tile: one per epilogue warp of the pair); the warp that arrives last
    // for its 32 x 128 region adds the partials in split order and writes the output.  split_k = 1: off.
    int split_k;
    int kb_per_split;
    float* partial;                 // workspace, nullable (then no split is made)
    int64_t partial_floats;         // its capacity
    unsigned int* tile_counters;    // zero before the launch; left zero by it
    int counter_words;

    // dequantisation: dq = (1 / *s0) * (1 / *s1); a null pointer stands for 1
    const float* s0;
    const float* s1;
    // EPI_F32: out = acc * dq; with row_s, dq = (1 / *s0) * (1 / row_s[m]).  Columns < n_split go to
    // out_f32_0[m*ld_out + n], the others to out_f32_1[m*ld_out + n - n_split].
    const float* row_s;
    float* out_f32_0;
    float* out_f32_1;
    int n_split;
    int64_t ld_out;
    int k_alternate;        // set by the launcher: every other wave of tiles walks the contraction backwards (L2 reuse)
    int tma_store;          // set by the launcher: the fp32 output leaves through shared memory and bulk tensor stores
    int stages;             // set by the launcher: operand stages in use (all of the kernel's, or two fewer when their
                            // shared memory stages the output)
    // EPI_BF16: out_bf16[m*ld_out + n] = bf16(acc * dq)
    uint16_t* out_bf16;
    // SwiGLU epilogues (f = N)
    const float* s_h;       // [f] per-channel scale of H
    int smooth;             // backward: multiply dH by s_h (Smooth-SwiGLU) or not (per-tensor scale)
    int store;              // 0: calibration pass, only the maxima are produced
    int wide;               // outputs may be written 32 bytes at a time (rows and bases 32-byte aligned)
    uint8_t* hq;            // fwd: E4M3 [M, f]
    uint16_t* hb;           // fwd: if not null, bf16 [M, f] = H unscaled, stored instead of hq (32-byte aligned rows)
    uint16_t* gu;           // fwd: out (nullable), bwd: in; bf16 [M, 2f] = G | U
    uint8_t* gu8;           // if not null: E4M3 [M, 2f] = Q(s_gu [G | U]) kept instead of the bf16 pair (fwd: out, bwd: in)
    const float* s_gu;      // scale of gu8
    unsigned int* amax_gu;  // fwd: bit pattern of max(|G|, |U|), raised atomically; null: not wanted
    unsigned int* amax_h;   // fwd: [f] bit patterns of max |H|, raised atomically; null: maxima not wanted
    const float* sdz;       // bwd: scale of dZ
    uint8_t* dzq;           // bwd: E5M2 [M, 2f] = dG | dU
    unsigned int* amax_dz;  // bwd: bit pattern of max(|dG|, |dU|), raised atomically
};

size_t gemm_smem_bytes();

// Encodes the 2-D tiled tensor map of an 8-bit matrix whose rows are `inner` bytes long and
// `row_stride` bytes apart: box = 128 bytes x 128 rows, 128-byte swizzle, zero fill out of bounds.
int make_tmap_u8(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t row_stride);
// General form: elem_bytes 1 (FP8) or 2 (bf16); inner / outer in elements, row stride in bytes; mn_major says how
// the GEMM will read the matrix (an MN-major 16-bit operand is fetched in boxes of 64 K-rows).
int make_tmap(CUtensorMap* map, const void* base, int elem_bytes, bool mn_major, uint64_t inner, uint64_t outer,
              uint64_t row_stride_bytes);

// Tensor map of the saved activations for the backward epilogue's ring: boxes of 64 bytes x 128 rows, 64-byte swizzle.
int make_tmap_ring(CUtensorMap* map, const void* base, int elem_bytes, uint64_t inner, uint64_t outer, uint64_t row_stride_bytes);
// Tensor map of an fp32 output matrix for bulk stores: boxes of 32 columns x 32 rows, 128-byte swizzle.
int make_tmap_out_f32(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t row_stride_bytes);
// The same for a bf16 output matrix: boxes of 32 columns x 32 rows, 64-byte swizzle.
int make_tmap_out_bf16(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t row_stride_bytes);

// How a GEMM will be run: fills in the tiling, rasterisation, split and output-path fields of `args` (all host
// arithmetic, nothing is launched) and returns the rest.  launch_gemm starts with this.
struct GemmPlan { bool pair, widen; int tile_m; int64_t items; };
GemmPlan plan_gemm(int epi, GemmArgs& args, int sm_count);

// Launches one GEMM.  a_mn / b_mn: the operand is MN-major.  The tensor maps describe A, and the
// two 128-wide halves of the B tile (the same map twice unless they come from different matrices).
// EPI_SWIGLU_BWD reads args.gu through TMA: the launcher builds those two tensor maps itself.
int launch_gemm(int epi, bool a_mn, bool b_mn, int a_fmt, int b_fmt, const CUtensorMap& tmA,
                const CUtensorMap& tmB0, const CUtensorMap& tmB1, GemmArgs args, int sm_count, cudaStream_t st);

}  // namespace fp8mlp

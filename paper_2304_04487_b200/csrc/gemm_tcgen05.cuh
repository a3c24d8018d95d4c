// Weight-streaming GEMM for the decoder's projections (library-private interface).
//
//   out[r, n] = sum_k W[n, k] * a[r, k],  r < 32 activation rows, W bf16 [n_out, k_in].
//
// The activations arrive split into two bf16 halves (ActLayout kActSplit: 64 rows, hi then lo);
// the MMA's N dimension is those 64 rows and the epilogue adds the hi and lo columns, so the
// product keeps 16 mantissa bits of the activations at no cost in weight traffic.
//
// The weight matrix is the MMA's M operand (128 output features per tile) and the
// activation rows are its N operand, so every weight byte crosses HBM exactly once per
// step however many rows are verified.  Work is the flat list of (tile, 64-wide k-chunk)
// pairs, cut into equal contiguous ranges, one per CTA; partial tiles are summed in a fixed
// order that depends on the matrix shape and grid only -- never on the rows in use.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace llma {

enum GemmMode : int32_t {
    kGemmQKV = 0,     // A maps = {wq, wk, wv}; rotary embedding; q -> qkv buffer, k/v -> cache
    kGemmResid = 1,   // x[r, n] += acc
    kGemmSwiGLU = 2,  // A maps = {w_gate, w_up}, 64 + 64 rows per tile; h = silu(g) * u (bf16)
    kGemmLmHead = 3,  // per-tile (max, argmax) per row; optional logits store
    kGemmStore = 4,   // out[r, n] = acc for all 32 rows (stand-alone product)
};

struct GemmArgs {
    int32_t mode;
    int32_t n_out;          // output features (per matrix for QKV; d_ffn for SwiGLU)
    int32_t n_tiles;        // tiles over all matrices
    int32_t chunks;         // k_in / 64
    int32_t tiles_per_map;  // tiles per A map
    const RowDesc* rows;    // nullptr: all 32 rows are in use
    const void* act;        // activation operand, ActLayout kActSplit [2 * kMaxRows][k_in] bf16
    float* ws;              // partial tiles [grid][2][128][32] fp32; slot 1 of every CTA all-ones (empty) at launch
    int32_t* cnt;           // unused by the kernel (kept for the layout of callers' scratch)
    int32_t* dev_err;
    float* out_f32;         // Resid: x; QKV: qkv buffer; LmHead: logits or nullptr
    int32_t ld;             // leading dimension of out_f32
    void* out_act;          // SwiGLU: h in ActLayout kActSplit [64][d_ffn]
    // RMSNorm folded into the projections: the producer of the residual stream x writes
    // xs = split(x * gain) and, per 128-column tile, the rows' sums of squares; the consumer
    // multiplies its accumulators by rsqrt(sum / norm_dim + eps), which equals projecting the
    // normalised row because the scale is one number per row.
    const float* ss_in;     // consumer: [ss_tiles][32] partial sums of squares, or nullptr
    int32_t ss_tiles;
    int32_t norm_dim;
    float norm_eps;
    const float* gain_next; // Resid producer: gain of the next norm [n_out], with xs_out / ss_out
    void* xs_out;           // ActLayout kActSplit [64][n_out], or nullptr
    float* ss_out;          // [n_tiles][32]
    // QKV
    ModelDims dims;
    int32_t layer;
    const float *rope_cos, *rope_sin;
    __nv_bfloat16 *kcache, *vcache;
    // LmHead
    float* part_max;        // [n_tiles][32]
    int32_t* part_idx;
};

constexpr int kGemmN = 2 * kMaxRows;  // rows of a split activation buffer: hi rows then lo rows
constexpr int kGemmThreads = 320;  // 4 epilogue warps, TMA producer, MMA issuer, 4 activation-loader warps
constexpr uint32_t kGemmABytes = 128 * 64 * 2;

// The kernel exists for NR = 16 or 32 activation rows per half (MMA N = 2 NR).  Ring depths are the
// ones measured fastest inside a decoding step (8 stages at NR 16, 6 at NR 32; deeper rings only
// lengthen the queues that the epilogue's traffic also waits in).  The activation tile of a stage
// is NOT fetched by TMA: a second, small TMA copy per stage slowed the weight stream by a
// quarter wherever it came from (shared buffer, per-CTA replica, one hot 4 KB block), whereas
// plain loads by otherwise idle warps cost almost nothing.  Four loader warps take turns copying
// the rows from global memory into the 128-byte-swizzled layout the MMA expects.
// The request is padded to more than half an SM's shared memory so that the CTAs of two
// consecutive projections never share an SM (measured 10 % slower when they do).
template <int NR> struct GemmCfg {
    static constexpr uint32_t kBBytes = 2 * NR * 64 * 2;
    static constexpr int kStages = NR == 16 ? 8 : 6;
    static constexpr size_t kRopeBytes = kMaxRows * 64 * 8;  // (cos, sin) of every row's position, 64 rotary pairs
    static constexpr size_t kUsedBytes = 1024 + (size_t)kStages * (kGemmABytes + kBBytes) + 128 * 33 * 4 + 1536 + kRopeBytes;
    static constexpr size_t kSmemBytes = kUsedBytes > 120 * 1024 ? kUsedBytes : 120 * 1024;
};

// grid size used for a problem with `work` = n_tiles * chunks (a function of the shape only)
int gemm_grid_for(int64_t work, int num_sms);

// Encode a 2-D bf16 row-major [rows, cols] tensor for TMA with a {64, box_rows} box and
// 128-byte swizzle.  Returns a CUresult (0 = success).
int make_tensor_map_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);

// Opt the kernel into its dynamic shared-memory size (once per process, outside any capture).
cudaError_t init_gemm_tcgen05();

// nr = 16 or 32 activation rows per half; pdl = launch with programmatic stream serialization (the
// kernel before it must be one of this library's)
void launch_gemm_tcgen05(cudaStream_t st, int grid, int nr, bool pdl, const GemmArgs& args, const CUtensorMap& a0,
                         const CUtensorMap& a1, const CUtensorMap& a2);

// out_tok[r] = index of the largest logit over all tiles (lowest index on ties)
void launch_argmax_final(cudaStream_t st, bool pdl, const RowDesc* rows, const float* part_max, const int32_t* part_idx,
                         int32_t n_tiles, int32_t* out_tok);

}  // namespace llma

// Weight-streaming GEMM for the decoder's projections (library-private interface).
//
//   out[r, n] = sum_k W[n, k] * a[r, k],  r < rows (up to 256 activation rows), W bf16 [n_out, k_in].
//
// The activations arrive split into two bf16 terms (ActLayout kActSplit: hi rows, then lo rows); both
// are multiplied by the same weight tile and summed in fp32, so the product keeps 16 mantissa bits
// of the activations at no cost in weight traffic.
//
// The weight matrix is the MMA's M operand (128 output features per tile) and the
// activation rows are its N operand, so every weight byte crosses HBM exactly once per
// step however many rows are verified.  Work is the flat list of (tile, 64-wide k-chunk)
// pairs, cut into equal contiguous ranges, one per CTA; partial tiles are summed in a fixed
// order that depends on the matrix shape and grid only -- never on the rows in use.
//
// Two kernels share the fused epilogues: gemm_ws_kernel<NR> for engines of at most 32 rows (NR = 16
// or 32 fixed per engine; activation tiles copied by loader warps) and gemm_wide_kernel for up to
// 256 rows (activation tiles by TMA, MMA N = the rows in use rounded up to 16, epilogue in blocks of
// 32 rows).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace llma {

enum GemmMode : int32_t {
    kGemmQKV = 0,     // A maps = {wq, wk, wv}; rotary embedding; q -> qkv buffer, k/v -> cache
    kGemmResid = 1,   // x[r, n] += acc
    kGemmSwiGLU = 2,  // A maps = {w_gate, w_up}, 64 + 64 rows per tile; h = silu(g) * u (split bf16)
    kGemmLmHead = 3,  // per-tile (max, argmax) per row; optional logits store
    kGemmStore = 4,   // out[r, n] = acc for all rows (stand-alone product)
};

struct GemmArgs {
    int32_t mode;
    int32_t n_out;          // output features (per matrix for QKV; d_ffn for SwiGLU)
    int32_t n_tiles;        // tiles over all matrices
    int32_t chunks;         // k_in / 64
    int32_t tiles_per_map;  // tiles per A map
    const RowDesc* rows;    // nullptr: all nr rows are in use
    const void* act;        // activation operand, ActLayout kActSplit [2 rc][k_in] bf16
    int32_t rc;             // row capacity of the activation buffers and per-row scratch arrays
    int32_t nr;             // rows the launch is shaped for (wide kernel: multiple of 16, <= 256)
    unsigned long long* stamps;  // measurement builds: timeline block (see LLMA_STAMPS), else unused
    int32_t launch_id;           // ... which launch of the step this is
    float* ws;              // partial tiles [grid][2][nr / 4][128] float4; slot 1 of every CTA all-ones (empty) at launch
    int32_t* dev_err;
    float* out_f32;         // Resid: x; QKV: qkv buffer; LmHead: logits or nullptr
    int32_t ld;             // leading dimension of out_f32
    void* out_act;          // SwiGLU: h in ActLayout kActSplit [2 rc][d_ffn]
    int32_t gate_second;    // SwiGLU: 1 when the tile's rows 0..63 are the up features and 64..127 the gate features
    // RMSNorm folded into the projections: the producer of the residual stream x writes
    // xs = split(x * gain) and, per 128-column tile, the rows' sums of squares; the consumer
    // multiplies its accumulators by rsqrt(sum / norm_dim + eps), which equals projecting the
    // normalised row because the scale is one number per row.
    const float* ss_in;     // consumer: [ss_tiles][rc] partial sums of squares, or nullptr
    int32_t ss_tiles;
    int32_t norm_dim;
    float norm_eps;
    const float* gain_next; // Resid producer: gain of the next norm [n_out], with xs_out / ss_out
    void* xs_out;           // ActLayout kActSplit [2 rc][n_out], or nullptr
    float* ss_out;          // [n_tiles][rc]
    // QKV
    ModelDims dims;
    int32_t layer;
    const float *rope_cos, *rope_sin;
    __nv_bfloat16 *kcache, *vcache;
    // LmHead
    float* part_max;        // [n_tiles][rc]
    int32_t* part_idx;
};

constexpr int kGemmThreads = 320;  // 4 epilogue warps, TMA producer, MMA issuer, 4 activation-loader warps
constexpr int kGemmWideThreads = 224;  // 4 epilogue warps, weight producer, MMA issuer, activation producer
constexpr uint32_t kGemmABytes = 128 * 64 * 2;  // one weight tile: 128 rows x one 64-wide k-chunk

// gemm_ws_kernel exists for NR = 16 or 32 activation rows (MMA N = 2 NR: hi and lo columns).
// A ring stage holds KC consecutive k-chunks of one weight tile, fetched by ONE TMA copy through a
// 3-D view of the matrix (64 columns, rows, chunk): with KC = 2 a copy moves 32 KB and reads 256
// contiguous bytes of every weight row, which streams at 5.85 TB/s where 16 KB copies (128 bytes per
// row) reach 4.86 TB/s (copy-only kernel, 148 CTAs, measured).  The gate/up projection, whose tile is
// 64 + 64 rows of two matrices, does the same through a 4-D view that spans both matrices (64 columns,
// rows, matrix, chunk): one copy lands, for each of the two chunks, the 64 gate rows followed by the 64 up rows.
// Ring depths are the ones measured fastest inside a decoding step (deeper rings only
// lengthen the queues that the epilogue's traffic also waits in).  The activation tile of a stage
// is NOT fetched by TMA here: a second, small TMA copy per stage slowed the weight stream by a
// quarter wherever it came from (shared buffer, per-CTA replica, one hot 4 KB block), whereas
// plain loads by otherwise idle warps cost almost nothing.  Four loader warps take turns copying
// the rows from global memory into the 128-byte-swizzled layout the MMA expects.
// The request is padded to more than half an SM's shared memory so that the CTAs of two
// consecutive projections never share an SM (measured 10 % slower when they do).
constexpr int kGemmKC = 2;  // 64-wide k-chunks per ring stage
template <int NR> struct GemmCfg {
    static constexpr uint32_t kABytes = kGemmKC * kGemmABytes;
    static constexpr uint32_t kBTile = 2 * NR * 64 * 2;   // activation rows (hi, lo) of one k-chunk
    static constexpr uint32_t kBBytes = kGemmKC * kBTile;
    static constexpr int kStages = 4;  // at 32 rows this fills the 227 KB of shared memory to the byte
    static constexpr size_t kRopeBytes = 32 * 64 * 8;  // (cos, sin) of every row's position, 64 rotary pairs
    static constexpr size_t kUsedBytes = 1024 + (size_t)kStages * (kABytes + kBBytes) + 128 * 33 * 4 + 1536 + kRopeBytes;
    static constexpr size_t kSmemBytes = kUsedBytes > 120 * 1024 ? kUsedBytes : 120 * 1024;
};

// Shared-memory plan of gemm_wide_kernel for nr rows: a ring of weight tiles (16 KB each) and a ring of
// activation tiles (nr rows of 128 bytes each: one term of one 64-wide k-chunk), as many as fit.
struct GemmWideCfg {
    uint32_t b_slot;    // bytes of one activation tile: nr rows of 128 bytes for each of the two terms
    int sa, sb;         // ring depths (each at most 8)
    uint32_t tmem_cols; // power of two >= the accumulators' columns (2 nr each; two of them up to 128 rows, else one)
    size_t smem_bytes;
};
GemmWideCfg gemm_wide_cfg(int nr);

// grid size used for a problem with `work` = n_tiles * chunks (a function of the shape only)
int gemm_grid_for(int64_t work, int num_sms);

// Encode a 2-D bf16 row-major [rows, cols] tensor for TMA with a {64, box_rows} box and
// 128-byte swizzle.  Returns a CUresult (0 = success).
int make_tensor_map_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// A split activation buffer [2 rc, cols] (hi rows, then lo rows) seen as (cols, rc rows, 2 terms) with a
// {64, box_rows, 2} box: one copy lands the hi rows of a 64-wide k-chunk followed by its lo rows.
int make_tensor_map_bf16_terms(CUtensorMap* out, const void* base, uint64_t rc, uint64_t cols, uint32_t box_rows);
// The same tensor seen as (64 columns, rows, cols / 64 chunks) with a {64, box_rows, 2} box: two
// consecutive k-chunks of box_rows rows per copy, landing as two tiles of the 2-D layout one after the other.
int make_tensor_map_bf16_chunks(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// Two matrices [rows, cols] of equal shape seen as (64 columns, rows, matrix, chunk) with a {64, 64, 2, 2} box: one
// copy lands [chunk][matrix][64 rows].  The matrix at the lower address comes first: *swapped = 1 if that is
// base1.  Fails (non-zero) when the two allocations are more than 2^40 bytes apart.
int make_tensor_map_bf16_pair(CUtensorMap* out, const void* base0, const void* base1, uint64_t rows, uint64_t cols,
                              int* swapped);

// Opt the kernel into its dynamic shared-memory size (once per process, outside any capture).
cudaError_t init_gemm_tcgen05();

// args.nr = 16 or 32 rows; a0..a2 are chunk-pair maps (make_tensor_map_bf16_chunks, 128-row boxes); in
// kGemmSwiGLU mode a0 is the map over both matrices (make_tensor_map_bf16_pair); pdl = launch with programmatic stream serialization
// (the kernel before it must be one of this library's)
void launch_gemm_tcgen05(cudaStream_t st, int grid, bool pdl, const GemmArgs& args, const CUtensorMap& a0,
                         const CUtensorMap& a1, const CUtensorMap& a2);

// args.nr = 32 .. 256 (multiple of 16); map_b[i] (make_tensor_map_bf16_terms) covers the split activation buffer
// with a box of wide_box_rows(nr, i) rows, i = 0 .. 3
cudaError_t init_gemm_wide();
void launch_gemm_wide(cudaStream_t st, int grid, bool pdl, const GemmArgs& args, const CUtensorMap& a0,
                      const CUtensorMap& a1, const CUtensorMap& a2, const CUtensorMap* map_b);
// Activation rows per copy of gemm_wide_kernel, candidate i of four: 32, 64, 128 (none above nr), then nr itself.
// A step takes the first candidate that holds its rows, so the activation traffic follows the rows in use, and
// up to 128 rows the hi and lo rows sit close enough for one MMA over both.
__host__ __device__ inline int wide_box_rows(int nr, int i) {
    const int c = i == 0 ? 32 : (i == 1 ? 64 : (i == 2 ? 128 : nr));
    return c < nr ? c : nr;
}

}  // namespace llma

// Epilogues of the weight-streaming GEMM: what happens to a finished 128 x 32 fp32 tile.
// Called by the 128 epilogue threads; thread `row` holds acc[0..31] = the 32 activation
// rows' results for output feature (tile, row).  `stage` is a [128][33] fp32 shared buffer.
#pragma once
#include "gemm_tcgen05.cuh"
#include "ptx_sm100.cuh"

namespace llma {

constexpr uint32_t kEpiBar = 1;  // named barrier of the 128 epilogue threads

__device__ __forceinline__ void epi_sync() { ptx::named_bar_sync(kEpiBar, 128); }

// x[r, n] += acc  (output projection and FFN down projection, residual stream in fp32).
// When the next RMSNorm is folded in (g.xs_out): also xs = split(x * gain) and this tile's
// per-row sums of squares, reduced over the 128 columns in a fixed shuffle/warp order.
__device__ __forceinline__ void epilogue_resid(const GemmArgs& g, int tile, int row, const float (&acc)[32],
                                               int rows_used, float (*stage)[33]) {
    const int col = tile * 128 + row;
    const bool valid = col < g.n_out;
    float xn[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        xn[j] = 0.f;
        if (j < rows_used && valid) {
            xn[j] = g.out_f32[(int64_t)j * g.ld + col] + acc[j];
            g.out_f32[(int64_t)j * g.ld + col] = xn[j];
        }
    }
    if (!g.xs_out) return;
    const float gain = valid ? g.gain_next[col] : 0.f;
    const int warp = row >> 5, lane = row & 31;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (j < rows_used) {
            if (valid) store_act(g.xs_out, kActSplit, j, col, g.n_out, xn[j] * gain);
            float sq = xn[j] * xn[j];
            for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
            if (lane == 0) stage[warp][j] = sq;
        }
    }
    epi_sync();
    if (row < rows_used) g.ss_out[(int64_t)tile * 32 + row] = ((stage[0][row] + stage[1][row]) + stage[2][row]) + stage[3][row];
    epi_sync();
}

// out[r, n] = acc
__device__ __forceinline__ void epilogue_store(const GemmArgs& g, int tile, int row, const float (&acc)[32],
                                               int rows_used) {
    const int col = tile * 128 + row;
    if (col >= g.n_out) return;
#pragma unroll
    for (int j = 0; j < 32; ++j)
        if (j < rows_used) g.out_f32[(int64_t)j * g.ld + col] = acc[j];
}

// QKV: rotary embedding on q and k (pair (i, i + hd/2)), q to the fp32 qkv buffer, k and v
// rows into the bf16 cache at (sequence, position) of every used row.
__device__ __forceinline__ void epilogue_qkv(const GemmArgs& g, int tile, int row, const float (&acc)[32],
                                             int rows_used, float (*stage)[33]) {
#pragma unroll
    for (int j = 0; j < 32; ++j) stage[row][j] = acc[j];
    epi_sync();
    const ModelDims& d = g.dims;
    const int mat = tile / g.tiles_per_map;
    const int col = (tile % g.tiles_per_map) * 128 + row;
    const int hd = d.head_dim, half = hd >> 1;
    const int head = col / hd, idx = col % hd;
    const bool lower = idx < half;
    const int prow = lower ? row + half : row - half;
    if (col < g.n_out) {
        for (int j = 0; j < rows_used; ++j) {
            const int pos = g.rows->pos[j];
            if (pos < 0) continue;
            float val = stage[row][j];
            if (mat < 2) {
                const float other = stage[prow][j];
                const float c = g.rope_cos[(int64_t)pos * half + (idx % half)];
                const float s = g.rope_sin[(int64_t)pos * half + (idx % half)];
                val = lower ? (val * c - other * s) : (other * s + val * c);
            }
            if (mat == 0) {
                g.out_f32[(int64_t)j * g.ld + col] = val;
            } else {
                __nv_bfloat16* cache = mat == 1 ? g.kcache : g.vcache;
                cache[kv_row_index(d, g.layer, g.rows->seq[j], head, pos) * hd + idx] = __float2bfloat16_rn(val);
            }
        }
    }
    epi_sync();
}

// SwiGLU: tile rows 0..63 are gate features, 64..127 the matching up features.
__device__ __forceinline__ void epilogue_swiglu(const GemmArgs& g, int tile, int row, const float (&acc)[32],
                                                int rows_used, float (*stage)[33]) {
#pragma unroll
    for (int j = 0; j < 32; ++j) stage[row][j] = acc[j];
    epi_sync();
    const int fi = row & 63, f = tile * 64 + fi;
    if (f < g.n_out) {
        for (int j = row >> 6; j < rows_used; j += 2) {
            const float gate = stage[fi][j], up = stage[64 + fi][j];
            store_act(g.out_act, kActSplit, j, f, g.n_out, gate / (1.f + expf(-gate)) * up);
        }
    }
    epi_sync();
}

// LM head: optional logits store, then the tile's (max, lowest argmax) for every used row.
__device__ __forceinline__ void epilogue_lmhead(const GemmArgs& g, int tile, int row, const float (&acc)[32],
                                                int rows_used, float (*stage)[33]) {
    const int v = tile * 128 + row;
    const bool valid = v < g.n_out;
    if (g.out_f32 && valid) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
            if (j < rows_used) g.out_f32[(int64_t)j * g.ld + v] = acc[j];
    }
    const int warp = row >> 5, lane = row & 31;
    float* red_v = &stage[0][0];                       // [4][32] values
    int* red_i = reinterpret_cast<int*>(&stage[8][0]);  // [4][32] indices
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (j < rows_used) {
            float bv = valid ? acc[j] : -INFINITY;
            int bi = valid ? v : 0x7fffffff;
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            if (lane == 0) { red_v[warp * 32 + j] = bv; red_i[warp * 32 + j] = bi; }
        }
    }
    epi_sync();
    if (row < rows_used) {
        float bv = red_v[row]; int bi = red_i[row];
        for (int w = 1; w < 4; ++w) {
            const float ov = red_v[w * 32 + row]; const int oi = red_i[w * 32 + row];
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        g.part_max[(int64_t)tile * 32 + row] = bv;
        g.part_idx[(int64_t)tile * 32 + row] = bi;
    }
    epi_sync();
}

}  // namespace llma

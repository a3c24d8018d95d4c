// Epilogues of the weight-streaming GEMM: what happens to a finished 128 x 32 fp32 block.
// Called by the 128 epilogue threads after the block has been staged in shared memory:
// stage[f][j] is the result for output feature f of the tile (thread `row` staged its own
// feature) and activation row jb + j, j < nj <= 32.  Engines of at most 32 rows have one
// block per tile (jb = 0); the wide kernel walks a tile in blocks of 32 rows.
// red_f / red_i are [4][32] scratch for per-warp reductions.
//
// The loops over activation rows are deliberately NOT unrolled over all 32 rows: this code
// runs once per tile, so its cost is dominated by instruction fetch, and compact loops
// with a few independent loads in flight beat long straight-line code.
#pragma once
#include "gemm_tcgen05.cuh"
#include "ptx_sm100.cuh"

namespace llma {

constexpr int kXPre = 13;  // residual epilogue: x rows 0..11 of the column, then the next norm's gain, requested early

constexpr uint32_t kEpiBar = 1;  // named barrier of the 128 epilogue threads

__device__ __forceinline__ void epi_sync() { ptx::named_bar_sync(kEpiBar, 128); }

__device__ __forceinline__ float warp_sum(float v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// x[r, n] += acc  (output projection and FFN down projection, residual stream in fp32).
// When the next RMSNorm is folded in (g.xs_out): also xs = split(x * gain) and this tile's
// per-row sums of squares, reduced over the 128 columns in an order fixed by the column index.
// With kHavePre (jb = 0 only), xpre holds x[0..11, col] and the gain, read earlier by the caller.
template <bool kHavePre>
__device__ __forceinline__ void epilogue_resid(const GemmArgs& g, int tile, int row, int jb, int nj,
                                               float (*stage)[33], float* red_f, const float (&xpre)[kXPre]) {
    const int col = tile * 128 + row;
    const bool valid = col < g.n_out;
    const bool fold = g.xs_out != nullptr;
    const float gain = kHavePre ? xpre[kXPre - 1] : ((fold && valid) ? __ldg(&g.gain_next[col]) : 0.f);
    const unsigned group = 0xffu << (row & 24);  // the eight lanes that share an activation row below
    // x is added into the staged tile with a few loads in flight; the per-row work is a rolled loop
    if (kHavePre) {
#pragma unroll
        for (int u = 0; u < kXPre - 1; ++u)
            if (u < nj) stage[row][u] += xpre[u];
    }
    for (int j0 = kHavePre ? kXPre - 1 : 0; j0 < nj; j0 += 8) {
        float xv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
            xv[u] = (valid && j0 + u < nj) ? __ldcg(&g.out_f32[(int64_t)(jb + j0 + u) * g.ld + col]) : 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (j0 + u < nj) stage[row][j0 + u] += xv[u];
    }
    if (!valid) {
        for (int j = 0; j < nj; ++j) stage[row][j] = 0.f;  // columns past the matrix add nothing to the sums of squares
    } else {
#pragma unroll 1
        for (int j = 0; j < nj; ++j) {
            const float xn = stage[row][j];
            g.out_f32[(int64_t)(jb + j) * g.ld + col] = xn;
            if (fold) store_act(g.xs_out, kActSplit, g.rc, jb + j, col, g.n_out, xn * gain);
        }
    }
    if (!fold) return;
    // Sums of squares: eight threads per activation row, each over sixteen consecutive features in
    // ascending order, then a three-step shuffle tree: the order depends on the feature index only.
    epi_sync();
    for (int j = row >> 3; j < nj; j += 16) {  // nj is uniform over the eight threads of a row
        const int f0 = (row & 7) * 16;
        float sq = 0.f;
#pragma unroll
        for (int u = 0; u < 16; ++u) { const float v = stage[f0 + u][j]; sq = __fmaf_rn(v, v, sq); }
        sq += __shfl_xor_sync(group, sq, 1);
        sq += __shfl_xor_sync(group, sq, 2);
        sq += __shfl_xor_sync(group, sq, 4);
        if ((row & 7) == 0) g.ss_out[(int64_t)tile * g.rc + jb + j] = sq;
    }
    epi_sync();
}

// out[r, n] = acc
__device__ __forceinline__ void epilogue_store(const GemmArgs& g, int tile, int row, int jb, int nj,
                                               float (*stage)[33]) {
    const int col = tile * 128 + row;
    if (col >= g.n_out) return;
#pragma unroll 1
    for (int j = 0; j < nj; ++j) g.out_f32[(int64_t)(jb + j) * g.ld + col] = stage[row][j];
}

// QKV: rotary embedding on q and k (pair (i, i + hd/2)), q to the fp32 qkv buffer, k and v
// rows into the bf16 cache at (sequence, position) of every used row.
//   row_pos[r] / row_seq[r]: position (-1: unused) and sequence slot of activation row r;
//   rope_s: (cos, sin) of rows jb .. jb+31 staged in shared memory, [j][hd/2], or nullptr to read
//   the tables in global memory.
__device__ __forceinline__ void epilogue_qkv(const GemmArgs& g, int tile, int row, int jb, int nj,
                                             float (*stage)[33], const int* row_pos, const int* row_seq,
                                             const float2* rope_s) {
    const ModelDims& d = g.dims;
    const int mat = tile / g.tiles_per_map;
    const int col = (tile % g.tiles_per_map) * 128 + row;
    const int hd = d.head_dim, half = hd >> 1;
    const int head = col / hd, idx = col % hd;
    const bool lower = idx < half;
    const int prow = lower ? row + half : row - half;
    const int fi = idx % half;
    if (col < g.n_out) {
#pragma unroll 1
        for (int j = 0; j < nj; ++j) {
            const int pos = row_pos[jb + j];
            if (pos < 0) continue;
            float val = stage[row][j];
            if (mat < 2) {
                const float2 cs = rope_s ? rope_s[j * half + fi]
                                         : make_float2(__ldg(&g.rope_cos[(int64_t)pos * half + fi]),
                                                       __ldg(&g.rope_sin[(int64_t)pos * half + fi]));
                const float other = stage[prow][j];
                val = lower ? (val * cs.x - other * cs.y) : (other * cs.y + val * cs.x);
            }
            if (mat == 0) {
                g.out_f32[(int64_t)(jb + j) * g.ld + col] = val;
            } else {
                __nv_bfloat16* cache = mat == 1 ? g.kcache : g.vcache;
                cache[kv_row_index(d, g.layer, row_seq[jb + j], head, pos) * hd + idx] = __float2bfloat16_rn(val);
            }
        }
    }
    epi_sync();
}

// The same for the wide kernel (blocks of up to 32 rows, rotary factors read from the tables in global
// memory): a tile of many rows is not latency-critical code, so eight rows are in flight at a time --
// their positions, rotary factors and staged values are all requested before any is used.
__device__ __forceinline__ void epilogue_qkv_wide(const GemmArgs& g, int tile, int row, int jb, int nj,
                                                  float (*stage)[33], const int* row_pos, const int* row_seq) {
    const ModelDims& d = g.dims;
    const int mat = tile / g.tiles_per_map;
    const int col = (tile % g.tiles_per_map) * 128 + row;
    const int hd = d.head_dim, half = hd >> 1;
    const int head = col / hd, idx = col % hd;
    const bool lower = idx < half;
    const int prow = lower ? row + half : row - half;
    const int fi = idx % half;
    if (col < g.n_out) {
        const int64_t thread_off = (((int64_t)g.layer * d.max_batch * d.n_heads + head) * d.max_seq) * hd + idx;
        const int64_t seq_stride = (int64_t)d.n_heads * d.max_seq * hd;
        constexpr int kU = 8;
#pragma unroll 1
        for (int j0 = 0; j0 < nj; j0 += kU) {
            int pos[kU];
            float2 cs[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                pos[u] = j0 + u < nj ? row_pos[jb + j0 + u] : -1;
                cs[u] = make_float2(1.f, 0.f);
                if (mat < 2 && pos[u] >= 0)
                    cs[u] = make_float2(__ldg(&g.rope_cos[(int64_t)pos[u] * half + fi]), __ldg(&g.rope_sin[(int64_t)pos[u] * half + fi]));
            }
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                if (pos[u] < 0) continue;
                const int j = j0 + u;
                float v = stage[row][j];
                if (mat < 2) {
                    const float other = stage[prow][j];
                    v = lower ? (v * cs[u].x - other * cs[u].y) : (other * cs[u].y + v * cs[u].x);
                }
                if (mat == 0) {
                    g.out_f32[(int64_t)(jb + j) * g.ld + col] = v;
                } else {
                    __nv_bfloat16* cache = mat == 1 ? g.kcache : g.vcache;
                    cache[thread_off + row_seq[jb + j] * seq_stride + (int64_t)pos[u] * hd] = __float2bfloat16_rn(v);
                }
            }
        }
    }
    epi_sync();
}

// Row-major variant for the wide kernel: thread t takes activation row j = t & 31 of the block and the 16 rotary
// pairs 16 (t >> 5) .. + 15 of the tile, i.e. two runs of 16 consecutive features.  The rotary factors of a row are
// then 64 contiguous bytes per table and the results leave as 16-byte stores; nothing in a thread's work depends
// on another load, so the whole block is one round trip instead of one per row.  Same arithmetic per element as
// epilogue_qkv.  Requires head_dim = 64 or 128 (a tile of 128 features holds whole heads).
__device__ __forceinline__ void epilogue_qkv_rows(const GemmArgs& g, int tile, int t, int jb, int nj,
                                                  float (*stage)[33], const int* row_pos, const int* row_seq) {
    const ModelDims& d = g.dims;
    const int mat = tile / g.tiles_per_map;
    const int col0 = (tile % g.tiles_per_map) * 128;
    const int hd = d.head_dim, half = hd >> 1;
    const int j = t & 31, p0 = (t >> 5) * 16;            // row of the block, first rotary pair
    const int f_lo = (p0 / half) * hd + (p0 % half);     // feature of the pair's lower element inside the tile
    const int f_hi = f_lo + half;
    const int fi0 = p0 % half;
    const int pos = j < nj ? row_pos[jb + j] : -1;
    if (pos >= 0) {
        float lo[16], hi[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) { lo[i] = stage[f_lo + i][j]; hi[i] = stage[f_hi + i][j]; }
        if (mat < 2) {
            float4 c4[4], s4[4];
            const float4* cp = reinterpret_cast<const float4*>(g.rope_cos + (int64_t)pos * half + fi0);
            const float4* sp = reinterpret_cast<const float4*>(g.rope_sin + (int64_t)pos * half + fi0);
#pragma unroll
            for (int u = 0; u < 4; ++u) { c4[u] = __ldg(cp + u); s4[u] = __ldg(sp + u); }
            const float* c = reinterpret_cast<const float*>(c4);
            const float* sn = reinterpret_cast<const float*>(s4);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float a = lo[i], b = hi[i];
                lo[i] = a * c[i] - b * sn[i];
                hi[i] = a * sn[i] + b * c[i];
            }
        }
        if (mat == 0) {
            float* o = g.out_f32 + (int64_t)(jb + j) * g.ld + col0;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                *reinterpret_cast<float4*>(o + f_lo + 4 * u) = make_float4(lo[4 * u], lo[4 * u + 1], lo[4 * u + 2], lo[4 * u + 3]);
                *reinterpret_cast<float4*>(o + f_hi + 4 * u) = make_float4(hi[4 * u], hi[4 * u + 1], hi[4 * u + 2], hi[4 * u + 3]);
            }
        } else {
            __nv_bfloat16* cache = mat == 1 ? g.kcache : g.vcache;
            const int head = (col0 + f_lo) / hd, idx = (col0 + f_lo) % hd;
            __nv_bfloat16* dst = cache + (kv_row_index(d, g.layer, row_seq[jb + j], head, pos) * hd + idx);
            auto pack = [](float x, float y) {
                return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(y)) << 16);
            };
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                *reinterpret_cast<uint4*>(dst + 8 * u) = make_uint4(pack(lo[8 * u], lo[8 * u + 1]), pack(lo[8 * u + 2], lo[8 * u + 3]),
                                                                     pack(lo[8 * u + 4], lo[8 * u + 5]), pack(lo[8 * u + 6], lo[8 * u + 7]));
                *reinterpret_cast<uint4*>(dst + half + 8 * u) = make_uint4(pack(hi[8 * u], hi[8 * u + 1]), pack(hi[8 * u + 2], hi[8 * u + 3]),
                                                                            pack(hi[8 * u + 4], hi[8 * u + 5]), pack(hi[8 * u + 6], hi[8 * u + 7]));
            }
        }
    }
    epi_sync();
}

// SwiGLU: tile rows 0..63 are gate features, 64..127 the matching up features.
__device__ __forceinline__ void epilogue_swiglu(const GemmArgs& g, int tile, int row, int jb, int nj,
                                                float (*stage)[33]) {
    const int fi = row & 63, f = tile * 64 + fi;
    if (f < g.n_out) {
#pragma unroll 1
        for (int j = row >> 6; j < nj; j += 2) {
            const float gate = stage[g.gate_second ? 64 + fi : fi][j], up = stage[g.gate_second ? fi : 64 + fi][j];
            store_act(g.out_act, kActSplit, g.rc, jb + j, f, g.n_out, gate / (1.f + expf(-gate)) * up);
        }
    }
    epi_sync();
}

// Row-major variants for the wide kernel (see epilogue_qkv_rows): thread t takes activation row j = t & 31 of
// the block and a run of consecutive features chosen by t >> 5, so that the residual stream, the split operand and
// the gains move as 16-byte accesses and nothing waits for an earlier load of the same thread.
__device__ __forceinline__ uint32_t pack_bf16x2(float x, float y) {
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(y)) << 16);
}
// hi = bf16(v), lo = bf16(v - hi) of 8 values, as the two 16-byte words of the split layout
__device__ __forceinline__ void split8(const float (&v)[8], uint4& hi, uint4& lo) {
    uint32_t h[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat16 a = __float2bfloat16_rn(v[2 * i]), b = __float2bfloat16_rn(v[2 * i + 1]);
        h[i] = (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
        l[i] = pack_bf16x2(v[2 * i] - __bfloat162float(a), v[2 * i + 1] - __bfloat162float(b));
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

// x[r, n] += acc for 32 features per thread; requires n_out % 128 == 0.  The sum of squares of a row is taken
// over ascending features: 32 per thread, then the four threads of the row in ascending order.
__device__ __forceinline__ void epilogue_resid_rows(const GemmArgs& g, int tile, int t, int jb, int nj,
                                                    float (*stage)[33], float* red_f) {
    const int j = t & 31, w = t >> 5, f0 = 32 * w;
    const int col0 = tile * 128 + f0;
    const bool fold = g.xs_out != nullptr;
    float sq = 0.f;
    if (j < nj) {
        float* xrow = g.out_f32 + (int64_t)(jb + j) * g.ld + col0;
        float4 x4[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x4[u] = __ldcg(reinterpret_cast<const float4*>(xrow) + u);
        float xn[32];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            xn[4 * u] = stage[f0 + 4 * u][j] + x4[u].x; xn[4 * u + 1] = stage[f0 + 4 * u + 1][j] + x4[u].y;
            xn[4 * u + 2] = stage[f0 + 4 * u + 2][j] + x4[u].z; xn[4 * u + 3] = stage[f0 + 4 * u + 3][j] + x4[u].w;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            reinterpret_cast<float4*>(xrow)[u] = make_float4(xn[4 * u], xn[4 * u + 1], xn[4 * u + 2], xn[4 * u + 3]);
        if (fold) {
            __nv_bfloat16* hi_row = reinterpret_cast<__nv_bfloat16*>(g.xs_out) + (int64_t)(jb + j) * g.n_out + col0;
            __nv_bfloat16* lo_row = hi_row + (int64_t)g.rc * g.n_out;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float4 ga = __ldg(reinterpret_cast<const float4*>(g.gain_next + col0) + 2 * u);
                const float4 gb = __ldg(reinterpret_cast<const float4*>(g.gain_next + col0) + 2 * u + 1);
                const float v[8] = {xn[8 * u] * ga.x, xn[8 * u + 1] * ga.y, xn[8 * u + 2] * ga.z, xn[8 * u + 3] * ga.w,
                                    xn[8 * u + 4] * gb.x, xn[8 * u + 5] * gb.y, xn[8 * u + 6] * gb.z, xn[8 * u + 7] * gb.w};
                uint4 hi, lo;
                split8(v, hi, lo);
                reinterpret_cast<uint4*>(hi_row)[u] = hi;
                reinterpret_cast<uint4*>(lo_row)[u] = lo;
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) sq = __fmaf_rn(xn[i], xn[i], sq);
        }
    }
    if (!fold) { epi_sync(); return; }
    red_f[w * 32 + j] = sq;
    epi_sync();
    if (w == 0 && j < nj)
        g.ss_out[(int64_t)tile * g.rc + jb + j] = ((red_f[j] + red_f[32 + j]) + red_f[64 + j]) + red_f[96 + j];
    epi_sync();
}

// h = silu(gate) * up for 16 features per thread; requires n_out % 16 == 0
__device__ __forceinline__ void epilogue_swiglu_rows(const GemmArgs& g, int tile, int t, int jb, int nj,
                                                     float (*stage)[33]) {
    const int j = t & 31, f0 = 16 * (t >> 5);
    const int f = tile * 64 + f0;
    if (j < nj && f < g.n_out) {
        const int gb = g.gate_second ? 64 : 0, ub = g.gate_second ? 0 : 64;
        __nv_bfloat16* hi_row = reinterpret_cast<__nv_bfloat16*>(g.out_act) + (int64_t)(jb + j) * g.n_out + f;
        __nv_bfloat16* lo_row = hi_row + (int64_t)g.rc * g.n_out;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            float v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float gate = stage[gb + f0 + 8 * u + i][j], up = stage[ub + f0 + 8 * u + i][j];
                v[i] = gate / (1.f + expf(-gate)) * up;
            }
            uint4 hi, lo;
            split8(v, hi, lo);
            reinterpret_cast<uint4*>(hi_row)[u] = hi;
            reinterpret_cast<uint4*>(lo_row)[u] = lo;
        }
    }
    epi_sync();
}

// LM head: optional logits store, then the tile's (max, lowest argmax) for every used row.
__device__ __forceinline__ void epilogue_lmhead(const GemmArgs& g, int tile, int row, int jb, int nj,
                                                float (*stage)[33], float* red_f, int* red_i) {
    const int v = tile * 128 + row;
    const bool valid = v < g.n_out;
    const int warp = row >> 5, lane = row & 31;
#pragma unroll 1
    for (int j = 0; j < nj; ++j) {
        const float a = stage[row][j];
        if (g.out_f32 && valid) g.out_f32[(int64_t)(jb + j) * g.ld + v] = a;
        float bv = valid ? a : -INFINITY;
        int bi = valid ? v : 0x7fffffff;
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { red_f[warp * 32 + j] = bv; red_i[warp * 32 + j] = bi; }
    }
    epi_sync();
    if (row < nj) {
        float bv = red_f[row]; int bi = red_i[row];
        for (int w = 1; w < 4; ++w) {
            const float ov = red_f[w * 32 + row]; const int oi = red_i[w * 32 + row];
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        g.part_max[(int64_t)tile * g.rc + jb + row] = bv;
        g.part_idx[(int64_t)tile * g.rc + jb + row] = bi;
    }
    epi_sync();
}

// Partial tiles in the workspace: [cta][slot][q][feature] float4, q = group of four activation rows
// (qn groups per slot).  The 32 features of a warp are 512 consecutive bytes, so one store or polling
// load of a warp touches four lines.
__device__ __forceinline__ float4* ws_slot(float* ws, int qn, int cta, int slot, int feature) {
    return reinterpret_cast<float4*>(ws) + ((int64_t)cta * 2 + slot) * ((int64_t)qn * 128) + feature;
}

// Range of flat (tile, chunk) work items owned by CTA b of G.
__device__ __forceinline__ int64_t cta_begin(int64_t work, int b, int G) { return work * b / G; }

}  // namespace llma

// Tensor-core split-KV attention (library-private interface).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace llma {

constexpr int kAttnChunk = 128;  // cache positions per CTA; chunk c covers [128c, 128c + 128)

struct AttnArgs {
    ModelDims dims;
    int32_t layer;
    int32_t n_chunks;        // grid.x = ceil(max_seq / chunk_pos); CTAs past a sequence's last position exit
    int32_t tiles;           // 128-position tiles per CTA: 1, or 2 / 4 (attention_long_kernel; steps of at most 16 rows per sequence)
    int32_t chunk_pos;       // cache positions per CTA = 128 * tiles
    const RowDesc* rows;
    const SeqState* seq_state;  // decode steps: kv_len here is the length committed before this step
    int32_t prompt;          // 1: a prompt pass (many rows of one sequence): the kernel instance with the per-warp query tiles
    int32_t early_kv;        // 1: chunks wholly below that length may be fetched before the predecessor has finished
    int32_t n_rows;          // row slots of this pass (grid of the merge kernel)
    const float* qkv;        // [rows][3*H*hd] fp32, q already rotated
    void* attn_out;          // ActLayout kActSplit [2 rc][H*hd]
    float* ws_o;             // chunk partials [head][chunk][rc][hd] fp32
    float* ws_ml;            // [head][chunk][rc][2] = (max, sum)
    unsigned long long* stamps;  // measurement builds: timeline block (see LLMA_STAMPS), else unused
    int32_t* dev_err;
};

cudaError_t init_attention_mma();
void launch_attention_mma(cudaStream_t st, const AttnArgs& a, const CUtensorMap& map_k, const CUtensorMap& map_v);

}  // namespace llma

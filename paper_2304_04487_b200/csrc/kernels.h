// Launch wrappers of the engine's kernels (library-private).
#pragma once
#include "common.cuh"

namespace llma {

// ---- integer side (kernels_int.cu) ----------------------------------------------------
// Arguments of step_tail_kernel: acceptance + K/V commit of the forward pass that has just finished
// (do_accept) and trigger search + copy + row packing for the one that follows (do_plan).
struct TailArgs {
    ModelDims dims;
    SeqState* st;
    RowDesc* rows;
    const int32_t *ref, *doc_start, *doc_end;
    int32_t* y;
    int32_t y_cap;
    int32_t n, k;
    int32_t do_accept, do_plan;
    // accept
    const float* part_max;     // [n_tiles][row_cap] per-tile maxima of the LM head, or nullptr: out_tok is final
    const int32_t* part_idx;
    int32_t n_tiles;
    int32_t* out_tok;          // [row_cap]
    int32_t n_rows;            // row slots of a decoding step (decode_rows)
    // replay
    const int32_t* trace;      // [max_batch][trace_cap][2] = (rows, emitted) of every step, or nullptr
    const int32_t* target;     // [max_batch][y_cap] the text to reproduce
    int32_t trace_cap;
    int32_t* dev_err;
};


void launch_step_tail(cudaStream_t st, const TailArgs& a);
// embedding gather over the first n_rows row slots (rows not in use are zero-filled)
void launch_embed(cudaStream_t st, const ModelDims& dims, bool bf16, int n_rows, const RowDesc* rows, const void* emb,
                  float* x, int32_t* dev_err);
// bf16 embedding gather with the first RMSNorm folded in: x, xs = split(x * gain), ss[tile][row]
void launch_embed_norm(cudaStream_t st, const ModelDims& dims, int n_rows, const RowDesc* rows, const void* emb,
                       const float* gain, float* x, void* xs, float* ss, int32_t* dev_err);

// ---- SIMT (CUDA-core) kernels, fp32 or bf16 storage (kernels_simt.cu) -------------------
// x_hat[r,:] = rmsnorm(x[r,:]) * g in the given ActLayout (rc = row capacity); unused rows are zero-filled
void launch_rmsnorm(cudaStream_t st, int act_layout, int n_rows, int rc, const RowDesc* rows, const float* x,
                    const float* g, void* x_hat, int32_t d, float eps);
// out[r, n] (+)= sum_k W[n,k] * a[r,k] for r < rows_used; a fp32 [rows][k_in]; out fp32, leading dimension ld_out
// (every launcher below takes n_rows = the row slots of the pass: the decode or the prompt-pass capacity)
void launch_gemm_simt(cudaStream_t st, bool bf16, const RowDesc* rows, const void* W, const float* a, float* out,
                      int32_t n_out, int32_t k_in, int32_t ld_out, bool accumulate);
// rotary embedding of q,k in qkv[r, 0:2*HD]; K/V rows appended to the cache at (seq, pos)
void launch_qkv_post(cudaStream_t st, bool bf16, const ModelDims& dims, int layer, int n_rows, const RowDesc* rows,
                     float* qkv, const float* rope_cos, const float* rope_sin, void* kcache, void* vcache);
// causal attention of every used row over its sequence's cache rows [0, pos]
void launch_attention_simt(cudaStream_t st, bool bf16, const ModelDims& dims, int layer, int n_rows,
                           const RowDesc* rows, const float* qkv, const void* kcache, const void* vcache,
                           void* attn_out, int act_layout);
// h = silu(gate) * up (fp32); gate_up is [rows][2*d_ffn] (gate first)
void launch_silu_mul(cudaStream_t st, int n_rows, const RowDesc* rows, const float* gate_up, float* h, int32_t d_ffn);
// out_tok[r] = argmax_v logits[r, v] (lowest index on ties)
void launch_argmax(cudaStream_t st, int n_rows, const RowDesc* rows, const float* logits, int32_t vocab, int32_t* out_tok);

}  // namespace llma

// Launch wrappers of the engine's kernels (library-private).
#pragma once
#include "common.cuh"

namespace llma {

// ---- integer side (kernels_int.cu) ----------------------------------------------------
void launch_plan(cudaStream_t st, const ModelDims& dims, SeqState* seq, RowDesc* rows, const int32_t* ref,
                 const int32_t* doc_start, const int32_t* doc_end, const int32_t* y, int32_t y_cap, int32_t n,
                 int32_t k, int32_t* dev_err);
void launch_embed(cudaStream_t st, const ModelDims& dims, bool bf16, const RowDesc* rows, const void* emb, float* x,
                  int32_t* dev_err);
// bf16 embedding gather with the first RMSNorm folded in: x, xs = split(x * gain), ss[tile][row]
void launch_embed_norm(cudaStream_t st, const ModelDims& dims, const RowDesc* rows, const void* emb, const float* gain,
                       float* x, void* xs, float* ss, int32_t* dev_err);
void launch_accept(cudaStream_t st, const ModelDims& dims, SeqState* seq, const int32_t* ref, const int32_t* out_tok,
                   int32_t* y, int32_t y_cap);

// ---- SIMT (CUDA-core) kernels, fp32 or bf16 storage (kernels_simt.cu) -------------------
// x_hat[r,:] = rmsnorm(x[r,:]) * g in the given ActLayout; unused rows are zero-filled
void launch_rmsnorm(cudaStream_t st, int act_layout, const RowDesc* rows, const float* x, const float* g, void* x_hat,
                    int32_t d, float eps);
// out[r, n] (+)= sum_k W[n,k] * a[r,k] for r < rows_used; a fp32 [rows][k_in]; out fp32, leading dimension ld_out
void launch_gemm_simt(cudaStream_t st, bool bf16, const RowDesc* rows, const void* W, const float* a, float* out,
                      int32_t n_out, int32_t k_in, int32_t ld_out, bool accumulate);
// rotary embedding of q,k in qkv[r, 0:2*HD]; K/V rows appended to the cache at (seq, pos)
void launch_qkv_post(cudaStream_t st, bool bf16, const ModelDims& dims, int layer, const RowDesc* rows, float* qkv,
                     const float* rope_cos, const float* rope_sin, void* kcache, void* vcache);
// causal attention of every used row over its sequence's cache rows [0, pos]
void launch_attention_simt(cudaStream_t st, bool bf16, const ModelDims& dims, int layer, const RowDesc* rows,
                           const float* qkv, const void* kcache, const void* vcache, void* attn_out, int act_layout);
// h = silu(gate) * up (fp32); gate_up is [rows][2*d_ffn] (gate first)
void launch_silu_mul(cudaStream_t st, const RowDesc* rows, const float* gate_up, float* h, int32_t d_ffn);
// out_tok[r] = argmax_v logits[r, v] (lowest index on ties)
void launch_argmax(cudaStream_t st, const RowDesc* rows, const float* logits, int32_t vocab, int32_t* out_tok);

}  // namespace llma

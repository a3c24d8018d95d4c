// Engine object behind the C ABI (library-private).
#pragma once
#include <map>
#include <utility>
#include <vector>

#include "../../include/llma.h"
#include "attention_mma.cuh"
#include "gemm_tcgen05.cuh"
#include "kernels.h"

struct llma_engine {
    llma_config cfg;
    llma::ModelDims dims;
    bool bf16 = false;
    int gemm_impl = LLMA_GEMM_SIMT;
    cudaStream_t stream = nullptr;
    int device = 0;

    // borrowed weights (host copies of the per-layer pointer arrays)
    const void *tok_emb = nullptr, *lm_head = nullptr;
    const float* final_norm = nullptr;
    std::vector<const float*> attn_norm, ffn_norm;
    std::vector<const void*> wq, wk, wv, wo, w_gate, w_up, w_down;

    // device state
    llma::SeqState* seq_state = nullptr;
    llma::RowDesc* rows = nullptr;
    int32_t *ref = nullptr, *doc_start = nullptr, *doc_end = nullptr, *y = nullptr, *out_tok = nullptr;
    int32_t* dev_err = nullptr;
    int32_t y_cap = 0;
    float *x = nullptr, *qkv = nullptr, *gate_up = nullptr, *logits = nullptr;
    void *x_hat = nullptr, *attn = nullptr, *h = nullptr;
    float *rope_cos = nullptr, *rope_sin = nullptr;
    void *kcache = nullptr, *vcache = nullptr;

    // tensor-core GEMM path (bf16): TMA descriptors of weights and activation buffers, work buffers
    struct LayerMaps { CUtensorMap wq, wk, wv, wo, w_gate, w_up, w_down; };
    std::vector<LayerMaps> maps;
    CUtensorMap map_lm_head;
    int decode_nr = 32;             // rows per half used by decoding steps (16 or 32); prefill always uses 32
    int cur_nr = 32;                // what the launches being enqueued use
    int num_sms = 0;
    float* gemm_ws = nullptr;       // split-k partial tiles [num_sms][2][128][32]
    int32_t* gemm_cnt = nullptr;    // (unused by the current kernels)
    float* norm_ss = nullptr;       // per-tile sums of squares of the residual rows [d/128][32]
    float* part_max = nullptr;      // LM-head per-tile maxima [tiles][32]
    int32_t* part_idx = nullptr;

    // tensor-core attention: TMA descriptors of the K/V cache, chunk partials
    CUtensorMap map_kcache, map_vcache;
    int attn_chunks = 0;
    float *attn_ws_o = nullptr, *attn_ws_ml = nullptr;
    int32_t* attn_cnt = nullptr;

    // pinned host staging
    llma::SeqState* h_state = nullptr;
    llma::RowDesc* h_rows = nullptr;
    int32_t* h_err = nullptr;

    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    std::map<std::pair<int, int>, cudaGraphExec_t> step_graphs;  // keyed by (n, k)
    int64_t launches_per_step = 0;
    int64_t launch_counter = 0;  // kernels enqueued since it was last cleared
    bool last_step_valid = false;
    bool prof_on = false;               // llma_profile_steps: record an event after every launch
    std::vector<cudaEvent_t> prof_ev;
    std::vector<int> prof_cls;
    size_t prof_n = 0;
    std::vector<int32_t> prompt_last;  // last prompt token of every sequence (the first pending input)
};

namespace llma {
void note_cuda_error(cudaError_t err);  // remembers the code for llma_last_cuda_error, clears the sticky flag
}

#define CU_TRY(expr)                          \
    do {                                      \
        cudaError_t _e = (expr);              \
        if (_e != cudaSuccess) {              \
            llma::note_cuda_error(_e);        \
            return LLMA_ERR_CUDA;             \
        }                                     \
    } while (0)

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

    // row capacities (multiples of 16): activation buffers hold row_cap rows; a decoding step uses at most
    // decode_rows = max_batch * (max_k + 1) of them, a prompt pass prefill_rows
    int row_cap = 0, decode_rows = 0, prefill_rows = 0;

    // tensor-core GEMM path (bf16): TMA descriptors of weights and activation buffers, work buffers
    struct LayerMaps { CUtensorMap wq, wk, wv, wo, w_gate, w_up, w_down; };
    std::vector<LayerMaps> maps;    // 2-D views (gemm_wide_kernel; gate/up of both kernels)
    std::vector<LayerMaps> maps2;   // chunk-pair views (gemm_ws_kernel; gate/up entries are the 2-D ones)
    CUtensorMap map_lm_head, map_lm_head2;
    struct PairMap { CUtensorMap map; int gate_second; };   // gate and up matrices of a layer in one view (gemm_ws_kernel)
    std::vector<PairMap> gate_up_map;
    // activation operands of gemm_wide_kernel: boxes of min(32, nr), min(64, nr), min(128, nr) and nr rows (the kernel
    // takes the smallest that holds the step's rows)
    struct ActMaps { CUtensorMap x_hat[4], attn[4], h[4]; };
    ActMaps act_decode, act_prefill;
    bool decode_wide = false;       // decoding steps of more than 32 rows use gemm_wide_kernel
    int decode_nr = 32;             // rows the decoding GEMMs are shaped for (16 / 32 narrow, decode_rows wide)
    // what the launches being enqueued use (decoding step or prompt pass)
    bool cur_wide = false, cur_prompt = false;
    int cur_nr = 32, cur_rows = 32;
    const ActMaps* cur_maps = nullptr;
    int num_sms = 0;
    unsigned long long* stamps = nullptr;  // timeline blocks (allocated in measurement builds only)
    int stamp_id = 0;                      // projections enqueued since the step began
    float* gemm_ws = nullptr;       // partial tiles of gemm_ws_kernel [num_sms][2][8][128] float4
    float* gemm_ws_wide = nullptr;  // partial tiles of gemm_wide_kernel [num_sms][2][wide_nr / 4][128] float4
    size_t gemm_ws_bytes = 0, gemm_ws_wide_bytes = 0;
    float* norm_ss = nullptr;       // per-tile sums of squares of the residual rows [d/128][row_cap]
    float* part_max = nullptr;      // LM-head per-tile maxima [tiles][row_cap]
    int32_t* part_idx = nullptr;

    // tensor-core attention: TMA descriptors of the K/V cache, chunk partials
    CUtensorMap map_kcache, map_vcache;
    int attn_chunks = 0;
    int attn_tiles = 1;             // 128-position tiles per attention CTA in decoding steps (a function of the capacity only)
    float *attn_ws_o = nullptr, *attn_ws_ml = nullptr;

    // replay of a given step sequence (llma_generate_forced)
    int32_t *trace = nullptr, *target = nullptr;
    int32_t trace_cap = 0;

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

// C ABI of the LLMA engine: object lifetime, prompt prefill, reference upload, the decoding
// step (Algorithm 1's loop body) and the whole decoding loop.  See include/llma.h.
#include "engine.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

using namespace llma;

static thread_local int g_last_cuda_error = 0;
void llma::note_cuda_error(cudaError_t err) {
    g_last_cuda_error = (int)err;
    (void)cudaGetLastError();
}

static size_t esize(const llma_engine* e) { return e->bf16 ? 2 : 4; }

template <typename T>
static cudaError_t dalloc(T** p, size_t count, bool zero = true) {
    cudaError_t r = cudaMalloc((void**)p, count * sizeof(T));
    if (r != cudaSuccess) return r;
    if (zero) r = cudaMemset(*p, 0, count * sizeof(T));
    return r;
}

extern "C" int llma_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" const char* llma_strerror(int s) {
    switch (s) {
        case LLMA_OK: return "ok";
        case LLMA_ERR_NULL: return "required pointer is NULL";
        case LLMA_ERR_CONFIG: return "unsupported or inconsistent configuration";
        case LLMA_ERR_TOKEN_RANGE: return "token id outside [0, vocab)";
        case LLMA_ERR_CAPACITY: return "sequence capacity (max_seq / max_batch) exceeded";
        case LLMA_ERR_REF_TOO_LONG: return "reference too long or malformed document offsets";
        case LLMA_ERR_STATE: return "call not valid in the current state";
        case LLMA_ERR_CUDA: return "CUDA call failed";
        case LLMA_ERR_DEVICE_TIMEOUT: return "bounded device-side wait ran out";
        case LLMA_ERR_ARG: return "argument out of range";
        default: return "unknown status";
    }
}

static void free_engine(llma_engine* e) {
    if (!e) return;
    for (auto& kv : e->step_graphs) cudaGraphExecDestroy(kv.second);
    cudaFree(e->seq_state); cudaFree(e->rows); cudaFree(e->ref); cudaFree(e->doc_start); cudaFree(e->doc_end);
    cudaFree(e->y); cudaFree(e->out_tok); cudaFree(e->dev_err); cudaFree(e->x); cudaFree(e->qkv);
    cudaFree(e->gate_up); cudaFree(e->logits); cudaFree(e->x_hat); cudaFree(e->attn); cudaFree(e->h);
    cudaFree(e->rope_cos); cudaFree(e->rope_sin); cudaFree(e->kcache); cudaFree(e->vcache);
    cudaFree(e->attn_ws_o); cudaFree(e->attn_ws_ml); cudaFree(e->trace); cudaFree(e->target);
    cudaFree(e->gemm_ws); cudaFree(e->stamps); cudaFree(e->gemm_ws_wide); cudaFree(e->part_max); cudaFree(e->part_idx); cudaFree(e->norm_ss);
    if (e->h_state) cudaFreeHost(e->h_state);
    if (e->h_rows) cudaFreeHost(e->h_rows);
    if (e->h_err) cudaFreeHost(e->h_err);
    for (cudaEvent_t ev : e->prof_ev) cudaEventDestroy(ev);
    if (e->ev0) cudaEventDestroy(e->ev0);
    if (e->ev1) cudaEventDestroy(e->ev1);
    delete e;
}

extern "C" int llma_create(const llma_config* cfg, const llma_weights* w, void* cuda_stream, llma_engine** out) {
    if (!cfg || !w || !out) return LLMA_ERR_NULL;
    *out = nullptr;
    const int L = cfg->n_layers;
    if (L < 1 || cfg->d_model < 64 || cfg->n_heads < 1 || cfg->d_ffn < 64 || cfg->vocab < 2) return LLMA_ERR_CONFIG;
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return LLMA_ERR_CONFIG;
    const int HD = cfg->n_heads * cfg->head_dim;
    if (cfg->d_model % 64 || HD % 64 || cfg->d_ffn % 64) return LLMA_ERR_CONFIG;
    if (cfg->dtype != LLMA_DTYPE_F32 && cfg->dtype != LLMA_DTYPE_BF16) return LLMA_ERR_CONFIG;
    if (cfg->max_batch < 1 || cfg->max_batch > kSeqCap || cfg->max_k < 0 ||
        (int64_t)cfg->max_batch * (cfg->max_k + 1) > kRowCap)
        return LLMA_ERR_CONFIG;
    if (cfg->max_seq < 2 || cfg->max_ref < 0 || !(cfg->rms_eps >= 0.f) || !(cfg->rope_theta > 0.f)) return LLMA_ERR_CONFIG;
    if (cfg->gemm_impl < LLMA_GEMM_AUTO || cfg->gemm_impl > LLMA_GEMM_TCGEN05) return LLMA_ERR_CONFIG;
    if (!w->tok_emb || !w->lm_head || !w->final_norm || !w->attn_norm || !w->wq || !w->wk || !w->wv || !w->wo ||
        !w->ffn_norm || !w->w_gate || !w->w_up || !w->w_down)
        return LLMA_ERR_NULL;
    for (int l = 0; l < L; ++l)
        if (!w->attn_norm[l] || !w->wq[l] || !w->wk[l] || !w->wv[l] || !w->wo[l] || !w->ffn_norm[l] ||
            !w->w_gate[l] || !w->w_up[l] || !w->w_down[l])
            return LLMA_ERR_NULL;

    int dev = 0;
    CU_TRY(cudaGetDevice(&dev));
    llma_engine* e = new (std::nothrow) llma_engine();
    if (!e) return LLMA_ERR_CUDA;
    e->cfg = *cfg;
    e->device = dev;
    e->stream = (cudaStream_t)cuda_stream;
    e->bf16 = cfg->dtype == LLMA_DTYPE_BF16;
    const bool tc_ok = cfg->dtype == LLMA_DTYPE_BF16 && HD % 128 == 0 && cfg->d_model % 128 == 0;
    if (cfg->gemm_impl == LLMA_GEMM_TCGEN05 && !tc_ok) { delete e; return LLMA_ERR_CONFIG; }
    e->gemm_impl = cfg->gemm_impl == LLMA_GEMM_AUTO ? (tc_ok ? LLMA_GEMM_TCGEN05 : LLMA_GEMM_SIMT) : cfg->gemm_impl;
    ModelDims& d = e->dims;
    d.n_layers = L; d.d_model = cfg->d_model; d.n_heads = cfg->n_heads; d.head_dim = cfg->head_dim;
    d.d_ffn = cfg->d_ffn; d.vocab = cfg->vocab; d.hd_total = HD; d.max_batch = cfg->max_batch;
    d.max_seq = cfg->max_seq; d.max_ref = cfg->max_ref > 0 ? cfg->max_ref : 1; d.kp1 = cfg->max_k + 1;
    d.rms_eps = cfg->rms_eps; d.eos_id = cfg->eos_id;
    // Row capacities.  Decoding steps hold at most max_batch * (max_k + 1) rows; prompt passes push up to
    // prefill_rows consecutive positions of one sequence through the same kernels (128 on the tensor-core
    // path, where the projections are compute-bound from about a hundred rows on).
    e->decode_rows = (d.max_batch * d.kp1 + 15) / 16 * 16;
    e->prefill_rows = std::max(e->decode_rows, e->gemm_impl == LLMA_GEMM_TCGEN05 ? 128 : 32);
    e->row_cap = e->prefill_rows;
    d.row_cap = e->row_cap;
    e->tok_emb = w->tok_emb; e->lm_head = w->lm_head; e->final_norm = w->final_norm;
    for (int l = 0; l < L; ++l) {
        e->attn_norm.push_back(w->attn_norm[l]); e->ffn_norm.push_back(w->ffn_norm[l]);
        e->wq.push_back(w->wq[l]); e->wk.push_back(w->wk[l]); e->wv.push_back(w->wv[l]); e->wo.push_back(w->wo[l]);
        e->w_gate.push_back(w->w_gate[l]); e->w_up.push_back(w->w_up[l]); e->w_down.push_back(w->w_down[l]);
    }
    e->y_cap = d.max_seq;
    e->prompt_last.assign((size_t)d.max_batch, 0);

#define CREATE_TRY(expr)                              \
    do {                                              \
        cudaError_t _e = (expr);                      \
        if (_e != cudaSuccess) {                      \
            llma::note_cuda_error(_e);                \
            free_engine(e);                           \
            return LLMA_ERR_CUDA;                     \
        }                                             \
    } while (0)

    const size_t B = d.max_batch, es = esize(e);
    CREATE_TRY(dalloc(&e->seq_state, B));
    CREATE_TRY(dalloc(&e->rows, 1));
    CREATE_TRY(dalloc(&e->ref, B * d.max_ref));
    CREATE_TRY(dalloc(&e->doc_start, B * d.max_ref));
    CREATE_TRY(dalloc(&e->doc_end, B * d.max_ref));
    CREATE_TRY(dalloc(&e->y, B * e->y_cap));
    const size_t RC = (size_t)e->row_cap;
    CREATE_TRY(dalloc(&e->out_tok, RC));
    e->trace_cap = e->y_cap;
    CREATE_TRY(dalloc(&e->trace, B * e->trace_cap * 2));
    CREATE_TRY(dalloc(&e->target, B * e->y_cap));
    CREATE_TRY(dalloc(&e->dev_err, 1));
    CREATE_TRY(dalloc(&e->x, RC * d.d_model));
    CREATE_TRY(dalloc(&e->qkv, RC * 3 * HD));
    if (e->gemm_impl != LLMA_GEMM_TCGEN05) CREATE_TRY(dalloc(&e->gate_up, RC * 2 * d.d_ffn));
    if (e->gemm_impl != LLMA_GEMM_TCGEN05 || cfg->keep_logits) CREATE_TRY(dalloc(&e->logits, RC * d.vocab));
    // activation operands: fp32 [rc][K] (CUDA-core GEMM) or split bf16 [2 rc][K] (tensor cores): 4 bytes per element
    CREATE_TRY(dalloc((char**)&e->x_hat, RC * d.d_model * 4));
    CREATE_TRY(dalloc((char**)&e->attn, RC * HD * 4));
    CREATE_TRY(dalloc((char**)&e->h, RC * d.d_ffn * 4));
    const size_t kv_elems = (size_t)L * B * d.n_heads * d.max_seq * d.head_dim;
    CREATE_TRY(dalloc((char**)&e->kcache, kv_elems * es));
    CREATE_TRY(dalloc((char**)&e->vcache, kv_elems * es));

    // rotary table: angle(pos, i) = pos * theta^(-2i/hd), evaluated in double on the host
    {
        const int half = d.head_dim / 2;
        std::vector<float> c((size_t)d.max_seq * half), s((size_t)d.max_seq * half);
        for (int i = 0; i < half; ++i) {
            const double inv = std::pow((double)cfg->rope_theta, -2.0 * (double)i / (double)d.head_dim);
            for (int p = 0; p < d.max_seq; ++p) {
                const double a = (double)p * inv;
                c[(size_t)p * half + i] = (float)std::cos(a);
                s[(size_t)p * half + i] = (float)std::sin(a);
            }
        }
        CREATE_TRY(dalloc(&e->rope_cos, c.size(), false));
        CREATE_TRY(dalloc(&e->rope_sin, s.size(), false));
        CREATE_TRY(cudaMemcpy(e->rope_cos, c.data(), c.size() * 4, cudaMemcpyHostToDevice));
        CREATE_TRY(cudaMemcpy(e->rope_sin, s.data(), s.size() * 4, cudaMemcpyHostToDevice));
    }
    if (e->gemm_impl == LLMA_GEMM_TCGEN05) {
        cudaDeviceProp prop;
        CREATE_TRY(cudaGetDeviceProperties(&prop, dev));
        if (prop.major != 10) { free_engine(e); return LLMA_ERR_CONFIG; }  // tcgen05 needs sm_100
        e->num_sms = prop.multiProcessorCount;
        const int vt = (d.vocab + 127) / 128;
        // hand-over slots start out empty: every word the all-ones pattern (see gemm_ws_kernel)
        e->gemm_ws_bytes = (size_t)e->num_sms * 2 * 128 * 32 * sizeof(float);
        CREATE_TRY(dalloc((char**)&e->gemm_ws, e->gemm_ws_bytes, false));
        CREATE_TRY(cudaMemset(e->gemm_ws, 0xFF, e->gemm_ws_bytes));
        e->gemm_ws_wide_bytes = (size_t)e->num_sms * 2 * 128 * RC * sizeof(float);
        CREATE_TRY(dalloc((char**)&e->gemm_ws_wide, e->gemm_ws_wide_bytes, false));
        CREATE_TRY(cudaMemset(e->gemm_ws_wide, 0xFF, e->gemm_ws_wide_bytes));
        CREATE_TRY(dalloc(&e->part_max, (size_t)vt * RC));
        CREATE_TRY(dalloc(&e->part_idx, (size_t)vt * RC));
        CREATE_TRY(dalloc(&e->norm_ss, (size_t)((d.d_model + 127) / 128) * RC));
#ifdef LLMA_STAMPS
        CREATE_TRY(dalloc(&e->stamps, (size_t)kStampLaunches * kStampSlots * 8));
#endif
        e->maps.resize(L);
        e->maps2.resize(L);
        e->gate_up_map.resize(L);
        bool pair_ok = true;
        int bad = 0;
        for (int l = 0; l < L; ++l) {
            llma_engine::LayerMaps& m = e->maps[l];
            bad |= make_tensor_map_bf16(&m.wq, e->wq[l], HD, d.d_model, 128);
            bad |= make_tensor_map_bf16(&m.wk, e->wk[l], HD, d.d_model, 128);
            bad |= make_tensor_map_bf16(&m.wv, e->wv[l], HD, d.d_model, 128);
            bad |= make_tensor_map_bf16(&m.wo, e->wo[l], d.d_model, HD, 128);
            bad |= make_tensor_map_bf16(&m.w_gate, e->w_gate[l], d.d_ffn, d.d_model, 64);
            bad |= make_tensor_map_bf16(&m.w_up, e->w_up[l], d.d_ffn, d.d_model, 64);
            bad |= make_tensor_map_bf16(&m.w_down, e->w_down[l], d.d_model, d.d_ffn, 128);
            llma_engine::LayerMaps& m2 = e->maps2[l];
            bad |= make_tensor_map_bf16_chunks(&m2.wq, e->wq[l], HD, d.d_model, 128);
            bad |= make_tensor_map_bf16_chunks(&m2.wk, e->wk[l], HD, d.d_model, 128);
            bad |= make_tensor_map_bf16_chunks(&m2.wv, e->wv[l], HD, d.d_model, 128);
            bad |= make_tensor_map_bf16_chunks(&m2.wo, e->wo[l], d.d_model, HD, 128);
            bad |= make_tensor_map_bf16_chunks(&m2.w_down, e->w_down[l], d.d_model, d.d_ffn, 128);
            m2.w_gate = m.w_gate; m2.w_up = m.w_up;
            // one view over both matrices; if they lie too far apart for one, every pass uses the wide kernel
            if (make_tensor_map_bf16_pair(&e->gate_up_map[l].map, e->w_gate[l], e->w_up[l], d.d_ffn, d.d_model,
                                          &e->gate_up_map[l].gate_second) != 0)
                pair_ok = false;
        }
        bad |= make_tensor_map_bf16(&e->map_lm_head, e->lm_head, d.vocab, d.d_model, 128);
        bad |= make_tensor_map_bf16_chunks(&e->map_lm_head2, e->lm_head, d.vocab, d.d_model, 128);
        // the MMA shape of decoding steps is fixed per engine (by its row capacity), never per step
        e->decode_wide = e->decode_rows > 32 || !pair_ok;
        e->decode_nr = e->decode_wide ? std::max(e->decode_rows, 32) : (e->decode_rows <= 16 ? 16 : 32);
        // activation operands of the wide kernel: one box of nr rows per (buffer, use)
        auto act_maps = [&](llma_engine::ActMaps& m, int nr) {
            int bad2 = 0;
            for (int i = 0; i < 4; ++i) {
                const int box = wide_box_rows(nr, i);
                bad2 |= make_tensor_map_bf16_terms(&m.x_hat[i], e->x_hat, RC, d.d_model, box);
                bad2 |= make_tensor_map_bf16_terms(&m.attn[i], e->attn, RC, HD, box);
                bad2 |= make_tensor_map_bf16_terms(&m.h[i], e->h, RC, d.d_ffn, box);
            }
            return bad2;
        };
        bad |= act_maps(e->act_prefill, e->prefill_rows);
        if (e->decode_wide) bad |= act_maps(e->act_decode, e->decode_nr);
        if (bad) { free_engine(e); return LLMA_ERR_CONFIG; }  // misaligned weight pointer or bad shape
        CREATE_TRY(init_gemm_tcgen05());
        CREATE_TRY(init_gemm_wide());
        e->attn_chunks = (d.max_seq + kAttnChunk - 1) / kAttnChunk;
        // With far more (sequence, head, 128-position tile) triples than CTAs fit on the GPU, a CTA takes several tiles in
        // a row: fewer chunk partials, and the next tile's copies overlap the arithmetic.  A function of the engine's
        // capacity only, so a row's result does not depend on the step.  Thresholds from the one-layer grid (batch x
        // cached length): from four CTAs per resident slot on two tiles pay, from eight on four; at about one CTA per
        // slot (one sequence, 2 k positions) two tiles cost 5 % of the step.
        {
            const long long triples = (long long)d.max_batch * d.n_heads * e->attn_chunks, slots = 3LL * e->num_sms;
            e->attn_tiles = (d.kp1 <= 16 && triples >= 8 * slots) ? 4 : ((d.kp1 <= 16 && triples >= 4 * slots) ? 2 : 1);
        }
        const size_t parts = (size_t)d.n_heads * e->attn_chunks * RC;
        CREATE_TRY(dalloc(&e->attn_ws_o, parts * d.head_dim));
        CREATE_TRY(dalloc(&e->attn_ws_ml, parts * 2));
        const uint64_t kv_rows = (uint64_t)L * B * d.n_heads * d.max_seq;
        if (make_tensor_map_bf16(&e->map_kcache, e->kcache, kv_rows, d.head_dim, kAttnChunk) ||
            make_tensor_map_bf16(&e->map_vcache, e->vcache, kv_rows, d.head_dim, kAttnChunk)) {
            free_engine(e);
            return LLMA_ERR_CONFIG;
        }
        CREATE_TRY(init_attention_mma());
    }
    CREATE_TRY(cudaMallocHost((void**)&e->h_state, B * sizeof(SeqState)));
    CREATE_TRY(cudaMallocHost((void**)&e->h_rows, sizeof(RowDesc)));
    CREATE_TRY(cudaMallocHost((void**)&e->h_err, sizeof(int32_t)));
    CREATE_TRY(cudaEventCreate(&e->ev0));
    CREATE_TRY(cudaEventCreate(&e->ev1));
    CREATE_TRY(cudaDeviceSynchronize());
#undef CREATE_TRY
    *out = e;
    return LLMA_OK;
}

extern "C" int llma_destroy(llma_engine* e) {
    if (!e) return LLMA_OK;
    cudaStreamSynchronize(e->stream);
    free_engine(e);
    return LLMA_OK;
}

// Decoding entry points of the C ABI: prefill, reference upload, step, generate.
#include <algorithm>
#include <climits>
#include <cstring>
#include <vector>

#include "engine.h"

using namespace llma;

// ---- one decoder forward over the rows described by e->rows ---------------------------------
// Every kernel reads the row descriptors from device memory, so the same launch sequence
// serves any mix of rows (greedy, copy steps, prompt chunks) and can be replayed as a graph.
// When profiling is on, an event after every launch lets llma_profile_steps attribute the
// stream time between consecutive events to the kernel class just launched.
static inline void mark(llma_engine* e, int cls) {
    if (!e->prof_on) return;
    if (e->prof_n >= e->prof_ev.size()) {
        cudaEvent_t ev = nullptr;
        if (cudaEventCreate(&ev) != cudaSuccess) { e->prof_on = false; return; }
        e->prof_ev.push_back(ev);
        e->prof_cls.push_back(cls);
    }
    e->prof_cls[e->prof_n] = cls;
    cudaEventRecord(e->prof_ev[e->prof_n++], e->stream);
}

static GemmArgs gemm_args(llma_engine* e, int mode, int n_out, int n_tiles, int k_in, int tiles_per_map) {
    GemmArgs a;
    std::memset(&a, 0, sizeof(a));
    a.mode = mode; a.n_out = n_out; a.n_tiles = n_tiles; a.chunks = k_in / 64; a.tiles_per_map = tiles_per_map;
    a.rows = e->rows; a.dev_err = e->dev_err;
    a.rc = e->row_cap; a.nr = e->cur_nr;
    a.stamps = e->stamps; a.launch_id = (e->stamp_id++) % kStampLaunches;
    a.ws = e->cur_wide ? e->gemm_ws_wide : e->gemm_ws;
    a.dims = e->dims;
    return a;
}

static void run_gemm(llma_engine* e, GemmArgs& a, const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& a2,
                     const void* act, const CUtensorMap* act_map) {
    a.act = act;
    int grid = gemm_grid_for((int64_t)a.n_tiles * a.chunks, e->num_sms);
    // Prompt passes (many rows: a tile's epilogue is long): where a projection has nearly as many tiles as there are
    // SMs, one whole tile per CTA spares every tile the hand-over between the CTAs that would share it.
    if (e->cur_wide && e->cur_prompt && a.n_tiles <= e->num_sms && 5 * a.n_tiles >= 3 * e->num_sms) grid = a.n_tiles;
    if (e->cur_wide) launch_gemm_wide(e->stream, grid, true, a, a0, a1, a2, act_map);
    else launch_gemm_tcgen05(e->stream, grid, true, a, a0, a1, a2);
}

// Tensor-core path (bf16): 5 kernels per layer.  Every projection is fused with what follows
// it, and the RMSNorms are folded into the projections around them: the producer of the
// residual stream emits split(x * gain) and per-tile sums of squares, the consumer scales its
// accumulators by rsqrt(mean square + eps).
static void with_norm(llma_engine* e, GemmArgs& a) {
    a.ss_in = e->norm_ss; a.ss_tiles = (e->dims.d_model + 127) / 128;
    a.norm_dim = e->dims.d_model; a.norm_eps = e->dims.rms_eps;
}

static void enqueue_forward_tc(llma_engine* e, bool lm_head) {
    const ModelDims& d = e->dims;
    cudaStream_t st = e->stream;
    const int HD = d.hd_total, F = d.d_ffn, D = d.d_model;
    const llma_engine::ActMaps* am = e->cur_maps;
    for (int l = 0; l < d.n_layers; ++l) {
        const llma_engine::LayerMaps& m = e->cur_wide ? e->maps[l] : e->maps2[l];
        GemmArgs q = gemm_args(e, kGemmQKV, HD, 3 * HD / 128, D, HD / 128);
        with_norm(e, q);
        q.out_f32 = e->qkv; q.ld = 3 * HD; q.layer = l; q.rope_cos = e->rope_cos; q.rope_sin = e->rope_sin;
        q.kcache = (__nv_bfloat16*)e->kcache; q.vcache = (__nv_bfloat16*)e->vcache;
        run_gemm(e, q, m.wq, m.wk, m.wv, e->x_hat, am ? am->x_hat : nullptr);
        mark(e, LLMA_K_GEMM_QKV);
        AttnArgs at;
        at.dims = d; at.layer = l; at.rows = e->rows; at.qkv = e->qkv;
        at.tiles = lm_head ? e->attn_tiles : 1;  // prompt passes keep one tile per CTA
        at.chunk_pos = kAttnChunk * at.tiles;
        at.n_chunks = (d.max_seq + at.chunk_pos - 1) / at.chunk_pos;
        at.n_rows = e->cur_rows;
        at.attn_out = e->attn; at.ws_o = e->attn_ws_o; at.ws_ml = e->attn_ws_ml;
        at.dev_err = e->dev_err;
        at.stamps = e->stamps;
        at.seq_state = e->seq_state; at.early_kv = lm_head ? 1 : 0; at.prompt = lm_head ? 0 : 1;  // prompt passes: the device-side length is stale
        launch_attention_mma(st, at, e->map_kcache, e->map_vcache);
        mark(e, LLMA_K_ATTN);
        GemmArgs o = gemm_args(e, kGemmResid, D, (D + 127) / 128, HD, (D + 127) / 128);
        o.out_f32 = e->x; o.ld = D; o.gain_next = e->ffn_norm[l]; o.xs_out = e->x_hat; o.ss_out = e->norm_ss;
        run_gemm(e, o, m.wo, m.wo, m.wo, e->attn, am ? am->attn : nullptr);
        mark(e, LLMA_K_GEMM_O);
        GemmArgs gu = gemm_args(e, kGemmSwiGLU, F, (F + 63) / 64, D, (F + 63) / 64);
        with_norm(e, gu);
        gu.out_act = e->h;
        if (e->cur_wide) {
            run_gemm(e, gu, m.w_gate, m.w_up, m.w_up, e->x_hat, am->x_hat);
        } else {  // one view over both matrices; whichever lies lower in memory fills the tile's first 64 rows
            gu.gate_second = e->gate_up_map[l].gate_second;
            run_gemm(e, gu, e->gate_up_map[l].map, e->gate_up_map[l].map, e->gate_up_map[l].map, e->x_hat, nullptr);
        }
        mark(e, LLMA_K_GEMM_GATEUP);
        GemmArgs dn = gemm_args(e, kGemmResid, D, (D + 127) / 128, F, (D + 127) / 128);
        dn.out_f32 = e->x; dn.ld = D; dn.xs_out = e->x_hat; dn.ss_out = e->norm_ss;
        dn.gain_next = l + 1 < d.n_layers ? e->attn_norm[l + 1] : e->final_norm;
        run_gemm(e, dn, m.w_down, m.w_down, m.w_down, e->h, am ? am->h : nullptr);
        mark(e, LLMA_K_GEMM_DOWN);
        e->launch_counter += 6;
    }
    if (lm_head) {
        const int vt = (d.vocab + 127) / 128;
        GemmArgs lm = gemm_args(e, kGemmLmHead, d.vocab, vt, D, vt);
        with_norm(e, lm);
        lm.out_f32 = e->cfg.keep_logits ? e->logits : nullptr; lm.ld = d.vocab;
        lm.part_max = e->part_max; lm.part_idx = e->part_idx;
        const CUtensorMap& lmm = e->cur_wide ? e->map_lm_head : e->map_lm_head2;
        run_gemm(e, lm, lmm, lmm, lmm, e->x_hat, am ? am->x_hat : nullptr);
        mark(e, LLMA_K_GEMM_LMHEAD);
        e->launch_counter += 1;
    }
}

static void enqueue_forward(llma_engine* e, bool lm_head) {
    if (e->gemm_impl == LLMA_GEMM_TCGEN05) { enqueue_forward_tc(e, lm_head); return; }

    const ModelDims& d = e->dims;
    cudaStream_t st = e->stream;
    const bool b = e->bf16;
    const int HD = d.hd_total, F = d.d_ffn, D = d.d_model;
    const int nr = e->cur_rows, rc = e->row_cap;
    for (int l = 0; l < d.n_layers; ++l) {
        launch_rmsnorm(st, kActF32, nr, rc, e->rows, e->x, e->attn_norm[l], e->x_hat, D, d.rms_eps);
        mark(e, LLMA_K_NORM);
        launch_gemm_simt(st, b, e->rows, e->wq[l], (const float*)e->x_hat, e->qkv, HD, D, 3 * HD, false);
        mark(e, LLMA_K_GEMM_QKV);
        launch_gemm_simt(st, b, e->rows, e->wk[l], (const float*)e->x_hat, e->qkv + HD, HD, D, 3 * HD, false);
        mark(e, LLMA_K_GEMM_QKV);
        launch_gemm_simt(st, b, e->rows, e->wv[l], (const float*)e->x_hat, e->qkv + 2 * HD, HD, D, 3 * HD, false);
        mark(e, LLMA_K_GEMM_QKV);
        launch_qkv_post(st, b, d, l, nr, e->rows, e->qkv, e->rope_cos, e->rope_sin, e->kcache, e->vcache);
        mark(e, LLMA_K_EPILOGUE);
        launch_attention_simt(st, b, d, l, nr, e->rows, e->qkv, e->kcache, e->vcache, e->attn, kActF32);
        mark(e, LLMA_K_ATTN);
        launch_gemm_simt(st, b, e->rows, e->wo[l], (const float*)e->attn, e->x, D, HD, D, true);
        mark(e, LLMA_K_GEMM_O);
        launch_rmsnorm(st, kActF32, nr, rc, e->rows, e->x, e->ffn_norm[l], e->x_hat, D, d.rms_eps);
        mark(e, LLMA_K_NORM);
        launch_gemm_simt(st, b, e->rows, e->w_gate[l], (const float*)e->x_hat, e->gate_up, F, D, 2 * F, false);
        mark(e, LLMA_K_GEMM_GATEUP);
        launch_gemm_simt(st, b, e->rows, e->w_up[l], (const float*)e->x_hat, e->gate_up + F, F, D, 2 * F, false);
        mark(e, LLMA_K_GEMM_GATEUP);
        launch_silu_mul(st, nr, e->rows, e->gate_up, (float*)e->h, F);
        mark(e, LLMA_K_EPILOGUE);
        launch_gemm_simt(st, b, e->rows, e->w_down[l], (const float*)e->h, e->x, D, F, D, true);
        mark(e, LLMA_K_GEMM_DOWN);
        e->launch_counter += 12;
    }
    if (lm_head) {
        launch_rmsnorm(st, kActF32, nr, rc, e->rows, e->x, e->final_norm, e->x_hat, D, d.rms_eps);
        mark(e, LLMA_K_NORM);
        launch_gemm_simt(st, b, e->rows, e->lm_head, (const float*)e->x_hat, e->logits, d.vocab, D, d.vocab, false);
        mark(e, LLMA_K_GEMM_LMHEAD);
        launch_argmax(st, nr, e->rows, e->logits, d.vocab, e->out_tok);
        mark(e, LLMA_K_ARGMAX);
        e->launch_counter += 3;
    }
}

static void enqueue_embed(llma_engine* e) {
    if (e->gemm_impl == LLMA_GEMM_TCGEN05)
        launch_embed_norm(e->stream, e->dims, e->cur_rows, e->rows, e->tok_emb, e->attn_norm[0], e->x, e->x_hat,
                          e->norm_ss, e->dev_err);
    else
        launch_embed(e->stream, e->dims, e->bf16, e->cur_rows, e->rows, e->tok_emb, e->x, e->dev_err);
}

// what the launches that follow are shaped for: a decoding step or a prompt pass
static void shape_for_decode(llma_engine* e) {
    e->cur_prompt = false;
    e->cur_wide = e->decode_wide; e->cur_nr = e->decode_nr; e->cur_rows = e->decode_rows;
    e->cur_maps = e->decode_wide ? &e->act_decode : nullptr;
}
static void shape_for_prefill(llma_engine* e) {
    e->cur_prompt = true;
    e->cur_wide = e->gemm_impl == LLMA_GEMM_TCGEN05; e->cur_nr = e->prefill_rows; e->cur_rows = e->prefill_rows;
    e->cur_maps = e->cur_wide ? &e->act_prefill : nullptr;
}

// the integer kernel between forward passes: acceptance + K/V commit of the pass that has finished,
// trigger search + copy + row packing for the one that follows
static void enqueue_tail(llma_engine* e, int n, int k, bool accept, bool plan) {
    TailArgs t;
    std::memset(&t, 0, sizeof(t));
    t.dims = e->dims; t.st = e->seq_state; t.rows = e->rows; t.ref = e->ref; t.doc_start = e->doc_start;
    t.doc_end = e->doc_end; t.y = e->y; t.y_cap = e->y_cap; t.n = n; t.k = k;
    t.do_accept = accept ? 1 : 0; t.do_plan = plan ? 1 : 0;
    if (e->gemm_impl == LLMA_GEMM_TCGEN05) {
        t.part_max = e->part_max; t.part_idx = e->part_idx; t.n_tiles = (e->dims.vocab + 127) / 128;
    }
    t.out_tok = e->out_tok; t.n_rows = e->decode_rows;
    t.trace = e->trace; t.target = e->target; t.trace_cap = e->trace_cap;
    t.dev_err = e->dev_err;
    launch_step_tail(e->stream, t);
    mark(e, accept ? LLMA_K_ACCEPT : LLMA_K_PLAN);
    e->launch_counter += 1;
}

// One decoding step after its plan: embedding gather -> forward -> accept + K/V commit, and (inside
// llma_generate's graph) the plan of the next step in the same launch.
static void enqueue_step_body(llma_engine* e, int n, int k, bool plan_next) {
    shape_for_decode(e);
    e->stamp_id = 0;
    enqueue_embed(e);
    mark(e, LLMA_K_EMBED);
    e->launch_counter += 1;
    enqueue_forward(e, true);
    enqueue_tail(e, n, k, true, plan_next);
}

static int check_device_error(llma_engine* e) {
    CU_TRY(cudaMemcpyAsync(e->h_err, e->dev_err, sizeof(int32_t), cudaMemcpyDeviceToHost, e->stream));
    CU_TRY(cudaStreamSynchronize(e->stream));
    const int32_t code = *e->h_err;
    if (code == kDevErrNone) return LLMA_OK;
    CU_TRY(cudaMemsetAsync(e->dev_err, 0, sizeof(int32_t), e->stream));
    // a kernel that gave up may have left partial tiles in the hand-over slots: empty them again, so that
    // a caller who carries on after the error does not sum stale partials into later projections
    if (code == kDevErrTimeout && e->gemm_ws) {
        CU_TRY(cudaMemsetAsync(e->gemm_ws, 0xFF, e->gemm_ws_bytes, e->stream));
        CU_TRY(cudaMemsetAsync(e->gemm_ws_wide, 0xFF, e->gemm_ws_wide_bytes, e->stream));
    }
    CU_TRY(cudaStreamSynchronize(e->stream));
    if (code == kDevErrTimeout) return LLMA_ERR_DEVICE_TIMEOUT;
    if (code == kDevErrCapacity) return LLMA_ERR_CAPACITY;
    return LLMA_ERR_TOKEN_RANGE;
}

static int read_state(llma_engine* e) {
    CU_TRY(cudaMemcpyAsync(e->h_state, e->seq_state, e->dims.max_batch * sizeof(SeqState), cudaMemcpyDeviceToHost,
                           e->stream));
    CU_TRY(cudaStreamSynchronize(e->stream));
    return LLMA_OK;
}

static int write_state(llma_engine* e, int seq) {
    CU_TRY(cudaMemcpyAsync(e->seq_state + seq, e->h_state + seq, sizeof(SeqState), cudaMemcpyHostToDevice, e->stream));
    CU_TRY(cudaStreamSynchronize(e->stream));
    return LLMA_OK;
}

extern "C" int llma_prefill(llma_engine* e, int32_t seq, const int32_t* prompt, int32_t n_prompt) {
    if (!e || !prompt) return LLMA_ERR_NULL;
    const ModelDims& d = e->dims;
    if (seq < 0 || seq >= d.max_batch) return LLMA_ERR_CAPACITY;
    if (n_prompt < 1) return LLMA_ERR_ARG;
    if (n_prompt > d.max_seq) return LLMA_ERR_CAPACITY;
    for (int i = 0; i < n_prompt; ++i)
        if (prompt[i] < 0 || prompt[i] >= d.vocab) return LLMA_ERR_TOKEN_RANGE;
    int rc = read_state(e);
    if (rc) return rc;
    // push prompt[0 .. P-2] through the decoder, prefill_rows consecutive positions per pass
    const int n_cache = n_prompt - 1;
    // positions per prompt pass: at most 128 on the tensor-core path, so that the wide GEMM needs one MMA per k-slice
    const int PR = e->gemm_impl == LLMA_GEMM_TCGEN05 ? std::min(e->prefill_rows, 128) : e->prefill_rows;
    shape_for_prefill(e);
    for (int p0 = 0; p0 < n_cache; p0 += PR) {
        const int cnt = std::min(PR, n_cache - p0);
        RowDesc* R = e->h_rows;
        for (int r = 0; r < kRowCap; ++r) {
            R->tok[r] = r < cnt ? prompt[p0 + r] : 0;
            R->pos[r] = r < cnt ? p0 + r : -1;
            R->seq[r] = seq;
        }
        for (int s2 = 0; s2 < kSeqCap; ++s2) { R->seq_first[s2] = 0; R->seq_cnt[s2] = 0; R->seq_maxpos[s2] = -1; }
        R->seq_first[seq] = 0; R->seq_cnt[seq] = cnt; R->seq_maxpos[seq] = p0 + cnt - 1;
        R->rows_used = cnt;
        R->max_pos = p0 + cnt - 1;
        CU_TRY(cudaMemcpyAsync(e->rows, R, sizeof(RowDesc), cudaMemcpyHostToDevice, e->stream));
        enqueue_embed(e);
        enqueue_forward(e, false);
        CU_TRY(cudaGetLastError());
        CU_TRY(cudaStreamSynchronize(e->stream));  // h_rows is reused by the next chunk
    }
    SeqState& S = e->h_state[seq];
    const int32_t keep_ref = S.ref_len;
    std::memset(&S, 0, sizeof(S));
    S.active = 1; S.kv_len = n_cache; S.pending = prompt[n_prompt - 1]; S.ref_len = keep_ref;
    S.prompt_len = n_prompt; S.pos = -1; S.last_pos = -1; S.target_len = 0; S.done = 1;
    rc = write_state(e, seq);
    if (rc) return rc;
    e->prompt_last[seq] = prompt[n_prompt - 1];
    e->last_step_valid = false;
    return check_device_error(e);
}

extern "C" int llma_set_reference(llma_engine* e, int32_t seq, const int32_t* tokens, int32_t n_tokens,
                                  const int32_t* doc_offsets, int32_t n_docs) {
    if (!e) return LLMA_ERR_NULL;
    const ModelDims& d = e->dims;
    if (seq < 0 || seq >= d.max_batch) return LLMA_ERR_CAPACITY;
    if (n_tokens < 0) return LLMA_ERR_ARG;
    if (n_tokens > 0 && !tokens) return LLMA_ERR_NULL;
    if (n_tokens > e->cfg.max_ref) return LLMA_ERR_REF_TOO_LONG;
    std::vector<int32_t> ds((size_t)std::max(n_tokens, 1)), de((size_t)std::max(n_tokens, 1));
    if (doc_offsets) {
        if (n_docs < 1 || doc_offsets[0] != 0 || doc_offsets[n_docs] != n_tokens) return LLMA_ERR_REF_TOO_LONG;
        for (int j = 0; j < n_docs; ++j) {
            if (doc_offsets[j + 1] < doc_offsets[j]) return LLMA_ERR_REF_TOO_LONG;
            for (int i = doc_offsets[j]; i < doc_offsets[j + 1]; ++i) { ds[i] = doc_offsets[j]; de[i] = doc_offsets[j + 1]; }
        }
    } else {
        for (int i = 0; i < n_tokens; ++i) { ds[i] = 0; de[i] = n_tokens; }
    }
    for (int i = 0; i < n_tokens; ++i)
        if (tokens[i] < 0 || tokens[i] >= d.vocab) return LLMA_ERR_TOKEN_RANGE;
    if (n_tokens > 0) {
        const size_t off = (size_t)seq * d.max_ref, nb = (size_t)n_tokens * sizeof(int32_t);
        CU_TRY(cudaMemcpyAsync(e->ref + off, tokens, nb, cudaMemcpyHostToDevice, e->stream));
        CU_TRY(cudaMemcpyAsync(e->doc_start + off, ds.data(), nb, cudaMemcpyHostToDevice, e->stream));
        CU_TRY(cudaMemcpyAsync(e->doc_end + off, de.data(), nb, cudaMemcpyHostToDevice, e->stream));
    }
    CU_TRY(cudaMemcpyAsync(&e->seq_state[seq].ref_len, &n_tokens, sizeof(int32_t), cudaMemcpyHostToDevice, e->stream));
    CU_TRY(cudaStreamSynchronize(e->stream));  // the host vectors die at return
    return LLMA_OK;
}

static int check_nk(const llma_engine* e, int n, int k) {
    if (n < 1 || k < 0 || k > e->cfg.max_k) return LLMA_ERR_ARG;
    return LLMA_OK;
}

extern "C" int llma_step(llma_engine* e, int32_t n, int32_t k, int32_t* out_tokens, int32_t* n_out) {
    if (!e || !out_tokens || !n_out) return LLMA_ERR_NULL;
    int rc = check_nk(e, n, k);
    if (rc) return rc;
    const ModelDims& d = e->dims;
    rc = read_state(e);
    if (rc) return rc;
    bool any = false;
    std::vector<int32_t> y0((size_t)d.max_batch, 0);
    for (int s = 0; s < d.max_batch; ++s) {
        SeqState& S = e->h_state[s];
        y0[s] = S.y_len;
        if (!S.active) continue;
        if (S.kv_len + 1 > d.max_seq || S.y_len + 1 > e->y_cap) return LLMA_ERR_CAPACITY;
        any = true;
    }
    if (!any) return LLMA_ERR_STATE;
    for (int s = 0; s < d.max_batch; ++s) {
        SeqState& S = e->h_state[s];
        if (!S.active) continue;
        // a lone step has no output budget of its own: only the capacities bound the copy
        S.target_len = std::min(e->y_cap, S.y_len + (d.max_seq - S.kv_len));
        S.done = 0;
        rc = write_state(e, s);
        if (rc) return rc;
    }
    enqueue_tail(e, n, k, false, true);
    enqueue_step_body(e, n, k, false);
    CU_TRY(cudaGetLastError());
    rc = check_device_error(e);
    if (rc) return rc;
    rc = read_state(e);
    if (rc) return rc;
    for (int s = 0; s < d.max_batch; ++s) {
        const SeqState& S = e->h_state[s];
        const int m = S.active ? S.y_len - y0[s] : 0;
        n_out[s] = m;
        if (m > 0)
            CU_TRY(cudaMemcpy(out_tokens + (size_t)s * d.kp1, e->y + (size_t)s * e->y_cap + y0[s],
                              (size_t)m * sizeof(int32_t), cudaMemcpyDeviceToHost));
    }
    e->last_step_valid = true;
    return LLMA_OK;
}

static int get_step_graph(llma_engine* e, int n, int k, cudaGraphExec_t* out) {
    auto it = e->step_graphs.find({n, k});
    if (it != e->step_graphs.end()) { *out = it->second; return LLMA_OK; }
    cudaGraph_t g = nullptr;
    const int64_t before = e->launch_counter;
    CU_TRY(cudaStreamBeginCapture(e->stream, cudaStreamCaptureModeThreadLocal));
    enqueue_step_body(e, n, k, true);
    cudaError_t ce = cudaStreamEndCapture(e->stream, &g);
    e->launches_per_step = e->launch_counter - before;
    e->launch_counter = before;
    CU_TRY(ce);
    cudaGraphExec_t ge = nullptr;
    ce = cudaGraphInstantiate(&ge, g, 0);
    cudaGraphDestroy(g);
    CU_TRY(ce);
    e->step_graphs[{n, k}] = ge;
    *out = ge;
    return LLMA_OK;
}

extern "C" int llma_generate(llma_engine* e, int32_t max_new, int32_t n, int32_t k, int32_t* out_tokens,
                             int32_t* n_out, llma_stats* stats) {
    if (!e || !out_tokens || !n_out) return LLMA_ERR_NULL;
    int rc = check_nk(e, n, k);
    if (rc) return rc;
    if (max_new < 0) return LLMA_ERR_ARG;
    const ModelDims& d = e->dims;
    rc = read_state(e);
    if (rc) return rc;
    bool any = false;
    std::vector<SeqState> s0(e->h_state, e->h_state + d.max_batch);
    for (int s = 0; s < d.max_batch; ++s) {
        const SeqState& S = s0[s];
        if (!S.active) continue;
        if (S.kv_len + max_new > d.max_seq || S.y_len + max_new > e->y_cap) return LLMA_ERR_CAPACITY;
        any = true;
    }
    if (!any) return LLMA_ERR_STATE;
    for (int s = 0; s < d.max_batch; ++s) {
        SeqState& S = e->h_state[s];
        if (!S.active) continue;
        S.target_len = S.y_len + max_new;
        S.done = max_new == 0;
        rc = write_state(e, s);
        if (rc) return rc;
    }
    cudaGraphExec_t graph = nullptr;
    rc = get_step_graph(e, n, k, &graph);
    if (rc) return rc;

    // Each step emits between 1 and k+1 tokens per sequence, so ceil(left / (k+1)) more steps
    // can never be too many.  Launch that many back to back, look at the counters once, repeat.
    int64_t launches = 0;
    CU_TRY(cudaEventRecord(e->ev0, e->stream));
    // the first step's plan; every graph launch then ends with the plan of the step after it
    {
        const int64_t before = e->launch_counter;
        enqueue_tail(e, n, k, false, true);
        launches += e->launch_counter - before;
        e->launch_counter = before;
    }
    for (;;) {
        int left = 0;
        for (int s = 0; s < d.max_batch; ++s) {
            const SeqState& S = e->h_state[s];
            if (S.active && !S.done) left = std::max(left, S.target_len - S.y_len);
        }
        if (left <= 0) break;
        const int batch = (left + k) / (k + 1);
        for (int i = 0; i < batch; ++i) CU_TRY(cudaGraphLaunch(graph, e->stream));
        launches += (int64_t)batch * e->launches_per_step;
        rc = read_state(e);
        if (rc) return rc;
    }
    CU_TRY(cudaEventRecord(e->ev1, e->stream));
    rc = check_device_error(e);
    if (rc) return rc;

    llma_stats st;
    std::memset(&st, 0, sizeof(st));
    for (int s = 0; s < d.max_batch; ++s) {
        const SeqState& S = e->h_state[s];
        const int m = S.active ? S.y_len - s0[s].y_len : 0;
        n_out[s] = m;
        if (m > 0)
            CU_TRY(cudaMemcpy(out_tokens + (size_t)s * max_new, e->y + (size_t)s * e->y_cap + s0[s].y_len,
                              (size_t)m * sizeof(int32_t), cudaMemcpyDeviceToHost));
        if (S.active) {
            st.steps += S.steps - s0[s].steps;
            st.trigger_steps += S.trigger_steps - s0[s].trigger_steps;
            st.copied_accepted += S.copied_accepted - s0[s].copied_accepted;
            st.tokens += m;
        }
    }
    st.launches = launches;
    CU_TRY(cudaEventElapsedTime(&st.device_ms, e->ev0, e->ev1));
    if (stats) *stats = st;
    e->last_step_valid = launches > 0;
    return LLMA_OK;
}

// Replay of a given sequence of step shapes (the paper's target-guided measurement, Section 3.2 and
// Algorithm 2): the forward passes are the real ones, the trigger and acceptance decisions come from the trace.
extern "C" int llma_generate_forced(llma_engine* e, int32_t seq, const int32_t* trace, int32_t n_steps,
                                    const int32_t* target, int32_t n_target, llma_stats* stats) {
    if (!e || !trace || !target) return LLMA_ERR_NULL;
    const ModelDims& d = e->dims;
    if (seq < -1 || seq >= d.max_batch) return LLMA_ERR_CAPACITY;
    if (n_steps < 1 || n_target < 1 || n_steps > e->trace_cap) return LLMA_ERR_ARG;
    int64_t total = 0;
    for (int i = 0; i < n_steps; ++i) {
        const int r = trace[2 * i], m = trace[2 * i + 1];
        if (r < 1 || r > d.kp1 || m < 1 || m > r) return LLMA_ERR_ARG;
        total += m;
    }
    if (total != n_target) return LLMA_ERR_ARG;
    for (int i = 0; i < n_target; ++i)
        if (target[i] < 0 || target[i] >= d.vocab) return LLMA_ERR_TOKEN_RANGE;
    int rc = read_state(e);
    if (rc) return rc;
    // the sequences that replay: the given one, or (seq = -1) every prefilled one; all others must be at rest
    std::vector<int> who;
    for (int s = 0; s < d.max_batch; ++s) {
        const SeqState& S = e->h_state[s];
        if (s == seq || (seq < 0 && S.active)) who.push_back(s);
        else if (S.active && !S.done) return LLMA_ERR_STATE;
    }
    if (who.empty()) return LLMA_ERR_STATE;
    std::vector<SeqState> s0(e->h_state, e->h_state + d.max_batch);
    for (int s : who) {
        if (!s0[s].active) return LLMA_ERR_STATE;
        if (s0[s].kv_len + n_target > d.max_seq || s0[s].y_len + n_target > e->y_cap) return LLMA_ERR_CAPACITY;
    }
    for (int s : who) {
        CU_TRY(cudaMemcpyAsync(e->trace + (size_t)s * e->trace_cap * 2, trace, (size_t)n_steps * 2 * sizeof(int32_t),
                               cudaMemcpyHostToDevice, e->stream));
        CU_TRY(cudaMemcpyAsync(e->target + (size_t)s * e->y_cap + s0[s].y_len, target, (size_t)n_target * sizeof(int32_t),
                               cudaMemcpyHostToDevice, e->stream));
        SeqState& S = e->h_state[s];
        S.target_len = S.y_len + n_target; S.done = 0; S.forced_rows = 1; S.forced_emit = 1; S.trace_step = 0;
        rc = write_state(e, s);  // synchronises: the host arrays may go after this
        if (rc) return rc;
    }
    cudaGraphExec_t graph = nullptr;
    rc = get_step_graph(e, 1, 0, &graph);
    if (rc) return rc;
    CU_TRY(cudaEventRecord(e->ev0, e->stream));
    const int64_t before = e->launch_counter;
    enqueue_tail(e, 1, 0, false, true);
    const int64_t tail_launches = e->launch_counter - before;
    e->launch_counter = before;
    for (int i = 0; i < n_steps; ++i) CU_TRY(cudaGraphLaunch(graph, e->stream));
    CU_TRY(cudaEventRecord(e->ev1, e->stream));
    rc = check_device_error(e);
    if (rc) return rc;
    rc = read_state(e);
    if (rc) return rc;
    llma_stats st;
    std::memset(&st, 0, sizeof(st));
    bool complete = true;
    for (int s : who) {
        SeqState& T = e->h_state[s];
        st.steps += T.steps - s0[s].steps; st.trigger_steps += T.trigger_steps - s0[s].trigger_steps;
        st.copied_accepted += T.copied_accepted - s0[s].copied_accepted; st.tokens += T.y_len - s0[s].y_len;
        complete = complete && T.y_len - s0[s].y_len == n_target;
        T.forced_rows = 0; T.forced_emit = 0; T.trace_step = 0;
        rc = write_state(e, s);
        if (rc) return rc;
    }
    st.launches = tail_launches + (int64_t)n_steps * e->launches_per_step;
    CU_TRY(cudaEventElapsedTime(&st.device_ms, e->ev0, e->ev1));
    if (stats) *stats = st;
    e->last_step_valid = false;
    return complete ? LLMA_OK : LLMA_ERR_STATE;
}

extern "C" int llma_debug_set_device_error(llma_engine* e, int32_t code) {
    if (!e) return LLMA_ERR_NULL;
    if (code < kDevErrNone || code > kDevErrToken) return LLMA_ERR_ARG;
    CU_TRY(cudaMemcpyAsync(e->dev_err, &code, sizeof(int32_t), cudaMemcpyHostToDevice, e->stream));
    CU_TRY(cudaStreamSynchronize(e->stream));
    return LLMA_OK;
}

extern "C" int llma_profile_steps(llma_engine* e, int32_t n, int32_t k, int32_t steps, llma_profile* out) {
    if (!e || !out) return LLMA_ERR_NULL;
    int rc = check_nk(e, n, k);
    if (rc) return rc;
    if (steps < 1) return LLMA_ERR_ARG;
    std::memset(out, 0, sizeof(*out));
    std::vector<int32_t> toks((size_t)e->dims.max_batch * e->dims.kp1), cnt((size_t)e->dims.max_batch);
    for (int i = 0; i < steps; ++i) {
        // same state handling as llma_step, but the launches are bracketed by events
        rc = read_state(e);
        if (rc) return rc;
        bool any = false;
        for (int s = 0; s < e->dims.max_batch; ++s) {
            SeqState& S = e->h_state[s];
            if (!S.active) continue;
            if (S.kv_len + 1 > e->dims.max_seq) return LLMA_ERR_CAPACITY;
            S.target_len = std::min(e->y_cap, S.y_len + (e->dims.max_seq - S.kv_len));
            S.done = 0;
            rc = write_state(e, s);
            if (rc) return rc;
            any = true;
        }
        if (!any) return LLMA_ERR_STATE;
        e->prof_on = true;
        e->prof_n = 0;
        mark(e, -1);
        enqueue_tail(e, n, k, false, true);
        enqueue_step_body(e, n, k, false);
        e->prof_on = false;
        CU_TRY(cudaGetLastError());
        rc = check_device_error(e);
        if (rc) return rc;
        for (size_t j = 1; j < e->prof_n; ++j) {
            float ms = 0.f;
            CU_TRY(cudaEventElapsedTime(&ms, e->prof_ev[j - 1], e->prof_ev[j]));
            const int c = e->prof_cls[j];
            if (c >= 0 && c < LLMA_K_COUNT) { out->ms[c] += ms; out->launches[c] += 1; }
            out->total_ms += ms;
        }
        out->steps += 1;
    }
    e->last_step_valid = true;
    return LLMA_OK;
}

// Small state-management and inspection entry points of the C ABI.
#include <algorithm>
#include <cstring>
#include <vector>

#include "engine.h"

using namespace llma;

static int fetch_state(llma_engine* e) {
    CU_TRY(cudaMemcpyAsync(e->h_state, e->seq_state, e->dims.max_batch * sizeof(SeqState), cudaMemcpyDeviceToHost,
                           e->stream));
    CU_TRY(cudaStreamSynchronize(e->stream));
    return LLMA_OK;
}

static int store_state(llma_engine* e, int seq) {
    CU_TRY(cudaMemcpyAsync(e->seq_state + seq, e->h_state + seq, sizeof(SeqState), cudaMemcpyHostToDevice, e->stream));
    CU_TRY(cudaStreamSynchronize(e->stream));
    return LLMA_OK;
}

extern "C" int llma_rewind(llma_engine* e, int32_t seq) {
    if (!e) return LLMA_ERR_NULL;
    if (seq < 0 || seq >= e->dims.max_batch) return LLMA_ERR_CAPACITY;
    int rc = fetch_state(e);
    if (rc) return rc;
    SeqState& S = e->h_state[seq];
    if (!S.active) return LLMA_ERR_STATE;
    const int32_t ref_len = S.ref_len, plen = S.prompt_len;
    const int32_t last_tok = e->prompt_last[seq];  // kept on the host by llma_prefill
    const int32_t k_min = S.k_min, k_start = S.k_start;
    std::memset(&S, 0, sizeof(S));
    S.k_min = k_min; S.k_start = k_start; S.k_cur = k_start;
    S.active = 1; S.kv_len = plen - 1; S.pending = last_tok; S.ref_len = ref_len; S.prompt_len = plen;
    S.pos = -1; S.last_pos = -1; S.done = 1;
    e->last_step_valid = false;
    return store_state(e, seq);
}

extern "C" int llma_set_adaptive_k(llma_engine* e, int32_t seq, int32_t k_min, int32_t k_start) {
    if (!e) return LLMA_ERR_NULL;
    if (seq < 0 || seq >= e->dims.max_batch) return LLMA_ERR_CAPACITY;
    const bool off = k_min == 0 && k_start == 0;
    if (!off && (k_min < 1 || k_start < k_min || k_start > e->dims.kp1 - 1)) return LLMA_ERR_ARG;
    int rc = fetch_state(e);
    if (rc) return rc;
    SeqState& S = e->h_state[seq];
    S.k_min = k_min; S.k_start = k_start; S.k_cur = k_start;
    return store_state(e, seq);
}

extern "C" int llma_reset(llma_engine* e, int32_t seq) {
    if (!e) return LLMA_ERR_NULL;
    if (seq < 0 || seq >= e->dims.max_batch) return LLMA_ERR_CAPACITY;
    int rc = fetch_state(e);
    if (rc) return rc;
    std::memset(&e->h_state[seq], 0, sizeof(SeqState));
    e->h_state[seq].pos = -1; e->h_state[seq].last_pos = -1;
    e->last_step_valid = false;
    return store_state(e, seq);
}

extern "C" int llma_last_step_info(llma_engine* e, llma_step_info* info) {
    if (!e || !info) return LLMA_ERR_NULL;
    int rc = fetch_state(e);
    if (rc) return rc;
    for (int s = 0; s < e->dims.max_batch; ++s) {
        const SeqState& S = e->h_state[s];
        info[s].pos = S.last_pos; info[s].k_eff = S.last_k_eff;
        info[s].accepted = S.last_accepted; info[s].emitted = S.last_emitted;
    }
    return LLMA_OK;
}

extern "C" int llma_debug_logits(llma_engine* e, float* out) {
    if (!e || !out) return LLMA_ERR_NULL;
    if (!e->cfg.keep_logits || !e->last_step_valid) return LLMA_ERR_STATE;
    CU_TRY(cudaStreamSynchronize(e->stream));
    // the rows of a step are packed; hand them out in the documented per-sequence slots
    CU_TRY(cudaMemcpy(e->h_rows, e->rows, sizeof(RowDesc), cudaMemcpyDeviceToHost));
    const size_t V = (size_t)e->dims.vocab;
    for (int s = 0; s < e->dims.max_batch; ++s) {
        const int first = e->h_rows->seq_first[s], cnt = std::min(e->h_rows->seq_cnt[s], e->dims.kp1);
        if (cnt <= 0 || first < 0 || first + cnt > e->row_cap) continue;
        CU_TRY(cudaMemcpy(out + (size_t)s * e->dims.kp1 * V, e->logits + (size_t)first * V, (size_t)cnt * V * sizeof(float),
                          cudaMemcpyDeviceToHost));
    }
    return LLMA_OK;
}

extern "C" int llma_debug_kv_row(llma_engine* e, int32_t layer, int32_t seq, int32_t pos, int32_t which, float* out) {
    if (!e || !out) return LLMA_ERR_NULL;
    const ModelDims& d = e->dims;
    if (layer < 0 || layer >= d.n_layers || seq < 0 || seq >= d.max_batch || pos < 0 || pos >= d.max_seq ||
        (which != 0 && which != 1))
        return LLMA_ERR_ARG;
    CU_TRY(cudaStreamSynchronize(e->stream));
    const char* base = (const char*)(which ? e->vcache : e->kcache);
    const size_t es = e->bf16 ? 2 : 4;
    // one strided copy: the row of every head (heads are max_seq rows apart in the cache)
    std::vector<unsigned char> tmp((size_t)d.n_heads * d.head_dim * es);
    const size_t off = (size_t)kv_row_index(d, layer, seq, 0, pos) * d.head_dim * es;
    CU_TRY(cudaMemcpy2D(tmp.data(), (size_t)d.head_dim * es, base + off, (size_t)d.max_seq * d.head_dim * es,
                        (size_t)d.head_dim * es, (size_t)d.n_heads, cudaMemcpyDeviceToHost));
    const size_t n = (size_t)d.n_heads * d.head_dim;
    for (size_t i = 0; i < n; ++i) {
        float v;
        if (e->bf16) {
            uint32_t u = (uint32_t)(((const uint16_t*)tmp.data())[i]) << 16;
            std::memcpy(&v, &u, 4);
        } else {
            v = ((const float*)tmp.data())[i];
        }
        out[i] = v;
    }
    return LLMA_OK;
}

extern "C" int llma_kv_len(llma_engine* e, int32_t seq) {
    if (!e) return LLMA_ERR_NULL;
    if (seq < 0 || seq >= e->dims.max_batch) return LLMA_ERR_CAPACITY;
    int rc = fetch_state(e);
    if (rc) return rc;
    if (!e->h_state[seq].active) return LLMA_ERR_STATE;
    return e->h_state[seq].kv_len;
}

extern "C" int llma_debug_timeline(llma_engine* e, int32_t clear, unsigned long long* out) {
    if (!e) return LLMA_ERR_NULL;
    if (!e->stamps) return LLMA_ERR_STATE;  // not a measurement build
    const size_t n = (size_t)kStampLaunches * kStampSlots * 8;
    CU_TRY(cudaStreamSynchronize(e->stream));
    if (out) CU_TRY(cudaMemcpy(out, e->stamps, n * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
    if (clear) {  // even words of the (min, max) blocks start at all-ones, everything else at zero
        std::vector<unsigned long long> h(n, 0ull);
        for (int l = 300; l < kStampLaunches; ++l)
            for (int j = 0; j < 8; j += 2) h[(size_t)l * kStampSlots * 8 + j] = ~0ull;
        CU_TRY(cudaMemcpy(e->stamps, h.data(), n * sizeof(unsigned long long), cudaMemcpyHostToDevice));
    }
    return LLMA_OK;
}

extern "C" int llma_debug_attention_tiles(llma_engine* e) {
    if (!e) return LLMA_ERR_NULL;
    return e->attn_tiles;
}

extern "C" int llma_row_capacity(llma_engine* e) {
    if (!e) return LLMA_ERR_NULL;
    return e->row_cap;
}

extern "C" int llma_gemm_impl(llma_engine* e) {
    if (!e) return LLMA_ERR_NULL;
    return e->gemm_impl;
}

extern "C" int llma_debug_buffer(llma_engine* e, int32_t which, float* out, int64_t count) {
    if (!e || !out) return LLMA_ERR_NULL;
    const ModelDims& d = e->dims;
    const int64_t cols = which == 0 ? d.d_model : which == 1 ? 3 * (int64_t)d.hd_total : which == 2 ? d.hd_total
                       : which == 3 ? d.d_ffn : -1;
    if (cols < 0 || count != cols * e->row_cap) return LLMA_ERR_ARG;
    CU_TRY(cudaStreamSynchronize(e->stream));
    if (which <= 1) {
        CU_TRY(cudaMemcpy(out, which == 0 ? e->x : e->qkv, (size_t)count * sizeof(float), cudaMemcpyDeviceToHost));
        return LLMA_OK;
    }
    const void* src = which == 2 ? e->attn : e->h;
    if (e->gemm_impl != LLMA_GEMM_TCGEN05) {  // fp32 [32][K]
        CU_TRY(cudaMemcpy(out, src, (size_t)count * sizeof(float), cudaMemcpyDeviceToHost));
        return LLMA_OK;
    }
    std::vector<uint16_t> raw((size_t)2 * count);  // split bf16 [2 rc][K]: hi rows then lo rows
    CU_TRY(cudaMemcpy(raw.data(), src, raw.size() * 2, cudaMemcpyDeviceToHost));
    for (int64_t i = 0; i < count; ++i) {
        uint32_t h = (uint32_t)raw[i] << 16, l = (uint32_t)raw[count + i] << 16;
        float fh, fl;
        std::memcpy(&fh, &h, 4); std::memcpy(&fl, &l, 4);
        out[i] = fh + fl;
    }
    return LLMA_OK;
}

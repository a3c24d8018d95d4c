// Integer side of an LLMA decoding step: trigger search + copy (Section 2.2 of the paper,
// Algorithm 1's match and copy steps), embedding gather, and acceptance + K/V
// commit (Algorithm 1's acceptance loop).  All results here are exact integer work.
#include "kernels.h"

namespace llma {

// --------------------------------------------------------------------------------------
// plan: one CTA per sequence.
//   Trigger: among reference positions `pos` (inside one document, with at least one token
//   after it) whose preceding n tokens equal the last n generated tokens, pick the one whose
//   agreement with the generated text extends furthest backwards; ties go to the smallest
//   position.  Copy: k_eff = min(k, tokens left in the document, tokens still to emit - 1,
//   K/V rows left - 1).  Rows of the step: [pending, ref[pos], ..., ref[pos+k_eff-1]] at
//   positions kv_len .. kv_len+k_eff.
// --------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) plan_kernel(ModelDims dims, SeqState* __restrict__ st,
                                                   RowDesc* __restrict__ rows, const int32_t* __restrict__ ref,
                                                   const int32_t* __restrict__ doc_start,
                                                   const int32_t* __restrict__ doc_end,
                                                   const int32_t* __restrict__ y, int32_t y_cap, int32_t n,
                                                   int32_t k, int32_t* __restrict__ dev_err) {
    pdl_trigger();
    pdl_wait();
    const int s = blockIdx.x;
    SeqState& S = st[s];
    __shared__ unsigned long long best;  // (ext << 32) | (0x7fffffff - pos): max = longest, then earliest
    if (threadIdx.x == 0) best = 0ull;
    __syncthreads();

    const bool live = S.active && !S.done && S.y_len < S.target_len;
    const int ylen = S.y_len;
    const int ref_len = S.ref_len;
    const int* ys = y + (int64_t)s * y_cap;
    const int* rs = ref + (int64_t)s * dims.max_ref;
    const int* ds = doc_start + (int64_t)s * dims.max_ref;
    const int* de = doc_end + (int64_t)s * dims.max_ref;

    if (live && k > 0 && n >= 1 && ylen >= n && ref_len > 0) {
        const int last = ys[ylen - 1];
        for (int pos = threadIdx.x + 1; pos < ref_len; pos += blockDim.x) {
            // candidate: ref[pos-1] is the last matched token; pos must stay inside its document
            if (rs[pos - 1] != last) continue;
            const int s0 = ds[pos - 1];
            if (pos >= de[pos - 1]) continue;  // nothing follows inside this document
            int t = 1;
            while (t < ylen && pos - t - 1 >= s0 && rs[pos - t - 1] == ys[ylen - t - 1]) ++t;
            if (t >= n) {
                unsigned long long key = ((unsigned long long)(unsigned)t << 32) | (unsigned)(0x7fffffff - pos);
                atomicMax(&best, key);
            }
        }
    }
    __syncthreads();

    if (threadIdx.x == 0) {
        int pos = -1, k_eff = 0;
        if (live) {
            if (best != 0ull) {
                pos = 0x7fffffff - (int)(unsigned)(best & 0xffffffffull);
                int room_doc = de[pos - 1] - pos;
                int room_out = S.target_len - ylen - 1;
                int room_kv = dims.max_seq - S.kv_len - 1;
                k_eff = min(min(k, room_doc), min(room_out, room_kv));
                if (k_eff <= 0) { k_eff = 0; pos = -1; }
            }
            if (S.kv_len + k_eff + 1 > dims.max_seq) {  // no room even for the pending token
                atomicExch(dev_err, kDevErrCapacity);
                S.nrows = 0; S.pos = -1; S.k_eff = 0;
            } else {
                S.pos = pos; S.k_eff = k_eff; S.nrows = k_eff + 1;
            }
        } else {
            S.pos = -1; S.k_eff = 0; S.nrows = 0;
        }
    }
    __syncthreads();

    // row descriptors of this sequence's slot
    const int row0 = s * dims.kp1;
    const int nrows = S.nrows, p0 = S.pos, L = S.kv_len, pend = S.pending;
    for (int j = threadIdx.x; j < dims.kp1; j += blockDim.x) {
        const int r = row0 + j;
        if (j < nrows) {
            rows->tok[r] = (j == 0) ? pend : rs[p0 + j - 1];
            rows->pos[r] = L + j;
        } else {
            rows->tok[r] = 0;
            rows->pos[r] = -1;
        }
        rows->seq[r] = s;
    }
}

// rows_used / max_pos after all sequences are planned (one small CTA)
__global__ void finish_plan_kernel(ModelDims dims, const SeqState* __restrict__ st, RowDesc* __restrict__ rows) {
    pdl_trigger();
    pdl_wait();
    if (threadIdx.x == 0) {
        int used = 0, mp = -1;
        for (int s = 0; s < dims.max_batch; ++s) {
            rows->seq_first[s] = s * dims.kp1;
            rows->seq_cnt[s] = st[s].nrows;
            rows->seq_maxpos[s] = st[s].nrows > 0 ? st[s].kv_len + st[s].nrows - 1 : -1;
            if (st[s].nrows > 0) {
                used = s * dims.kp1 + st[s].nrows;
                mp = max(mp, st[s].kv_len + st[s].nrows - 1);
            }
        }
        for (int r = dims.max_batch * dims.kp1; r < kMaxRows; ++r) {
            rows->pos[r] = -1; rows->tok[r] = 0; rows->seq[r] = 0;
        }
        rows->rows_used = used;
        rows->max_pos = mp;
    }
}

// --------------------------------------------------------------------------------------
// embedding gather: x[r, :] = tok_emb[tok[r], :] as fp32 (zero for unused rows)
// --------------------------------------------------------------------------------------
template <typename T>
__global__ void embed_kernel(ModelDims dims, const RowDesc* __restrict__ rows, const T* __restrict__ emb,
                             float* __restrict__ x, int32_t* __restrict__ dev_err) {
    pdl_trigger();
    pdl_wait();
    const int r = blockIdx.x;
    const int d = dims.d_model;
    float* xr = x + (int64_t)r * d;
    const int tok = rows->tok[r];
    const bool used = rows->pos[r] >= 0;
    const bool ok = used && tok >= 0 && tok < dims.vocab;
    if (used && !ok && threadIdx.x == 0) atomicExch(dev_err, kDevErrToken);
    const T* er = emb + (int64_t)(ok ? tok : 0) * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) xr[i] = ok ? to_f32<T>(er[i]) : 0.f;
}

// Embedding gather for the tensor-core path, with the first RMSNorm folded in: besides x it
// writes xs = split(x * gain) and, per 128-column tile, each row's sum of squares (the
// projections multiply by rsqrt(mean square + eps) afterwards).  One CTA of 128 threads per (row, 128-column tile).
__global__ void __launch_bounds__(128) embed_norm_kernel(ModelDims dims, const RowDesc* __restrict__ rows,
                                                         const __nv_bfloat16* __restrict__ emb,
                                                         const float* __restrict__ gain, float* __restrict__ x,
                                                         void* __restrict__ xs, float* __restrict__ ss,
                                                         int32_t* __restrict__ dev_err) {
    pdl_trigger();
    pdl_wait();
    const int r = blockIdx.x, t = blockIdx.y, d = dims.d_model;
    const int tok = rows->tok[r];
    const bool used = rows->pos[r] >= 0;
    const bool ok = used && tok >= 0 && tok < dims.vocab;
    if (used && !ok && t == 0 && threadIdx.x == 0) atomicExch(dev_err, kDevErrToken);
    const __nv_bfloat16* er = emb + (int64_t)(ok ? tok : 0) * d;
    __shared__ float red[4];
    const int col = t * 128 + threadIdx.x;
    float v = 0.f;
    if (col < d) {
        v = ok ? __bfloat162float(er[col]) : 0.f;
        x[(int64_t)r * d + col] = v;
        store_act(xs, kActSplit, r, col, d, v * gain[col]);
    }
    float sq = v * v;
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0) ss[(int64_t)t * 32 + r] = ((red[0] + red[1]) + red[2]) + red[3];
}

// --------------------------------------------------------------------------------------
// accept: o_0 is always kept; o_{i+1} is kept while o_i equals the copied token d_{pos+i}.
// Appends the kept outputs to y, advances kv_len past the rows whose inputs were valid
// (rows after them stay in the cache as garbage and are overwritten by later steps),
// sets the next pending token, updates the decode statistics.
// --------------------------------------------------------------------------------------
__global__ void accept_kernel(ModelDims dims, SeqState* __restrict__ st, const int32_t* __restrict__ ref,
                              const int32_t* __restrict__ out_tok, int32_t* __restrict__ y, int32_t y_cap) {
    pdl_trigger();
    pdl_wait();
    const int s = blockIdx.x;
    if (threadIdx.x != 0) return;
    SeqState& S = st[s];
    if (S.nrows <= 0) {
        S.last_pos = -1; S.last_k_eff = 0; S.last_accepted = 0; S.last_emitted = 0;
        return;
    }
    const int* rs = ref + (int64_t)s * dims.max_ref;
    const int* o = out_tok + s * dims.kp1;
    int a = 0;
    while (a < S.k_eff && o[a] == rs[S.pos + a]) ++a;
    int m = a + 1;
    int done = 0;
    if (dims.eos_id >= 0) {
        for (int j = 0; j < m; ++j)
            if (o[j] == dims.eos_id) { m = j + 1; done = 1; break; }
    }
    int* ys = y + (int64_t)s * y_cap;
    for (int j = 0; j < m; ++j) ys[S.y_len + j] = o[j];
    S.y_len += m;
    S.kv_len += m;
    S.pending = o[m - 1];
    S.steps += 1;
    S.trigger_steps += (S.k_eff > 0);
    S.copied_accepted += m - 1;
    S.last_pos = S.pos; S.last_k_eff = S.k_eff; S.last_accepted = m - 1; S.last_emitted = m;
    if (S.y_len >= S.target_len) done = 1;
    S.done = done;
    S.nrows = 0;
}

// ---- launchers -----------------------------------------------------------------------
void launch_plan(cudaStream_t st, const ModelDims& dims, SeqState* seq, RowDesc* rows, const int32_t* ref,
                 const int32_t* doc_start, const int32_t* doc_end, const int32_t* y, int32_t y_cap, int32_t n,
                 int32_t k, int32_t* dev_err) {
    launch_pdl(st, true, dim3(dims.max_batch), dim3(256), 0, plan_kernel, dims, seq, rows, ref, doc_start, doc_end, y, y_cap, n, k, dev_err);
    launch_pdl(st, true, dim3(1), dim3(32), 0, finish_plan_kernel, dims, seq, rows);
}

void launch_embed(cudaStream_t st, const ModelDims& dims, bool bf16, const RowDesc* rows, const void* emb, float* x,
                  int32_t* dev_err) {
    if (bf16)
        launch_pdl(st, true, dim3(kMaxRows), dim3(256), 0, embed_kernel<__nv_bfloat16>, dims, rows, (const __nv_bfloat16*)emb, x, dev_err);
    else
        launch_pdl(st, true, dim3(kMaxRows), dim3(256), 0, embed_kernel<float>, dims, rows, (const float*)emb, x, dev_err);
}

void launch_embed_norm(cudaStream_t st, const ModelDims& dims, const RowDesc* rows, const void* emb, const float* gain,
                       float* x, void* xs, float* ss, int32_t* dev_err) {
    launch_pdl(st, true, dim3(kMaxRows, (dims.d_model + 127) / 128), dim3(128), 0, embed_norm_kernel, dims, rows, (const __nv_bfloat16*)emb, gain, x,
               xs, ss, dev_err);
}

void launch_accept(cudaStream_t st, const ModelDims& dims, SeqState* seq, const int32_t* ref, const int32_t* out_tok,
                   int32_t* y, int32_t y_cap) {
    launch_pdl(st, true, dim3(dims.max_batch), dim3(32), 0, accept_kernel, dims, seq, ref, out_tok, y, y_cap);
}

}  // namespace llma

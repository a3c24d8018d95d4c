// Integer side of an LLMA decoding step: trigger search + copy (Section 2.2 of the paper,
// Algorithm 1's match and copy steps), embedding gather, and acceptance + K/V
// commit (Algorithm 1's acceptance loop).  All results here are exact integer work.
#include "kernels.h"

namespace llma {

// --------------------------------------------------------------------------------------
// step_tail_kernel: ONE CTA does the integer work between two forward passes, for all sequences:
//
//   accept (Algorithm 1's acceptance loop, when a forward pass has just finished)
//     final argmax of every row over the LM head's per-tile partials (tensor-core path);
//     o_0 is always kept, o_{i+1} is kept while o_i equals the copied token d_{pos+i};
//     the kept outputs are appended to y, kv_len advances past the rows whose inputs were
//     valid (later rows stay in the cache as garbage and are overwritten by later steps),
//     the last kept output becomes the pending input, statistics are updated.
//   plan (Section 2.2: trigger and copy, when a forward pass follows)
//     one warp per sequence: among reference positions `pos` (inside one document, with at
//     least one token after it) whose preceding n tokens equal the last n generated tokens,
//     pick the one whose agreement with the generated text extends furthest backwards; ties go
//     to the smallest position.  k_eff = min(k, tokens left in the document, tokens still to
//     emit - 1, K/V rows left - 1).  Rows of the step: [pending, ref[pos], ..., ref[pos+k_eff-1]]
//     at positions kv_len .. kv_len+k_eff; the rows of all sequences are packed back to back.
//
// A sequence in replay mode (forced_rows > 0 in its state) skips both decisions: the shapes come
// from a trace and the tokens from a target text (Algorithm 2's use in Section 3.2).
// --------------------------------------------------------------------------------------
constexpr int kTailThreads = 1024;

__global__ void __launch_bounds__(kTailThreads) step_tail_kernel(const TailArgs a) {
    pdl_trigger();
    pdl_wait();
    const ModelDims& dims = a.dims;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = kTailThreads / 32;
    const int B = dims.max_batch;
    __shared__ int s_first[kSeqCap];

    if (a.do_accept) {
        // ---- final argmax of every row in use (lowest index on ties) -----------------------------------
        if (a.part_max) {
            const int rows_used = a.rows->rows_used;
            for (int r = warp; r < rows_used; r += n_warps) {
                float bv = -INFINITY; int bi = 0x7fffffff;
                for (int t = lane; t < a.n_tiles; t += 32) {
                    const float v = __ldcg(&a.part_max[(int64_t)t * dims.row_cap + r]);
                    const int i = __ldcg(&a.part_idx[(int64_t)t * dims.row_cap + r]);
                    if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
                }
                for (int o = 16; o > 0; o >>= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
                }
                if (lane == 0) a.out_tok[r] = bi;
            }
            __syncthreads();
        }
        // ---- acceptance + commit, one thread per sequence ------------------------------------------------
        for (int s = threadIdx.x; s < B; s += kTailThreads) {
            SeqState& S = a.st[s];
            if (S.nrows <= 0) {
                S.last_pos = -1; S.last_k_eff = 0; S.last_accepted = 0; S.last_emitted = 0;
                continue;
            }
            const int* rs = a.ref + (int64_t)s * dims.max_ref;
            const int* o = a.out_tok + a.rows->seq_first[s];
            int* ys = a.y + (int64_t)s * a.y_cap;
            int m, done = 0;
            if (S.forced_rows > 0) {
                // replay: the trace says how many tokens the step emits, the target text which ones
                m = S.forced_emit;
                const int* tg = a.target + (int64_t)s * a.y_cap;
                for (int j = 0; j < m; ++j) ys[S.y_len + j] = tg[S.y_len + j];
                S.pending = tg[S.y_len + m - 1];
            } else {
                int acc = 0;
                while (acc < S.k_eff && o[acc] == rs[S.pos + acc]) ++acc;
                m = acc + 1;
                if (dims.eos_id >= 0) {
                    for (int j = 0; j < m; ++j)
                        if (o[j] == dims.eos_id) { m = j + 1; done = 1; break; }
                }
                for (int j = 0; j < m; ++j) ys[S.y_len + j] = o[j];
                S.pending = o[m - 1];
            }
            S.y_len += m;
            S.kv_len += m;
            S.steps += 1;
            S.trigger_steps += (S.k_eff > 0);
            S.copied_accepted += m - 1;
            S.last_pos = S.pos; S.last_k_eff = S.k_eff; S.last_accepted = m - 1; S.last_emitted = m;
            if (S.y_len >= S.target_len) done = 1;
            S.done = done;
            S.nrows = 0;
        }
        __syncthreads();
    }
    if (!a.do_plan) return;

    // ---- trigger search + copy length, one warp per sequence ---------------------------------------------
    for (int s = warp; s < B; s += n_warps) {
        SeqState& S = a.st[s];
        const bool live = S.active && !S.done && S.y_len < S.target_len;
        const int ylen = S.y_len, ref_len = S.ref_len;
        const int* ys = a.y + (int64_t)s * a.y_cap;
        const int* rs = a.ref + (int64_t)s * dims.max_ref;
        const int* ds = a.doc_start + (int64_t)s * dims.max_ref;
        const int* de = a.doc_end + (int64_t)s * dims.max_ref;
        int pos = -1, k_eff = 0, nrows = 0;
        if (live && a.trace && S.forced_rows != 0) {
            // replay: shape of step number S.steps from the trace
            const int step = S.trace_step;
            int fr = 1, fe = 1;
            if (step < a.trace_cap) {
                fr = a.trace[((int64_t)s * a.trace_cap + step) * 2];
                fe = a.trace[((int64_t)s * a.trace_cap + step) * 2 + 1];
            }
            fr = max(1, min(fr, min(dims.kp1, dims.max_seq - S.kv_len)));
            fe = max(1, min(fe, min(fr, S.target_len - ylen)));
            nrows = fr; k_eff = fr - 1;
            if (lane == 0) { S.forced_rows = fr; S.forced_emit = fe; S.trace_step = step + 1; }
        } else if (live) {
            // (ext << 32) | (0x7fffffff - pos): the maximum is the longest agreement, then the earliest position
            unsigned long long best = 0ull;
            if (a.k > 0 && a.n >= 1 && ylen >= a.n && ref_len > 0) {
                const int last = ys[ylen - 1];
                for (int p0 = 1; p0 < ref_len; p0 += 32) {
                    const int p = p0 + lane;
                    // candidate: ref[p-1] is the last matched token; p must stay inside its document
                    if (p < ref_len && rs[p - 1] == last && p < de[p - 1]) {
                        const int s0 = ds[p - 1];
                        int t = 1;
                        while (t < ylen && p - t - 1 >= s0 && rs[p - t - 1] == ys[ylen - t - 1]) ++t;
                        if (t >= a.n) {
                            const unsigned long long key = ((unsigned long long)(unsigned)t << 32) | (unsigned)(0x7fffffff - p);
                            best = key > best ? key : best;
                        }
                    }
                }
                for (int o = 16; o > 0; o >>= 1) {
                    const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
                    best = other > best ? other : best;
                }
            }
            if (best != 0ull) {
                pos = 0x7fffffff - (int)(unsigned)(best & 0xffffffffull);
                const int room_doc = de[pos - 1] - pos;
                const int room_out = S.target_len - ylen - 1;
                const int room_kv = dims.max_seq - S.kv_len - 1;
                k_eff = min(min(a.k, room_doc), min(room_out, room_kv));
                if (k_eff <= 0) { k_eff = 0; pos = -1; }
            }
            nrows = k_eff + 1;
            if (S.kv_len + nrows > dims.max_seq) {  // no room even for the pending token
                if (lane == 0) atomicExch(a.dev_err, kDevErrCapacity);
                nrows = 0; pos = -1; k_eff = 0;
            }
        }
        if (lane == 0) { S.pos = pos; S.k_eff = k_eff; S.nrows = nrows; }
    }
    __syncthreads();

    // ---- pack the rows: sequence s owns rows first[s] .. first[s] + nrows - 1 -----------------------------
    if (threadIdx.x == 0) {
        int used = 0, mp = -1;
        for (int s = 0; s < B; ++s) {
            const int nr = a.st[s].nrows;
            s_first[s] = used;
            a.rows->seq_first[s] = used;
            a.rows->seq_cnt[s] = nr;
            a.rows->seq_maxpos[s] = nr > 0 ? a.st[s].kv_len + nr - 1 : -1;
            if (nr > 0) mp = max(mp, a.st[s].kv_len + nr - 1);
            used += nr;
        }
        if (used > dims.row_cap) { atomicExch(a.dev_err, kDevErrCapacity); used = 0; }
        a.rows->rows_used = used;
        a.rows->max_pos = mp;
        s_first[B < kSeqCap ? B : kSeqCap - 1] = used;
    }
    __syncthreads();
    const int used = a.rows->rows_used;
    for (int s = warp; s < B; s += n_warps) {
        const SeqState& S = a.st[s];
        const int* rs = a.ref + (int64_t)s * dims.max_ref;
        const int* tg = a.target ? a.target + (int64_t)s * a.y_cap : nullptr;
        const int first = s_first[s];
        if (first + S.nrows > used) continue;  // the capacity error above voided the step
        for (int j = lane; j < S.nrows; j += 32) {
            int tok;
            if (j == 0) tok = S.pending;
            else if (S.forced_rows > 0) tok = tg[min(S.y_len + j - 1, a.y_cap - 1)];  // replay: the target's next tokens
            else tok = rs[S.pos + j - 1];
            a.rows->tok[first + j] = tok;
            a.rows->pos[first + j] = S.kv_len + j;
            a.rows->seq[first + j] = s;
        }
    }
    for (int r = used + threadIdx.x; r < dims.row_cap; r += kTailThreads) {
        a.rows->tok[r] = 0; a.rows->pos[r] = -1; a.rows->seq[r] = 0;
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
                                                         void* __restrict__ xs, int xs_layout, float* __restrict__ ss,
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
        store_act(xs, xs_layout, dims.row_cap, r, col, d, v * gain[col]);
    }
    float sq = v * v;
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0) ss[(int64_t)t * dims.row_cap + r] = ((red[0] + red[1]) + red[2]) + red[3];
}

// ---- launchers -----------------------------------------------------------------------
void launch_step_tail(cudaStream_t st, const TailArgs& a) {
    launch_pdl(st, true, dim3(1), dim3(kTailThreads), 0, step_tail_kernel, a);
}

void launch_embed(cudaStream_t st, const ModelDims& dims, bool bf16, int n_rows, const RowDesc* rows, const void* emb,
                  float* x, int32_t* dev_err) {
    if (bf16)
        launch_pdl(st, true, dim3(n_rows), dim3(256), 0, embed_kernel<__nv_bfloat16>, dims, rows, (const __nv_bfloat16*)emb, x, dev_err);
    else
        launch_pdl(st, true, dim3(n_rows), dim3(256), 0, embed_kernel<float>, dims, rows, (const float*)emb, x, dev_err);
}

void launch_embed_norm(cudaStream_t st, const ModelDims& dims, int n_rows, const RowDesc* rows, const void* emb,
                       const float* gain, float* x, void* xs, int xs_layout, float* ss, int32_t* dev_err) {
    launch_pdl(st, true, dim3(n_rows, (dims.d_model + 127) / 128), dim3(128), 0, embed_norm_kernel, dims, rows,
               (const __nv_bfloat16*)emb, gain, x, xs, xs_layout, ss, dev_err);
}

}  // namespace llma

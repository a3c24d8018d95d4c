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
//     among reference positions `pos` (inside one document, with at
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
constexpr int kStateWords = sizeof(SeqState) / sizeof(int32_t);

// The kernel is a chain of small dependent steps, so what it costs is the number of global-memory round
// trips on that chain: the sequences' state is staged in shared memory once and written back at the end,
// the rows' final tokens stay in shared memory, and loads that do not depend on one another are issued together.
__global__ void __launch_bounds__(kTailThreads) step_tail_kernel(const TailArgs a) {
    pdl_trigger();
    pdl_wait();
    const ModelDims& dims = a.dims;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = kTailThreads / 32;
    const int B = dims.max_batch;
    __shared__ SeqState s_st[kSeqCap];
    __shared__ int s_first[kSeqCap + 1];
    __shared__ int s_tok[kRowCap];
    __shared__ unsigned long long s_best[kSeqCap];

    {
        const int32_t* src = reinterpret_cast<const int32_t*>(a.st);
        int32_t* dst = reinterpret_cast<int32_t*>(s_st);
        for (int i = threadIdx.x; i < B * kStateWords; i += kTailThreads) dst[i] = __ldcg(src + i);
        for (int s = threadIdx.x; s < B; s += kTailThreads) { s_first[s] = __ldcg(&a.rows->seq_first[s]); s_best[s] = 0ull; }
    }
    if (a.do_accept) {
        // ---- final token of every row slot a decoding step can use (lowest index on ties) --------------------
        const int n_slots = a.n_rows;
        if (a.part_max) {
            for (int r = warp; r < n_slots; r += n_warps) {
                float bv = -INFINITY; int bi = 0x7fffffff;
                for (int t0 = 0; t0 < a.n_tiles; t0 += 32 * 8) {  // eight loads of each array in flight per lane
                    float v[8]; int ix[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int t = t0 + u * 32 + lane;
                        v[u] = t < a.n_tiles ? __ldcg(&a.part_max[(int64_t)t * dims.row_cap + r]) : -INFINITY;
                        ix[u] = t < a.n_tiles ? __ldcg(&a.part_idx[(int64_t)t * dims.row_cap + r]) : 0x7fffffff;
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (v[u] > bv || (v[u] == bv && ix[u] < bi)) { bv = v[u]; bi = ix[u]; }
                }
                for (int o = 16; o > 0; o >>= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
                }
                if (lane == 0) { s_tok[r] = bi; a.out_tok[r] = bi; }
            }
        } else {
            for (int r = threadIdx.x; r < n_slots; r += kTailThreads) s_tok[r] = __ldcg(&a.out_tok[r]);
        }
        __syncthreads();
        // ---- acceptance + commit, one warp per sequence -------------------------------------------------------
        for (int s = warp; s < B; s += n_warps) {
            SeqState& S = s_st[s];
            const int nrows = S.nrows;
            if (nrows <= 0) {
                if (lane == 0) { S.last_pos = -1; S.last_k_eff = 0; S.last_accepted = 0; S.last_emitted = 0; }
                continue;
            }
            const int* rs = a.ref + (int64_t)s * dims.max_ref;
            const int* o = s_tok + s_first[s];
            int* ys = a.y + (int64_t)s * a.y_cap;
            const int k_eff = S.k_eff, pos = S.pos, ylen = S.y_len;
            int m, done = 0, pending;
            if (S.forced_rows > 0) {
                // replay: the trace says how many tokens the step emits, the target text which ones
                m = S.forced_emit;
                const int* tg = a.target + (int64_t)s * a.y_cap;
                for (int j = lane; j < m; j += 32) ys[ylen + j] = tg[ylen + j];
                pending = tg[ylen + m - 1];
            } else {
                // first copied token the model disagrees with (32 comparisons per round), then the first EOS
                int acc = k_eff;
                for (int j0 = 0; j0 < k_eff; j0 += 32) {
                    const int j = j0 + lane;
                    const bool differs = j < k_eff && o[j] != __ldg(&rs[pos + j]);
                    const unsigned mask = __ballot_sync(0xffffffffu, differs);
                    if (mask) { acc = j0 + __ffs(mask) - 1; break; }
                }
                m = acc + 1;
                if (dims.eos_id >= 0) {
                    for (int j0 = 0; j0 < m; j0 += 32) {
                        const int j = j0 + lane;
                        const unsigned mask = __ballot_sync(0xffffffffu, j < m && o[j] == dims.eos_id);
                        if (mask) { m = j0 + __ffs(mask); done = 1; break; }
                    }
                }
                for (int j = lane; j < m; j += 32) ys[ylen + j] = o[j];
                pending = o[m - 1];
                // adaptive copy length: twice as many tokens after a copy the model agreed with in full, half as
                // many (rounded up) after one it cut short; within [k_min, the engine's largest k]
                if (lane == 0 && S.k_cur > 0 && k_eff > 0)
                    S.k_cur = acc == k_eff ? min(2 * S.k_cur, dims.kp1 - 1) : max(S.k_min, (S.k_cur + 1) >> 1);
            }
            __syncwarp();
            if (lane == 0) {
                S.pending = pending;
                S.y_len = ylen + m;
                S.kv_len += m;
                S.steps += 1;
                S.trigger_steps += (k_eff > 0);
                S.copied_accepted += m - 1;
                S.last_pos = pos; S.last_k_eff = k_eff; S.last_accepted = m - 1; S.last_emitted = m;
                if (ylen + m >= S.target_len) done = 1;
                S.done = done;
                S.nrows = 0;
            }
        }
    }
    __syncthreads();
    if (a.do_plan) {
        // ---- trigger search: every thread takes reference positions of every live sequence ---------------------
        // key = (ext << 32) | (0x7fffffff - pos): the maximum is the longest agreement, then the earliest position
        if (a.k > 0 && a.n >= 1) {
            // the 32 warps are dealt over the sequences (all of them on one sequence at batch 1, two per sequence at
            // batch 16, one warp for several sequences beyond 32), so that every sequence's loads are in flight at once
            const int per_seq = B >= n_warps ? 1 : n_warps / B;      // warps that share a sequence
            const int groups = n_warps / per_seq;                    // sequences scanned at a time
            const int sub = warp % per_seq;
            for (int s = warp / per_seq; s < B; s += groups) {
                const SeqState& S = s_st[s];
                const int ylen = S.y_len, ref_len = S.ref_len;
                const bool live = S.active && !S.done && ylen < S.target_len;
                if (!live || S.forced_rows != 0 || ylen < a.n || ref_len <= 0) continue;   // uniform over the warp
                const int* ys = a.y + (int64_t)s * a.y_cap;
                const int* rs = a.ref + (int64_t)s * dims.max_ref;
                const int* ds = a.doc_start + (int64_t)s * dims.max_ref;
                const int* de = a.doc_end + (int64_t)s * dims.max_ref;
                const int last = S.pending;  // the newest generated token (ylen >= 1 here)
                const int stride = 32 * per_seq;
                for (int p0 = 1 + sub * 32 + lane; p0 < ref_len; p0 += 2 * stride) {
                    // two candidates per round, their loads in flight together
                    int tokv[2], endv[2], begv[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int p = p0 + u * stride;
                        const bool in = p < ref_len;
                        tokv[u] = in ? __ldg(&rs[p - 1]) : -1;
                        endv[u] = in ? __ldg(&de[p - 1]) : 0;
                        begv[u] = in ? __ldg(&ds[p - 1]) : 0;
                    }
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int p = p0 + u * stride;
                        // candidate: ref[p-1] is the last matched token; p must stay inside its document
                        if (p >= ref_len || tokv[u] != last || p >= endv[u]) continue;
                        int t = 1;
                        while (t < ylen && p - t - 1 >= begv[u] && __ldg(&rs[p - t - 1]) == __ldcg(&ys[ylen - t - 1])) ++t;
                        if (t >= a.n) atomicMax(&s_best[s], ((unsigned long long)(unsigned)t << 32) | (unsigned)(0x7fffffff - p));
                    }
                }
            }
        }
        __syncthreads();
        // ---- copy length, one thread per sequence ---------------------------------------------------------------
        for (int s = threadIdx.x; s < B; s += kTailThreads) {
            SeqState& S = s_st[s];
            const bool live = S.active && !S.done && S.y_len < S.target_len;
            const int ylen = S.y_len;
            int pos = -1, k_eff = 0, nrows = 0;
            if (live && a.trace && S.forced_rows != 0) {
                // replay: shape of the next step from the trace
                const int step = S.trace_step;
                int fr = 1, fe = 1;
                if (step < a.trace_cap) {
                    fr = a.trace[((int64_t)s * a.trace_cap + step) * 2];
                    fe = a.trace[((int64_t)s * a.trace_cap + step) * 2 + 1];
                }
                fr = max(1, min(fr, min(dims.kp1, dims.max_seq - S.kv_len)));
                fe = max(1, min(fe, min(fr, S.target_len - ylen)));
                nrows = fr; k_eff = fr - 1;
                S.forced_rows = fr; S.forced_emit = fe; S.trace_step = step + 1;
            } else if (live) {
                const unsigned long long best = s_best[s];
                if (best != 0ull) {
                    const int* de = a.doc_end + (int64_t)s * dims.max_ref;
                    pos = 0x7fffffff - (int)(unsigned)(best & 0xffffffffull);
                    const int room_doc = __ldg(&de[pos - 1]) - pos;
                    const int room_out = S.target_len - ylen - 1;
                    const int room_kv = dims.max_seq - S.kv_len - 1;
                    const int k_want = S.k_cur > 0 ? min(S.k_cur, a.k) : a.k;
                    k_eff = min(min(k_want, room_doc), min(room_out, room_kv));
                    if (k_eff <= 0) { k_eff = 0; pos = -1; }
                }
                nrows = k_eff + 1;
                if (S.kv_len + nrows > dims.max_seq) {  // no room even for the pending token
                    atomicExch(a.dev_err, kDevErrCapacity);
                    nrows = 0; pos = -1; k_eff = 0;
                }
            }
            S.pos = pos; S.k_eff = k_eff; S.nrows = nrows;
        }
        __syncthreads();
        // ---- pack the rows: sequence s owns rows first[s] .. first[s] + nrows - 1 -------------------------------
        if (threadIdx.x == 0) {
            int used = 0, mp = -1;
            for (int s = 0; s < B; ++s) {
                const int nr = s_st[s].nrows;
                s_first[s] = used;
                if (nr > 0) mp = max(mp, s_st[s].kv_len + nr - 1);
                used += nr;
            }
            if (used > a.n_rows) { atomicExch(a.dev_err, kDevErrCapacity); used = 0; }
            s_first[kSeqCap] = used;
            a.rows->rows_used = used;
            a.rows->max_pos = mp;
        }
        __syncthreads();
        const int used = s_first[kSeqCap];
        for (int s = threadIdx.x; s < B; s += kTailThreads) {
            const int nr = used > 0 ? s_st[s].nrows : 0;
            a.rows->seq_first[s] = s_first[s];
            a.rows->seq_cnt[s] = nr;
            a.rows->seq_maxpos[s] = nr > 0 ? s_st[s].kv_len + nr - 1 : -1;
        }
        for (int s = warp; s < B; s += n_warps) {
            const SeqState& S = s_st[s];
            if (used == 0) break;  // the capacity error above voided the step
            const int* rs = a.ref + (int64_t)s * dims.max_ref;
            const int* tg = a.target ? a.target + (int64_t)s * a.y_cap : nullptr;
            const int first = s_first[s];
            for (int j = lane; j < S.nrows; j += 32) {
                int tok;
                if (j == 0) tok = S.pending;
                else if (S.forced_rows > 0) tok = tg[min(S.y_len + j - 1, a.y_cap - 1)];  // replay: the target's next tokens
                else tok = __ldg(&rs[S.pos + j - 1]);
                a.rows->tok[first + j] = tok;
                a.rows->pos[first + j] = S.kv_len + j;
                a.rows->seq[first + j] = s;
            }
        }
        for (int r = used + threadIdx.x; r < dims.row_cap; r += kTailThreads) {
            a.rows->tok[r] = 0; a.rows->pos[r] = -1; a.rows->seq[r] = 0;
        }
    }
    __syncthreads();
    {
        const int32_t* src = reinterpret_cast<const int32_t*>(s_st);
        int32_t* dst = reinterpret_cast<int32_t*>(a.st);
        for (int i = threadIdx.x; i < B * kStateWords; i += kTailThreads) dst[i] = src[i];
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
        store_act(xs, kActSplit, dims.row_cap, r, col, d, v * gain[col]);
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
                       const float* gain, float* x, void* xs, float* ss, int32_t* dev_err) {
    launch_pdl(st, true, dim3(n_rows, (dims.d_model + 127) / 128), dim3(128), 0, embed_norm_kernel, dims, rows,
               (const __nv_bfloat16*)emb, gain, x, xs, ss, dev_err);
}

}  // namespace llma

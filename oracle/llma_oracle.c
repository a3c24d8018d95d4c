/*
 * CPU oracle for the LLaMA-style decoder forward used by LLMA decoding.
 *
 * THIS IS TEST INFRASTRUCTURE.  It is the slow, plain statement of what the
 * decoder computes for ONE token at ONE position; only the tests, the smoke
 * check and the CPU-baseline leg of the benchmark may call it.  It shares no
 * code with the CUDA library.
 *
 * What it follows:
 *   - Eq. 2 of the paper (greedy: y_i = argmax_y P(y | x, y_<i)) needs the
 *     next-token logits of a causal decoder; Eq. 3 needs the same logits at
 *     k+1 consecutive positions.  The Python side obtains the latter by calling
 *     this one-position forward k+1 times in order, which makes causality and
 *     independence from k true by construction.
 *   - The paper only says the model is LLaMA run through a standard library
 *     (Section 3.3).  The architecture written out here is that family's:
 *     pre-norm RMSNorm, rotary position embedding with the half-split pairing
 *     (i, i + head_dim/2), multi-head causal softmax attention scaled by
 *     1/sqrt(head_dim), SiLU-gated feed-forward, no biases, untied LM head.
 *
 * Precision: every stored activation is fp32; every reduction (dot products,
 * sum of squares, softmax normaliser) is accumulated in fp64 so the result does
 * not depend on summation order to fp32 accuracy.  With bf16 storage the
 * weights are widened exactly, and K/V rows are rounded to bf16 (nearest-even)
 * when they enter the cache, because the cache itself is defined to be bf16.
 *
 * Parity pins: every function below is pinned by tests that do not reuse this
 * code (closed forms, invariants, brute force, and an independent library
 * implementation of the same decoder family); none is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
    int32_t weights_bf16;  /* 0: matrices are float32; 1: uint16 bf16 bit patterns */
    int32_t kv_round_bf16; /* 1: round cached K/V rows to bf16 */
    int32_t max_seq;
    float rms_eps, rope_theta;
} oracle_config;

typedef struct {
    const void *tok_emb, *lm_head; /* [vocab, d] */
    const float *final_norm;       /* [d] */
    const float *const *attn_norm; /* per layer [d] */
    const void *const *wq, *const *wk, *const *wv; /* [H*hd, d] */
    const void *const *wo;         /* [d, H*hd] */
    const float *const *ffn_norm;  /* [d] */
    const void *const *w_gate, *const *w_up; /* [F, d] */
    const void *const *w_down;     /* [d, F] */
} oracle_weights;

typedef struct {
    oracle_config cfg;
    oracle_weights w;
    float *kcache, *vcache; /* [layer][pos][H*hd] */
    float *x, *h, *q, *k, *v, *att, *gate, *up, *tmp;
    double *scores;
    /* prescribed cache codes for the next forward call (see oracle_prescribe_kv), or NULL */
    const float *given_k, *given_v;
    double given_tol;
    double *given_stats;
} oracle_model;

/* ---- scalar helpers ------------------------------------------------------- */

static inline float widen_bf16(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* fp32 -> nearest bf16 (ties to even), returned as fp32 */
float oracle_round_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return f; /* inf / nan pass through */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return f;
}

/* out[r] = sum_c W[r, c] * x[c]; W row-major, float32 or bf16 bits */
void oracle_matvec(const void *W, int32_t w_bf16, int64_t rows, int64_t cols, const float *x, float *out) {
    int64_t r;
#pragma omp parallel for schedule(static) if (rows * cols > 65536)
    for (r = 0; r < rows; ++r) {
        double acc = 0.0;
        if (w_bf16) {
            const uint16_t *w = (const uint16_t *)W + r * cols;
            for (int64_t c = 0; c < cols; ++c) acc += (double)widen_bf16(w[c]) * (double)x[c];
        } else {
            const float *w = (const float *)W + r * cols;
            for (int64_t c = 0; c < cols; ++c) acc += (double)w[c] * (double)x[c];
        }
        out[r] = (float)acc;
    }
}

/* RMSNorm: out = x / sqrt(mean(x^2) + eps) * g */
void oracle_rmsnorm(const float *x, const float *g, int32_t n, float eps, float *out) {
    double ss = 0.0;
    for (int32_t i = 0; i < n; ++i) ss += (double)x[i] * (double)x[i];
    double inv = 1.0 / sqrt(ss / (double)n + (double)eps);
    for (int32_t i = 0; i < n; ++i) out[i] = (float)((double)x[i] * inv * (double)g[i]);
}

/* Rotary embedding of one head vector in place: pair (i, i+hd/2) is rotated by
 * the angle pos * theta^(-2i/hd). */
void oracle_rope(float *vec, int32_t head_dim, int32_t pos, float theta) {
    int32_t half = head_dim / 2;
    for (int32_t i = 0; i < half; ++i) {
        double ang = (double)pos * pow((double)theta, -2.0 * (double)i / (double)head_dim);
        double c = cos(ang), s = sin(ang);
        double a = vec[i], b = vec[i + half];
        vec[i] = (float)(a * c - b * s);
        vec[i + half] = (float)(a * s + b * c);
    }
}

/* One query against n_pos cached rows of one head.
 * K, V: row p of the head starts at K + p*stride.  out[hd]. scores: scratch [n_pos]. */
void oracle_attention(const float *q, const float *K, const float *V, int32_t n_pos, int64_t stride,
                      int32_t head_dim, float *out, double *scores) {
    double scale = 1.0 / sqrt((double)head_dim);
    double mx = -INFINITY;
    for (int32_t p = 0; p < n_pos; ++p) {
        const float *kr = K + (int64_t)p * stride;
        double s = 0.0;
        for (int32_t i = 0; i < head_dim; ++i) s += (double)q[i] * (double)kr[i];
        s *= scale;
        scores[p] = s;
        if (s > mx) mx = s;
    }
    double denom = 0.0;
    for (int32_t p = 0; p < n_pos; ++p) {
        scores[p] = exp(scores[p] - mx);
        denom += scores[p];
    }
    for (int32_t i = 0; i < head_dim; ++i) {
        double acc = 0.0;
        for (int32_t p = 0; p < n_pos; ++p) acc += scores[p] * (double)V[(int64_t)p * stride + i];
        out[i] = (float)(acc / denom);
    }
}

/* out = silu(g) * u, silu(g) = g / (1 + exp(-g)) */
void oracle_silu_mul(const float *g, const float *u, int32_t n, float *out) {
    for (int32_t i = 0; i < n; ++i) {
        double gg = g[i];
        out[i] = (float)(gg / (1.0 + exp(-gg)) * (double)u[i]);
    }
}

/* ---- prescribed cache codes -------------------------------------------------
 * The cache is bf16 by definition, so a cached element is a quantised code decided by an
 * fp32 value.  Two correct computations whose values differ in their last bits can fall on
 * different sides of a rounding boundary, and the two codes then differ by a whole bf16 step,
 * a difference thousands of times larger than its cause.  A comparison may therefore
 * PRESCRIBE the codes.  A prescribed code g is accepted for an element whose unrounded value
 * here is x iff
 *        |g - x| <= step(x) / 2 + tol * max(1, max |row|)
 * i.e. iff g is what rounding to nearest gives for SOME value within the stated absolute
 * tolerance of x (step = spacing of bf16 values at the larger of |x|, |g|; the tolerance is the
 * one the projection itself is held to).  Anything else is counted as a violation and the
 * oracle keeps its own code.  stats[0] counts elements whose prescribed code differs from the
 * oracle's own rounding, stats[1] the violations, stats[2] is the largest share of the
 * tolerance an accepted difference needed, (|g - x| - step / 2) / (tol * max(1, max|row|)),
 * stats[3] counts all elements seen. */
static void adopt_codes(const float *own, const float *given, float *dst, int64_t n, double tol, double *stats) {
    double rowmax = 1.0;
    for (int64_t i = 0; i < n; ++i)
        if (fabs((double)own[i]) > rowmax) rowmax = fabs((double)own[i]);
    const double slack = tol * rowmax;
    for (int64_t i = 0; i < n; ++i) {
        const float r = oracle_round_bf16(own[i]);
        const float g = given[i];
        stats[3] += 1.0;
        if (g == r) { dst[i] = r; continue; }
        stats[0] += 1.0;
        const double x = own[i];
        const double big = fabs((double)g) > fabs(x) ? fabs((double)g) : fabs(x);
        int e;
        (void)frexp(big, &e);
        const double step = ldexp(1.0, e - 8); /* spacing of bf16 values at this magnitude */
        const double excess = fabs((double)g - x) - 0.5 * step;
        if (excess <= slack) {
            if (excess / slack > stats[2]) stats[2] = excess / slack;
            dst[i] = g;
        } else {
            stats[1] += 1.0;
            dst[i] = r;
        }
    }
}

/* k_rows, v_rows: [n_layers][H*hd] codes for the position of the NEXT oracle_forward call (used once);
 * tol: the relative tolerance above; stats: double[4], accumulated into (the caller zeroes it). */
void oracle_prescribe_kv(oracle_model *m, const float *k_rows, const float *v_rows, double tol, double *stats) {
    m->given_k = k_rows; m->given_v = v_rows; m->given_tol = tol; m->given_stats = stats;
}

/* ---- model ---------------------------------------------------------------- */

oracle_model *oracle_create(const oracle_config *cfg, const oracle_weights *w) {
    oracle_model *m = (oracle_model *)calloc(1, sizeof(oracle_model));
    if (!m) return NULL;
    m->cfg = *cfg;
    m->w = *w;
    int64_t hh = (int64_t)cfg->n_heads * cfg->head_dim;
    int64_t kv = (int64_t)cfg->n_layers * cfg->max_seq * hh;
    m->kcache = (float *)calloc((size_t)kv, sizeof(float));
    m->vcache = (float *)calloc((size_t)kv, sizeof(float));
    m->x = (float *)calloc((size_t)cfg->d_model, sizeof(float));
    m->h = (float *)calloc((size_t)cfg->d_model, sizeof(float));
    m->q = (float *)calloc((size_t)hh, sizeof(float));
    m->k = (float *)calloc((size_t)hh, sizeof(float));
    m->v = (float *)calloc((size_t)hh, sizeof(float));
    m->att = (float *)calloc((size_t)hh, sizeof(float));
    m->gate = (float *)calloc((size_t)cfg->d_ffn, sizeof(float));
    m->up = (float *)calloc((size_t)cfg->d_ffn, sizeof(float));
    m->tmp = (float *)calloc((size_t)(cfg->d_model > cfg->d_ffn ? cfg->d_model : cfg->d_ffn), sizeof(float));
    m->scores = (double *)calloc((size_t)cfg->max_seq, sizeof(double));
    if (!m->kcache || !m->vcache || !m->x || !m->h || !m->q || !m->k || !m->v || !m->att || !m->gate ||
        !m->up || !m->tmp || !m->scores)
        return NULL;
    return m;
}

void oracle_destroy(oracle_model *m) {
    if (!m) return;
    free(m->kcache); free(m->vcache); free(m->x); free(m->h); free(m->q); free(m->k); free(m->v);
    free(m->att); free(m->gate); free(m->up); free(m->tmp); free(m->scores);
    free(m);
}

/* Push `token` through the decoder at position `pos`: its K/V rows are written
 * to cache row `pos` (overwriting whatever a discarded token left there) and it
 * attends to rows 0..pos.  If logits != NULL the next-token logits [vocab] are
 * written.  If hidden != NULL the final residual stream [d] is written.
 * Returns 0, or -1 on a bad token / position. */
int32_t oracle_forward(oracle_model *m, int32_t token, int32_t pos, float *logits, float *hidden) {
    const oracle_config *c = &m->cfg;
    if (token < 0 || token >= c->vocab || pos < 0 || pos >= c->max_seq) return -1;
    const int32_t d = c->d_model, H = c->n_heads, hd = c->head_dim, F = c->d_ffn;
    const int64_t hh = (int64_t)H * hd;
    const int32_t wb = c->weights_bf16;

    for (int32_t i = 0; i < d; ++i)
        m->x[i] = wb ? widen_bf16(((const uint16_t *)m->w.tok_emb)[(int64_t)token * d + i])
                     : ((const float *)m->w.tok_emb)[(int64_t)token * d + i];

    for (int32_t l = 0; l < c->n_layers; ++l) {
        float *Kl = m->kcache + (int64_t)l * c->max_seq * hh;
        float *Vl = m->vcache + (int64_t)l * c->max_seq * hh;
        /* attention block */
        oracle_rmsnorm(m->x, m->w.attn_norm[l], d, c->rms_eps, m->h);
        oracle_matvec(m->w.wq[l], wb, hh, d, m->h, m->q);
        oracle_matvec(m->w.wk[l], wb, hh, d, m->h, m->k);
        oracle_matvec(m->w.wv[l], wb, hh, d, m->h, m->v);
        for (int32_t hI = 0; hI < H; ++hI) {
            oracle_rope(m->q + (int64_t)hI * hd, hd, pos, c->rope_theta);
            oracle_rope(m->k + (int64_t)hI * hd, hd, pos, c->rope_theta);
        }
        if (m->given_k && c->kv_round_bf16) {
            adopt_codes(m->k, m->given_k + (int64_t)l * hh, Kl + (int64_t)pos * hh, hh, m->given_tol, m->given_stats);
            adopt_codes(m->v, m->given_v + (int64_t)l * hh, Vl + (int64_t)pos * hh, hh, m->given_tol, m->given_stats);
        } else {
            for (int64_t i = 0; i < hh; ++i) {
                Kl[(int64_t)pos * hh + i] = c->kv_round_bf16 ? oracle_round_bf16(m->k[i]) : m->k[i];
                Vl[(int64_t)pos * hh + i] = c->kv_round_bf16 ? oracle_round_bf16(m->v[i]) : m->v[i];
            }
        }
        for (int32_t hI = 0; hI < H; ++hI)
            oracle_attention(m->q + (int64_t)hI * hd, Kl + (int64_t)hI * hd, Vl + (int64_t)hI * hd, pos + 1, hh, hd,
                             m->att + (int64_t)hI * hd, m->scores);
        oracle_matvec(m->w.wo[l], wb, d, hh, m->att, m->tmp);
        for (int32_t i = 0; i < d; ++i) m->x[i] += m->tmp[i];
        /* feed-forward block */
        oracle_rmsnorm(m->x, m->w.ffn_norm[l], d, c->rms_eps, m->h);
        oracle_matvec(m->w.w_gate[l], wb, F, d, m->h, m->gate);
        oracle_matvec(m->w.w_up[l], wb, F, d, m->h, m->up);
        oracle_silu_mul(m->gate, m->up, F, m->gate);
        oracle_matvec(m->w.w_down[l], wb, d, F, m->gate, m->tmp);
        for (int32_t i = 0; i < d; ++i) m->x[i] += m->tmp[i];
    }
    m->given_k = m->given_v = NULL;
    if (hidden) memcpy(hidden, m->x, (size_t)d * sizeof(float));
    if (logits) {
        oracle_rmsnorm(m->x, m->w.final_norm, d, c->rms_eps, m->h);
        oracle_matvec(m->w.lm_head, wb, c->vocab, d, m->h, logits);
    }
    return 0;
}

/* Read back one cached row (for tests): which = 0 for K, 1 for V. out[H*hd]. */
int32_t oracle_read_cache(const oracle_model *m, int32_t layer, int32_t pos, int32_t which, float *out) {
    const oracle_config *c = &m->cfg;
    if (layer < 0 || layer >= c->n_layers || pos < 0 || pos >= c->max_seq) return -1;
    int64_t hh = (int64_t)c->n_heads * c->head_dim;
    const float *src = (which ? m->vcache : m->kcache) + ((int64_t)layer * c->max_seq + pos) * hh;
    memcpy(out, src, (size_t)hh * sizeof(float));
    return 0;
}

/*
 * llma.h -- C ABI of the LLMA reference-copy decoding engine for one NVIDIA B200 (sm_100a).
 *
 * LLMA ("inference with reference", arXiv 2304.04487) speeds up greedy decoding when the
 * output shares token spans with reference documents.  At every decoding step the last n
 * generated tokens are matched against the references (Section 2.2); on a match the k
 * tokens that follow it are copied into the decoder input and all k+1 positions are
 * evaluated in ONE causal forward pass (Eq. 3); the longest prefix of copied tokens that
 * agrees with the model's own argmax outputs is kept, plus one more output token
 * (Algorithm 1, the acceptance loop).  The result is token-for-token what greedy decoding (Eq. 2)
 * produces.
 *
 * Every step of that path -- trigger search, copy + embedding gather, the decoder layers
 * (RMSNorm, QKV projection + rotary embedding + K/V append, causal attention over the K/V
 * cache, output projection, SiLU-gated feed-forward), LM head + per-row argmax, acceptance
 * and K/V commit -- runs in CUDA kernels of this library.  There is no CPU fallback: every
 * entry point fails with LLMA_ERR_CUDA if no usable device is present.
 *
 * Conventions
 *   - All functions return 0 (LLMA_OK) or a negative llma_status; nothing throws or aborts.
 *     After an argument error the engine is unchanged and usable.
 *   - "device" pointers are CUDA device pointers valid on the engine's device; "host"
 *     pointers are ordinary process memory.  The library never frees caller memory.
 *   - Weight matrices are row-major [out_features, in_features] with no padding, fp32
 *     (dtype LLMA_DTYPE_F32) or bf16 (LLMA_DTYPE_BF16); norm gains are always fp32.  The
 *     engine BORROWS them: keep them alive and unmodified until llma_destroy.
 *   - Token ids are int32 in [0, vocab).
 *   - Calls on one engine must not overlap in time; different engines are independent.
 */
#ifndef LLMA_H_
#define LLMA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct llma_engine llma_engine; /* opaque */

typedef enum {
    LLMA_OK = 0,
    LLMA_ERR_NULL = -1,           /* a required pointer was NULL */
    LLMA_ERR_CONFIG = -2,         /* unsupported or inconsistent llma_config */
    LLMA_ERR_TOKEN_RANGE = -3,    /* a token id outside [0, vocab) */
    LLMA_ERR_CAPACITY = -4,       /* sequence would exceed max_seq, or batch index out of range */
    LLMA_ERR_REF_TOO_LONG = -5,   /* reference longer than max_ref or malformed doc_offsets */
    LLMA_ERR_STATE = -6,          /* call not valid in the sequence's current state */
    LLMA_ERR_CUDA = -7,           /* a CUDA call failed (llma_last_cuda_error has the code) */
    LLMA_ERR_DEVICE_TIMEOUT = -8, /* a bounded on-device wait ran out; the step's results are void */
    LLMA_ERR_ARG = -9             /* n < 1, k outside [0, max_k], max_new < 0 ... */
} llma_status;

enum { LLMA_DTYPE_F32 = 0, LLMA_DTYPE_BF16 = 1 };
enum { LLMA_GEMM_AUTO = 0, LLMA_GEMM_SIMT = 1, LLMA_GEMM_TCGEN05 = 2 };

typedef struct {
    int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
    int32_t dtype;        /* storage type of weights and K/V cache: LLMA_DTYPE_* */
    int32_t max_batch;    /* sequences held at once (<= 256); max_batch * (max_k + 1) must be <= 256 */
    int32_t max_seq;      /* K/V rows per sequence */
    int32_t max_ref;      /* reference tokens per sequence */
    int32_t max_k;        /* largest copy length k that will be requested (0..255) */
    float rms_eps;        /* RMSNorm epsilon */
    float rope_theta;     /* rotary base; pairing is (i, i + head_dim/2) */
    int32_t eos_id;       /* -1: none.  Otherwise a sequence stops after emitting this id */
    int32_t gemm_impl;    /* LLMA_GEMM_*; AUTO = tensor-core kernels for bf16, SIMT for fp32 */
    int32_t keep_logits;  /* 1: keep the last step's logits for llma_debug_logits */
} llma_config;

/* Device pointers.  Per-layer arrays are HOST arrays of n_layers device pointers. */
typedef struct {
    const void *tok_emb;           /* [vocab, d_model] */
    const void *lm_head;           /* [vocab, d_model] */
    const float *final_norm;       /* [d_model] */
    const float *const *attn_norm; /* [d_model] each */
    const void *const *wq;         /* [n_heads*head_dim, d_model] each */
    const void *const *wk;
    const void *const *wv;
    const void *const *wo;         /* [d_model, n_heads*head_dim] */
    const float *const *ffn_norm;  /* [d_model] */
    const void *const *w_gate;     /* [d_ffn, d_model] */
    const void *const *w_up;       /* [d_ffn, d_model] */
    const void *const *w_down;     /* [d_model, d_ffn] */
} llma_weights;

/* Decode statistics of Section 4.2 (triggers, accepted copied tokens, decoding steps),
 * summed over the sequences of the last llma_generate call, plus device time. */
typedef struct {
    int64_t steps;            /* decoding steps taken (forward passes), per-sequence sum */
    int64_t trigger_steps;    /* steps in which a copy was applied */
    int64_t copied_accepted;  /* copied tokens that survived verification */
    int64_t tokens;           /* tokens emitted = steps + copied_accepted */
    int64_t launches;         /* kernels launched by this library during the call */
    float device_ms;          /* CUDA-event time from first to last kernel of the call */
} llma_stats;

/* Per-sequence record of the most recent step (for tests and tracing). */
typedef struct {
    int32_t pos;       /* first copied reference index, -1 when nothing was copied */
    int32_t k_eff;     /* copied tokens fed to the model */
    int32_t accepted;  /* copied tokens kept */
    int32_t emitted;   /* tokens appended this step (0 if the sequence was idle) */
} llma_step_info;

/*
 * Create an engine on the current CUDA device.  `cuda_stream` is a cudaStream_t (may be
 * NULL for the default stream); all work of the engine is issued on it.  Allocates the K/V
 * cache ([layer][seq][head][max_seq][head_dim], zero-filled), reference storage and
 * workspaces.  Supported: head_dim 64 or 128; d_model, n_heads*head_dim and d_ffn multiples
 * of 64; max_batch <= 256 and max_batch*(max_k+1) <= 256 rows per decoding step (the rows of a
 * step are packed, so a sequence without a copy takes one row).  Errors: NULL, CONFIG, CUDA.
 */
int llma_create(const llma_config *cfg, const llma_weights *w, void *cuda_stream, llma_engine **out);

/* Free everything the engine owns (synchronises the stream first).  NULL is allowed. */
int llma_destroy(llma_engine *e);

/*
 * Load a prompt x (host, n_prompt >= 1 tokens) into sequence slot `seq`: positions
 * 0..n_prompt-2 are pushed through the decoder (128 positions per pass on the tensor-core path) and
 * cached; the last prompt token becomes
 * the pending input of the first decoding step (Algorithm 1 starts with y empty and calls
 * the model inside its loop, so prefill emits nothing).  Clears the sequence's output and
 * statistics; keeps its reference.  Synchronous.  Errors: NULL, CAPACITY, TOKEN_RANGE, CUDA.
 */
int llma_prefill(llma_engine *e, int32_t seq, const int32_t *prompt, int32_t n_prompt);

/*
 * Set the reference documents D of a sequence (Section 2.2): `tokens` (host, n_tokens ids)
 * is the concatenation of n_docs documents; doc_offsets (host, n_docs+1 non-decreasing
 * values from 0 to n_tokens) delimits them, or NULL for a single document.  Neither the
 * matched n-gram nor the copied span crosses a document boundary.  n_tokens = 0 clears the
 * reference (plain greedy).  Copied to the device during the call.
 * Errors: NULL, REF_TOO_LONG, TOKEN_RANGE, CAPACITY, CUDA.
 */
int llma_set_reference(llma_engine *e, int32_t seq, const int32_t *tokens, int32_t n_tokens,
                       const int32_t *doc_offsets, int32_t n_docs);

/*
 * One iteration of Algorithm 1's loop body for every prefilled, unfinished sequence:
 * trigger search with match length n >= 1, copy of up to k (0 <= k <= max_k) tokens, one
 * (k+1)-row forward pass, acceptance, K/V commit.  Synchronous.  out_tokens (host,
 * [max_batch][max_k+1]) receives each sequence's new tokens, n_out (host, [max_batch]) how
 * many (0 for idle slots).  The copy is additionally capped so the sequence never exceeds
 * max_seq.  k = 0 or an empty reference is a plain greedy step (Eq. 2).
 * Errors: NULL, ARG, STATE (no sequence prefilled), CAPACITY, CUDA, DEVICE_TIMEOUT.
 */
int llma_step(llma_engine *e, int32_t n, int32_t k, int32_t *out_tokens, int32_t *n_out);

/*
 * Algorithm 1's whole loop: decode exactly max_new further tokens for every prefilled
 * sequence (fewer only if eos_id is hit), with no host involvement inside a step and no
 * per-step host synchronisation.  out_tokens (host, [max_batch][max_new]) and n_out (host,
 * [max_batch]) receive the tokens; stats may be NULL.  The copy length of a step is
 * k_eff = min(k, tokens left in the matched document, tokens still to emit - 1), so exactly
 * max_new tokens come out.  Requires kv_len + max_new <= max_seq for every active sequence.
 * Errors: NULL, ARG, STATE, CAPACITY, CUDA, DEVICE_TIMEOUT.
 */
int llma_generate(llma_engine *e, int32_t max_new, int32_t n, int32_t k, int32_t *out_tokens,
                  int32_t *n_out, llma_stats *stats);

/*
 * Roll a sequence back to the state right after llma_prefill (output emptied, K/V length
 * reset to n_prompt-1; the cached prompt rows are reused, later rows are overwritten by the
 * next steps).  Lets several decodes share one prefill.  Errors: CAPACITY, STATE, CUDA.
 */
int llma_rewind(llma_engine *e, int32_t seq);

/*
 * Copy length chosen per step from how the last copy fared (a variant: the paper fixes n and k for a
 * whole run and sweeps them, Section 3.5; nothing in it adapts k).  While it is on for a sequence, a
 * step asks for min(k_cur, k) copied tokens instead of k, with k the argument of llma_step /
 * llma_generate; k_cur starts at k_start and, after every step that copied something, becomes
 * min(2 k_cur, max_k) if the model agreed with every copied token and max(k_min, ceil(k_cur / 2))
 * otherwise.  The output stays the greedy output: only the number of rows per step changes.
 * Call after llma_prefill; llma_rewind keeps the setting and puts k_cur back to k_start,
 * llma_prefill and llma_reset clear it.  k_min = k_start = 0 switches it off.
 * Errors: NULL, CAPACITY (seq), ARG (not 1 <= k_min <= k_start <= max_k), CUDA.
 */
int llma_set_adaptive_k(llma_engine *e, int32_t seq, int32_t k_min, int32_t k_start);

/* Forget a sequence entirely (slot becomes idle; its reference is cleared). */
int llma_reset(llma_engine *e, int32_t seq);

/* Record of the last step for each sequence: info is a host array [max_batch]. */
int llma_last_step_info(llma_engine *e, llma_step_info *info);

/*
 * Parity harness only (requires keep_logits = 1): copy the logits of the last step to
 * `out` (host, [rows][vocab] fp32) where row j of sequence s is at index s*(max_k+1)+j and
 * rows is max_batch*(max_k+1).  Rows that were not part of the step hold stale values.
 * Errors: NULL, STATE, CUDA.
 */
int llma_debug_logits(llma_engine *e, float *out);

/* Parity harness only: copy K (which=0) or V (which=1) cache row `pos` of a layer and
 * sequence to `out` (host, [n_heads*head_dim] fp32, widened exactly).  Errors: ARG, CUDA. */
int llma_debug_kv_row(llma_engine *e, int32_t layer, int32_t seq, int32_t pos, int32_t which, float *out);

/* Parity harness only: copy an internal activation buffer of the last forward pass to `out` (host,
 * fp32), rc = llma_row_capacity rows (row r = packed row r of the step).  which = 0: residual stream
 * x [rc][d_model]; 1: qkv [rc][3*n_heads*head_dim] (q rotated; the k and v thirds are only filled on the
 * CUDA-core path); 2: attention output [rc][n_heads*head_dim]; 3: gated FFN activation h [rc][d_ffn].
 * Split bf16 buffers are returned as hi + lo.  `count` must be the buffer's element count.
 * Errors: NULL, ARG, CUDA. */
int llma_debug_buffer(llma_engine *e, int32_t which, float *out, int64_t count);

/*
 * Replay of a given step sequence for one sequence slot, as the paper times its method (Section 3.2,
 * "target guided simulation", Algorithm 2): step i feeds trace[2i] >= 1 input rows (the pending token and
 * the next trace[2i]-1 tokens of `target`) through the real forward pass and then appends trace[2i+1]
 * tokens of `target` (1 <= trace[2i+1] <= trace[2i] <= max_k+1), whatever the model's own outputs are.
 * trace (host, [n_steps][2]); target (host, n_target ids) is the text to reproduce; the trace's emitted
 * counts must sum to n_target.  seq = -1 replays the same trace and target on every prefilled sequence
 * at once (one forward pass per step for all of them); otherwise every other sequence must be idle or
 * finished.  Output tokens are the target's; stats (may be NULL) carry steps, launches and device time.
 * Errors: NULL, ARG, CAPACITY, TOKEN_RANGE, STATE, CUDA, DEVICE_TIMEOUT.
 */
int llma_generate_forced(llma_engine *e, int32_t seq, const int32_t *trace, int32_t n_steps,
                         const int32_t *target, int32_t n_target, llma_stats *stats);

/* Parity harness only: preset the device-side error word (0 none, 1 a bounded wait ran out, 2 capacity,
 * 3 token range), as a kernel that gave up would have left it; the next step reports it.  Errors: ARG, CUDA. */
int llma_debug_set_device_error(llma_engine *e, int32_t code);

/* Measurement aid: in-kernel timestamps of the last decoding step's kernels (globaltimer, ns), copied to `out`
 * (host, 512 x 160 x 8 words) when out != NULL and reset when clear != 0.  Block i < 300 belongs to the i-th
 * projection launch of the step (one 8-word slot per CTA: CTA start, dependency released, first stage ready,
 * last MMA issued, last accumulator ready, CTA end); blocks 300 + layer and 400 + layer hold (min, max) pairs
 * of the attention kernel (CTA start, dependency released, K tile landed, CTA end) and of its merge kernel.
 * Only a library built with -DLLMA_STAMPS records anything; otherwise LLMA_ERR_STATE.  Errors: NULL, STATE, CUDA. */
int llma_debug_timeline(llma_engine *e, int32_t clear, unsigned long long *out);

/* Inspection: how many 128-position tiles of the K/V cache one attention CTA takes in a decoding step of this engine
 * (1, 2 or 4; chosen at llma_create from max_batch, max_seq and the head count alone).  Errors: NULL. */
int llma_debug_attention_tiles(llma_engine *e);

/* Rows the engine's activation buffers hold (the leading dimension of llma_debug_buffer), or a negative
 * status. */
int llma_row_capacity(llma_engine *e);

/* Committed K/V length of a sequence (prompt rows + emitted tokens - 1), or a negative status. */
int llma_kv_len(llma_engine *e, int32_t seq);

/* Kernel classes reported by llma_profile_steps. */
enum {
    LLMA_K_PLAN = 0,      /* trigger search + copy planning (the step-tail kernel launched for the plan alone) */
    LLMA_K_EMBED,         /* embedding gather */
    LLMA_K_NORM,          /* RMSNorm */
    LLMA_K_GEMM_QKV,      /* QKV projection (tensor-core path: + rotary + K/V append) */
    LLMA_K_ATTN,          /* causal attention over the K/V cache */
    LLMA_K_GEMM_O,        /* output projection + residual */
    LLMA_K_GEMM_GATEUP,   /* gate/up projections (tensor-core path: + SiLU gating) */
    LLMA_K_GEMM_DOWN,     /* down projection + residual */
    LLMA_K_GEMM_LMHEAD,   /* LM head (tensor-core path: + per-tile argmax) */
    LLMA_K_ARGMAX,        /* final per-row argmax (CUDA-core path; folded into ACCEPT on the tensor-core path) */
    LLMA_K_ACCEPT,        /* final argmax + acceptance + K/V commit (+ the next step's plan inside llma_generate) */
    LLMA_K_EPILOGUE,      /* separate rotary / gating kernels of the SIMT path */
    LLMA_K_COUNT
};

typedef struct {
    double ms[LLMA_K_COUNT];        /* stream time attributed to each class, summed over the steps */
    int64_t launches[LLMA_K_COUNT]; /* kernel launches of each class */
    int64_t steps;
    double total_ms;
} llma_profile;

/*
 * Measurement aid: run `steps` decoding steps exactly like llma_step (state advances, tokens
 * are appended) but with a CUDA event recorded on the engine's stream after every kernel
 * launch; the time between consecutive events is attributed to the kernel just launched.
 * Launches are direct (no graph), so the figures include the gap to the previous kernel.
 * Errors: as llma_step.
 */
int llma_profile_steps(llma_engine *e, int32_t n, int32_t k, int32_t steps, llma_profile *out);

/*
 * Measurement aid (no counterpart in the paper): the time one tcgen05.mma of the projection kernels' shape
 * (M 128, K 16, bf16 inputs, fp32 accumulator) occupies the tensor core, measured on the current device by one
 * CTA that issues 4 * groups MMAs of width n on operands resident in shared memory, dealt over `regions`
 * accumulator regions of n TMEM columns each, with commits_per_group tcgen05.commit between groups of four.
 * ns_per_mma (host pointer) receives the wall time from the first issue to the completion of the last MMA,
 * divided by the number of MMAs.  Allocates and frees two words of device memory; synchronises the device.
 * Errors: NULL; ARG (n not a multiple of 16 in [16, 256], regions * n > 512, groups outside [1, 65536],
 * commits_per_group outside [0, 4]); CONFIG (not an sm_100 device); CUDA; DEVICE_TIMEOUT.
 */
int llma_microbench_mma(int32_t n, int32_t regions, int32_t groups, int32_t commits_per_group, double *ns_per_mma);

/*
 * The engine's projection kernel on its own: out[r, n] = sum_k W[n, k] * a[r, k] for the 32
 * activation rows a step can hold (Eq. 3 evaluates k+1 <= 32 positions against every weight
 * matrix in one pass).  W: device, bf16, row-major [n_out, k_in]; a: device, bf16, row-major
 * [32, k_in]; out: device, fp32, row-major [32, n_out].  k_in must be a multiple of 64; W and a
 * 16-byte aligned.  Allocates its split-k scratch with cudaMalloc and frees it before returning;
 * synchronous.  Errors: NULL, ARG, CONFIG (not an sm_100 device), CUDA, DEVICE_TIMEOUT.
 */
int llma_gemm_rows32_bf16(const void *W, const void *a, float *out, int32_t n_out, int32_t k_in,
                          void *cuda_stream);

/*
 * The same product as llma_gemm_rows32_bf16 for callers that cannot allocate device memory.
 * (The paper has no counterpart to this entry point; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is forbidden or unsafe -- inside a host
 * process whose memory pool owns the whole GPU and treats any outside allocation as a
 * budget violation, in a latency-critical serving loop where an allocation would serialise
 * the device, or in a plug-in that is only handed pre-allocated buffers.  This call performs
 * no cudaMalloc, cudaFree or any other allocating routine.
 *
 * Arguments, layouts and results are exactly those of llma_gemm_rows32_bf16 (W, a, out are
 * caller-owned device buffers).  The partial tiles handed between CTAs, the error word and the operand
 * staging live in a fixed array of about 7 MiB that is part of the library image: every GPU
 * that loads the library holds it until the process exits.  Limits that follow from its size:
 * n_out <= 262144 and k_in <= 16384; larger sizes return LLMA_ERR_CAPACITY and do nothing.
 *
 * The first call on a device resolves the array's device address (with the caller's current
 * device) and opts the kernel into its shared-memory size.  All calls on a device share the array
 * and it keeps the previous call's contents: the call itself puts the hand-over slots into their
 * empty state and clears the error word, but two calls that overlap on the GPU (different streams,
 * or different threads) race on it and give wrong results -- serialise them.  The call is
 * synchronous: it waits for the kernel and reads its error word back before it returns.
 * Errors: NULL, ARG, CAPACITY, CONFIG (not an sm_100 device), CUDA, DEVICE_TIMEOUT.
 */
int llma_gemm_rows32_bf16_noalloc(const void *W, const void *a, float *out, int32_t n_out, int32_t k_in,
                                  void *cuda_stream);

/* Which GEMM implementation the engine resolved to (LLMA_GEMM_SIMT or LLMA_GEMM_TCGEN05), or a
 * negative status. */
int llma_gemm_impl(llma_engine *e);

/* The CUDA error code behind the most recent LLMA_ERR_CUDA on this thread (0 if none). */
int llma_last_cuda_error(void);

/* Static description of a status code. */
const char *llma_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* LLMA_H_ */

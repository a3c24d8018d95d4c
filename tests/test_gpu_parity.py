"""GPU parity tests: the CUDA engine (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest

from oracle import decoding as D
from oracle import model as OM
from workloads import SHAPES, ModelShape, build_reference, make_prompt, make_weights

from parity import BF16_LOGIT_TOL, step_parity, step_parity_batch

pytestmark = pytest.mark.gpu


def _engine(shape, w, **kw):
    from paper_2304_04487_b200 import Engine
    return Engine(shape, w, **kw)


_cache = {}


def _weights(shape, seed=0, std=0.02):
    key = (shape.name, seed, std)
    if key not in _cache:
        _cache[key] = make_weights(shape, seed=seed, std=std)
    return _cache[key]


def _greedy_star(shape, w, prompt, n_new, max_seq):
    key = ("y*", shape.name, id(w), len(prompt), n_new)
    if key not in _cache:
        _cache[key] = D.greedy_decode(OM.OracleModel(shape, w, max_seq=max_seq), prompt, n_new).tokens
    return _cache[key]


# ---- configuration 1 of the benchmark set: tiny fp32 decoder, n=2, k=4, 64 new tokens ---------------
def test_tiny_fp32_stepwise_parity():
    shape = SHAPES["tiny-fp32"]
    w = _weights(shape)
    prompt = make_prompt(128, shape.vocab, seed=1)
    N, max_seq = 64, 256
    y_star = _greedy_star(shape, w, prompt, N, max_seq)
    ref, offs, info = build_reference(y_star, [256], 0.6, shape.vocab, seed=0)
    eng = _engine(shape, w, max_seq=max_seq, max_ref=256, max_k=4, keep_logits=True)
    rep = step_parity(eng, OM.OracleModel(shape, w, max_seq=max_seq), prompt, ref, offs, 2, 4, N, "fp32")
    assert rep.near_ties == 0
    assert rep.tokens[:N] == y_star                      # lossless: equals the oracle's greedy output
    assert rep.trigger_steps > 5 and rep.copied_accepted > 10, (rep, info)
    assert rep.max_logit_err <= 1e-4 * max(1.0, rep.max_logit_scale)


@pytest.mark.parametrize("name,n,k,P,N", [("tiny-bf16", 1, 8, 70, 48), ("small-bf16", 1, 5, 45, 40),
                                           ("small-bf16", 2, 16, 33, 40), ("mid-bf16", 1, 8, 50, 32),
                                           # contexts spanning several 128-position attention chunks with a ragged tail
                                           ("tiny-bf16", 1, 8, 300, 24), ("small-bf16", 1, 20, 250, 30)])
def test_bf16_stepwise_parity(name, n, k, P, N):
    shape = SHAPES[name]
    w = _weights(shape)
    prompt = make_prompt(P, shape.vocab, seed=2)
    max_seq = P + N + 40
    y_star = _greedy_star(shape, w, prompt, N, max_seq)
    ref, offs, _ = build_reference(y_star, [60, 60, 40], 0.7, shape.vocab, seed=1)
    eng = _engine(shape, w, max_seq=max_seq, max_ref=200, max_k=k, keep_logits=True)
    assert eng.llma_gemm_impl() == 2                     # bf16 shapes run the tensor-core GEMMs
    rep = step_parity(eng, OM.OracleModel(shape, w, max_seq=max_seq), prompt, ref, offs, n, k, N, "bf16")
    assert rep.max_logit_err <= 2e-2
    assert rep.near_ties <= 3, rep.near_ties
    assert rep.trigger_steps > 0


def test_bf16_parity_with_prescribed_cache_codes():
    """The same comparison with the cache's quantisation decisions taken alike on both sides: every code the engine
    stored must be the rounding of a value within 1e-4 of the row scale of the oracle's unrounded value, differing
    codes must be rare, and the logits then agree far inside the tolerance."""
    shape = SHAPES["small-bf16"]
    w = _weights(shape)
    P, N, k = 150, 24, 8
    prompt = make_prompt(P, shape.vocab, seed=2)
    max_seq = P + N + 40
    y_star = _greedy_star(shape, w, prompt, N, max_seq)
    ref, offs, _ = build_reference(y_star, [60, 60, 40], 0.7, shape.vocab, seed=1)
    eng = _engine(shape, w, max_seq=max_seq, max_ref=200, max_k=k, keep_logits=True)
    rep = step_parity(eng, OM.OracleModel(shape, w, max_seq=max_seq), prompt, ref, offs, 1, k, N, "bf16",
                      prescribe_kv=True)
    assert rep.code_violations == 0 and rep.codes_seen > 100000
    assert rep.code_flips <= 0.01 * rep.codes_seen
    assert rep.max_logit_err <= 5e-3 and rep.near_ties <= 1
    eng.llma_destroy()


# ---- the whole loop: llma_generate vs Algorithm 1 on the oracle, LLMA == greedy on the GPU -----------
@pytest.mark.parametrize("name", ["tiny-fp32", "tiny-bf16"])
def test_generate_lossless_and_trace(name):
    shape = SHAPES[name]
    w = _weights(shape)
    prompt = make_prompt(40, shape.vocab, seed=3)
    N, max_seq = 64, 128
    eng = _engine(shape, w, max_seq=max_seq, max_ref=300, max_k=18)
    eng.llma_prefill(0, prompt)
    (g_tokens,), g_stats = eng.llma_generate(N, 1, 0)
    assert len(g_tokens) == N and g_stats.steps == N and g_stats.trigger_steps == 0 and g_stats.tokens == N
    if name == "tiny-fp32":
        assert g_tokens == _greedy_star(shape, w, prompt, N, max_seq)
    # references built from the engine's own greedy output: integer behaviour is then fully
    # determined by (y, D, n, k) and must equal Algorithm 2's model-free prediction
    refs = {
        "spliced": build_reference(g_tokens, [100, 100, 60], 0.8, shape.vocab, seed=4)[:2],
        "self": (np.asarray(g_tokens, np.int32), None),
        "repeats": (np.asarray(g_tokens[5:15] * 3 + g_tokens[30:50] + g_tokens[5:12], np.int32),
                    np.asarray([0, 30, 30, 50, 57], np.int32)),
        "empty": (np.zeros(0, np.int32), None),
    }
    for rname, (ref, offs) in refs.items():
        eng.llma_set_reference(0, ref, offs)
        for n, k in ((1, 4), (1, 8), (2, 3), (3, 18), (1, 1)):
            eng.llma_rewind(0)
            (toks,), st = eng.llma_generate(N, n, k)
            assert toks == g_tokens, (rname, n, k)                       # identical to greedy on the same engine
            sim = D.simulate_decoding_sequence(g_tokens, ref.tolist(), None if offs is None else offs.tolist(), n, k)
            assert st.steps == len(sim), (rname, n, k, st.steps, len(sim))
            assert st.tokens == N == st.steps + st.copied_accepted
            assert st.trigger_steps == sum(1 for i, _ in sim if i > 1)
            assert st.launches > 0 and st.device_ms > 0
    # stepping by hand gives the same per-step (inputs, outputs) sequence as Algorithm 2
    ref, offs = refs["spliced"]
    eng.llma_set_reference(0, ref, offs)
    eng.llma_rewind(0)
    sim = D.simulate_decoding_sequence(g_tokens, ref.tolist(), offs.tolist(), 1, 6)
    # (llma_step has no output budget of its own; far from the end of y that makes no difference)
    got, out = [], []
    while len(out) < 20:
        t = eng.llma_step(1, 6)[0]
        i = eng.llma_last_step_info()[0]
        got.append((1 + i.k_eff, i.emitted)); out += t
    assert out == g_tokens[:len(out)]
    assert got == sim[:len(got)]


def test_logits_bitwise_independent_of_k():
    """Rows of a (k+1)-row verification step must be bit-identical to the rows that one-token
    greedy steps compute at the same positions."""
    for name in ("tiny-fp32", "small-bf16"):
        shape = SHAPES[name]
        w = _weights(shape)
        prompt = make_prompt(37, shape.vocab, seed=5)
        N, max_seq = 24, 96
        eng = _engine(shape, w, max_seq=max_seq, max_ref=64, max_k=16, keep_logits=True)
        eng.llma_prefill(0, prompt)
        rows_greedy, toks = [], []
        for _ in range(N):
            toks += eng.llma_step(1, 0)[0]
            rows_greedy.append(eng.llma_debug_logits()[0].copy())
        eng.llma_set_reference(0, toks, None)
        for k in (1, 4, 7, 16):
            eng.llma_rewind(0)
            i = 0
            while i < N - 17:
                t = eng.llma_step(1, k)[0]
                lg = eng.llma_debug_logits()
                for j in range(len(t)):
                    assert np.array_equal(lg[j].view(np.uint32), rows_greedy[i + j].view(np.uint32)), (name, k, i, j)
                assert t == toks[i:i + len(t)]
                i += len(t)
        # run twice: same bits (no race in any reduction)
        eng.llma_rewind(0)
        eng.llma_step(1, 0); a = eng.llma_debug_logits()[0].copy()
        eng.llma_rewind(0)
        eng.llma_step(1, 0); b = eng.llma_debug_logits()[0].copy()
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_kv_rows_match_oracle():
    shape = SHAPES["small-bf16"]
    w = _weights(shape)
    prompt = make_prompt(40, shape.vocab, seed=6)
    eng = _engine(shape, w, max_seq=64, max_ref=8, max_k=0)
    om = OM.OracleModel(shape, w, max_seq=64)
    eng.llma_prefill(0, prompt)
    D.prefill(om, prompt)
    for layer in (0, shape.n_layers - 1):
        for pos in (0, 17, 31, 32, 38):
            for which in (0, 1):
                got = eng.llma_debug_kv_row(layer, 0, pos, which)
                want = om.read_cache(layer, pos, which)
                # bf16 rows: the engine feeds bf16 activations to its matrix products, so rows agree
                # to a couple of steps of the stored type rather than bit for bit
                assert np.abs(got - want).max() <= 2.0 ** -7 * max(1e-3, np.abs(want).max())


def test_two_sequences_ragged():
    shape = SHAPES["tiny-bf16"]
    w = _weights(shape)
    N, max_seq = 40, 128
    prompts = [make_prompt(30, shape.vocab, seed=7), make_prompt(51, shape.vocab, seed=8)]
    singles = []
    for p in prompts:
        e1 = _engine(shape, w, max_seq=max_seq, max_ref=128, max_k=7)
        e1.llma_prefill(0, p)
        (t,), _ = e1.llma_generate(N, 1, 0)
        singles.append(t)
    eng = _engine(shape, w, max_seq=max_seq, max_ref=128, max_k=7, max_batch=2)
    for s, p in enumerate(prompts):
        eng.llma_prefill(s, p)
    eng.llma_set_reference(0, singles[0][4:30], None)
    eng.llma_set_reference(1, build_reference(singles[1], [64, 64], 0.6, shape.vocab, seed=9)[0], [0, 64, 128])
    toks, st = eng.llma_generate(N, 1, 7)
    assert toks[0] == singles[0] and toks[1] == singles[1]        # each sequence unaffected by its neighbour
    assert st.tokens == 2 * N and st.copied_accepted > 0
    infos = eng.llma_last_step_info()
    assert len(infos) == 2


@pytest.mark.parametrize("name,B,k", [("tiny-bf16", 16, 8),     # 144 rows: the multi-turn serving shape (16 x (8+1))
                                      ("small-bf16", 5, 6),     # 35 rows, head_dim 128
                                      ("tiny-fp32", 4, 4)])     # CUDA-core path, 20 rows
def test_batched_ragged_stepwise_parity(name, B, k):
    """Several sequences of different lengths, references and overlaps decoded in one forward pass per
    step; every sequence is checked against an oracle run of its own (trace, logits, tokens)."""
    shape = SHAPES[name]
    w = _weights(shape)
    N = 20
    prompts = [make_prompt(18 + 7 * s, shape.vocab, seed=20 + s) for s in range(B)]
    max_seq = max(len(p) for p in prompts) + N + 2 * k + 8
    refs, offs_list, models = [], [], []
    for s in range(B):
        y_star = D.greedy_decode(OM.OracleModel(shape, w, max_seq=max_seq), prompts[s], N).tokens
        if s % 5 == 4:
            ref, offs = np.zeros(0, np.int32), None                       # a sequence with no reference: plain greedy
        else:
            ref, offs, _ = build_reference(y_star, [30, 34], 0.5 + 0.1 * (s % 5), shape.vocab, seed=s)
        refs.append(ref); offs_list.append(offs)
        models.append(OM.OracleModel(shape, w, max_seq=max_seq))
    eng = _engine(shape, w, max_seq=max_seq, max_ref=64, max_k=k, max_batch=B, keep_logits=True)
    mode = "fp32" if shape.dtype == "fp32" else "bf16"
    reps = step_parity_batch(eng, models, prompts, refs, offs_list, 1, k, N, mode)
    assert sum(r.trigger_steps for r in reps) > B and sum(r.copied_accepted for r in reps) > 2 * B
    assert sum(r.near_ties for r in reps) <= 3
    for s in range(B):
        assert reps[s].max_logit_err <= (2e-2 if mode == "bf16" else 1e-4 * max(1.0, reps[s].max_logit_scale))
        if s % 5 == 4:
            assert reps[s].trigger_steps == 0 and reps[s].steps == len(reps[s].tokens)
    eng.llma_destroy()


@pytest.mark.parametrize("name,B,k_max,adaptive", [("tiny-bf16", 6, 16, (1, 2)), ("tiny-fp32", 3, 8, (2, 4))])
def test_adaptive_copy_length_stepwise_parity(name, B, k_max, adaptive):
    """The adaptive copy length (a variant beyond the paper): every step's plan must be the one the oracle's
    rule gives, per sequence, and llma_generate over the whole loop must follow the oracle's trace too."""
    from paper_2304_04487_b200 import LlmaError
    shape = SHAPES[name]
    w = _weights(shape)
    N = 40
    prompts = [make_prompt(15 + 6 * s, shape.vocab, seed=60 + s) for s in range(B)]
    max_seq = max(len(p) for p in prompts) + N + 2 * k_max + 8
    refs, offs_list, models = [], [], []
    for s in range(B):
        y_star = D.greedy_decode(OM.OracleModel(shape, w, max_seq=max_seq), prompts[s], N).tokens
        ref, offs, _ = build_reference(y_star, [40, 40], 0.6 + 0.08 * s, shape.vocab, seed=70 + s)
        refs.append(ref); offs_list.append(offs)
        models.append(OM.OracleModel(shape, w, max_seq=max_seq))
    eng = _engine(shape, w, max_seq=max_seq, max_ref=80, max_k=k_max, max_batch=B, keep_logits=True)
    mode = "fp32" if shape.dtype == "fp32" else "bf16"
    reps = step_parity_batch(eng, models, prompts, refs, offs_list, 1, k_max, N, mode, adaptive=adaptive)
    assert sum(r.trigger_steps for r in reps) > B and sum(r.copied_accepted for r in reps) > 2 * B
    for r in reps:
        assert r.max_logit_err <= (2e-2 if mode == "bf16" else 1e-4 * max(1.0, r.max_logit_scale))
    # the whole loop on the device: sequence 0 alone after a rewind, against the oracle's adaptive decode
    for s in range(1, B):
        eng.llma_reset(s)
    eng.llma_rewind(0)                                            # keeps the setting, k_cur back to k_start
    outs, st = eng.llma_generate(N, 1, k_max)
    got = outs[0]
    want = D.llma_decode(OM.OracleModel(shape, w, max_seq=max_seq), prompts[0], refs[0], offs_list[0], 1, k_max, N,
                         adaptive=(adaptive[0], adaptive[1], k_max))
    fixed = D.llma_decode(OM.OracleModel(shape, w, max_seq=max_seq), prompts[0], refs[0], offs_list[0], 1, k_max, N)
    assert list(got) == want.tokens == fixed.tokens
    assert (st.steps, st.trigger_steps, st.copied_accepted) == (want.steps, want.trigger_steps, want.copied_accepted)
    assert want.steps != fixed.steps or [r.k_eff for r in want.trace] != [r.k_eff for r in fixed.trace]
    # switched off again: the fixed-k trace
    eng.llma_set_adaptive_k(0, 0, 0)
    eng.llma_rewind(0)
    outs, st = eng.llma_generate(N, 1, k_max)
    got = outs[0]
    assert list(got) == fixed.tokens and st.steps == fixed.steps
    for bad in ((0, 3), (3, 2), (1, k_max + 1), (-1, 2)):
        with pytest.raises(LlmaError):
            eng.llma_set_adaptive_k(0, *bad)
    eng.llma_destroy()


@pytest.mark.parametrize("name,max_seq,tiles", [("tiny-bf16", 5000, 2), ("tiny-bf16", 7300, 4), ("small-bf16", 7300, 4)])
def test_long_context_batch_attention_tiles(name, max_seq, tiles):
    """Engines whose capacity makes an attention CTA take several K/V tiles in a row (many sequences, long max_seq):
    stepwise parity of 16 sequences whose contexts span one to several such chunks, ragged tails included
    (head_dim 64 and 128)."""
    shape = SHAPES[name]
    w = _weights(shape)
    B, k, N = 16, 4, 10
    prompts = [make_prompt(90 + 61 * s, shape.vocab, seed=80 + s) for s in range(B)]     # 90 .. 1005 cached positions
    refs, offs_list, models = [], [], []
    o_seq = max(len(p) for p in prompts) + N + 2 * k + 8
    for s in range(B):
        y_star = D.greedy_decode(OM.OracleModel(shape, w, max_seq=o_seq), prompts[s], N).tokens
        ref, offs, _ = build_reference(y_star, [24], 0.7, shape.vocab, seed=90 + s)
        refs.append(ref); offs_list.append(offs)
        models.append(OM.OracleModel(shape, w, max_seq=o_seq))
    eng = _engine(shape, w, max_seq=max_seq, max_ref=32, max_k=k, max_batch=B, keep_logits=True)
    assert eng.llma_debug_attention_tiles() == tiles
    reps = step_parity_batch(eng, models, prompts, refs, offs_list, 1, k, N, "bf16")
    assert sum(r.trigger_steps for r in reps) > 4
    assert sum(r.near_ties for r in reps) <= 3
    for r in reps:
        assert r.max_logit_err <= 2e-2
    eng.llma_destroy()


def test_batched_generate_equals_single_sequence_runs():
    """llma_generate over 16 sequences: each output equals what the same sequence gives alone (greedy on a
    one-sequence engine), and the whole-loop statistics add up."""
    shape = SHAPES["tiny-bf16"]
    w = _weights(shape)
    B, N, k = 16, 40, 8
    prompts = [make_prompt(25 + 9 * s, shape.vocab, seed=40 + s) for s in range(B)]
    max_seq = 25 + 9 * B + N + 32
    singles = []
    e1 = _engine(shape, w, max_seq=max_seq, max_ref=8, max_k=0)
    for p in prompts:
        e1.llma_reset(0)
        e1.llma_prefill(0, p)
        (t,), _ = e1.llma_generate(N, 1, 0)
        singles.append(t)
    e1.llma_destroy()
    eng = _engine(shape, w, max_seq=max_seq, max_ref=128, max_k=k, max_batch=B)
    for s, p in enumerate(prompts):
        eng.llma_prefill(s, p)
        ref, offs, _ = build_reference(singles[s], [64, 64], 0.7 + 0.02 * (s % 10), shape.vocab, seed=s)
        eng.llma_set_reference(s, ref, offs)
    toks, st = eng.llma_generate(N, 1, k)
    for s in range(B):
        assert toks[s] == singles[s], s
    assert st.tokens == B * N == st.steps + st.copied_accepted and st.trigger_steps > B
    eng.llma_destroy()


def test_device_timeout_is_reported_and_engine_recovers():
    """A kernel whose bounded wait ran out leaves a code in the device error word; here the word is preset
    through the debug hook (no wait is made to run out on the GPU).  The step must report it, and the steps
    after it must be those of an undisturbed run."""
    from paper_2304_04487_b200 import LlmaError
    shape = SHAPES["tiny-bf16"]
    w = _weights(shape)
    prompt = make_prompt(30, shape.vocab, seed=50)
    eng = _engine(shape, w, max_seq=96, max_ref=8, max_k=4)
    eng.llma_prefill(0, prompt)
    (want,), _ = eng.llma_generate(6, 1, 0)
    eng.llma_rewind(0)
    got = eng.llma_step(1, 0)[0]
    eng.llma_debug_set_device_error(1)
    with pytest.raises(LlmaError) as ei:
        eng.llma_step(1, 0)
    assert ei.value.status == -8
    for _ in range(4):
        got += eng.llma_step(1, 0)[0]
    # the flagged step itself ran (only its report was forced), so the run continues from token 3
    assert got == [want[0]] + want[2:6]
    for code, status in ((2, -4), (3, -3)):
        eng.llma_debug_set_device_error(code)
        with pytest.raises(LlmaError) as ei:
            eng.llma_step(1, 0)
        assert ei.value.status == status
    eng.llma_destroy()


@pytest.mark.parametrize("name", ["tiny-bf16", "tiny-fp32"])
def test_forced_replay_follows_algorithm2_trace(name):
    """Section 3.2's measurement device: the engine is driven along the (inputs, outputs) sequence that
    Algorithm 2 derives from a target text and the references, and must reproduce the target with exactly
    those steps; the K/V rows it leaves behind are real, so ordinary decoding can go on afterwards."""
    shape = SHAPES[name]
    w = _weights(shape)
    prompt = make_prompt(33, shape.vocab, seed=60)
    N, k, max_seq = 48, 6, 128
    eng = _engine(shape, w, max_seq=max_seq, max_ref=128, max_k=k)
    eng.llma_prefill(0, prompt)
    (y_star,), _ = eng.llma_generate(N + 5, 1, 0)
    ref, offs, _ = build_reference(y_star[:N], [60, 60], 0.7, shape.vocab, seed=3)
    trace = D.simulate_decoding_sequence(y_star[:N], ref.tolist(), offs.tolist(), 1, k)
    assert sum(o for _, o in trace) == N and max(i for i, _ in trace) > 1
    eng.llma_rewind(0)
    st = eng.llma_generate_forced(0, trace, y_star[:N])
    assert st.steps == len(trace) and st.tokens == N and st.copied_accepted == N - len(trace)
    assert eng.llma_kv_len(0) == len(prompt) - 1 + N
    # the cache now holds the target's rows: greedy decoding continues with the engine's own next tokens
    (more,), _ = eng.llma_generate(5, 1, 0)
    assert more == y_star[N:N + 5]
    # a real LLMA decode of the same text takes the same steps (Algorithm 2 predicts Algorithm 1)
    eng.llma_set_reference(0, ref, offs)
    eng.llma_rewind(0)
    (toks,), st2 = eng.llma_generate(N, 1, k)
    assert toks == y_star[:N] and st2.steps == len(trace)
    eng.llma_destroy()


@pytest.mark.parametrize("name,k", [("llama13b-2layer", 8),      # 13B widths: d 5120, 40 heads, F 13824
                                    ("llama7b-2layer", 16)])     # 7B widths in the 32-row MMA shape
def test_wide_two_layer_stepwise_parity(name, k):
    """The widths of the large benchmark shapes on two layers, which the oracle steps through in seconds:
    every projection is split over many CTAs along k exactly as in the full-depth model."""
    shape = SHAPES[name]
    w = _weights(shape)
    P, N = 24, 20
    prompt = make_prompt(P, shape.vocab, seed=12)
    max_seq = 96
    y_star = _greedy_star(shape, w, prompt, N, max_seq)
    ref, offs, _ = build_reference(y_star, [40, 40], 0.8, shape.vocab, seed=2)
    eng = _engine(shape, w, max_seq=max_seq, max_ref=80, max_k=k, keep_logits=True)
    assert eng.llma_gemm_impl() == 2
    rep = step_parity(eng, OM.OracleModel(shape, w, max_seq=max_seq), prompt, ref, offs, 1, k, N, "bf16")
    assert rep.max_logit_err <= 2e-2
    assert rep.trigger_steps > 0 and rep.copied_accepted > 0
    assert rep.tokens[:N] == y_star or rep.near_ties > 0
    eng.llma_destroy()
    _cache.clear()


def test_llama7b_shape_sampled_parity():
    """Full-size check in the configuration the benchmark times (7B-shaped bf16 decoder, engine created
    for k = 8): a short prompt, then LLMA steps whose every logits row is compared with the oracle.  The
    oracle needs about a second per position at this size, so only a few dozen positions are sampled.

    Two runs.  (1) Both sides take the cache's quantisation decisions alike (the oracle adopts the engine's bf16
    code wherever it is the rounding of a value within 1e-4 of the row scale of its own unrounded value): logits
    within the flat 2e-2, no code outside that rule, differing codes rare.  (2) Free-running: every layer's flips feed
    the next layer, the effect on the logits grows with depth (about 2.4e-2 at 32 layers with tensor-core
    accumulation, 1.3e-2 with fp32 FMA accumulation, unchanged by a third bf16 term of the activations); the
    figure is printed, tokens must still agree except at near-ties."""
    shape = SHAPES["llama7b-shape"]
    w = _weights(shape)
    prompt = make_prompt(20, shape.vocab, seed=11)
    max_seq = 64
    om = OM.OracleModel(shape, w, max_seq=max_seq)
    y_star = D.greedy_decode(om, prompt, 10).tokens                     # 29 oracle positions
    ref = y_star[:8] + [shape.vocab - 1, shape.vocab - 2]                 # one span that is accepted, then junk
    eng = _engine(shape, w, max_seq=max_seq, max_ref=32, max_k=8, keep_logits=True)
    assert eng.llma_gemm_impl() == 2
    rep = step_parity(eng, OM.OracleModel(shape, w, max_seq=max_seq), prompt, ref, None, 1, 8, 10, "bf16",
                      prescribe_kv=True)
    assert rep.max_logit_err <= BF16_LOGIT_TOL
    assert rep.code_violations == 0
    assert rep.code_flips <= 0.05 * rep.codes_seen                        # about 2 % at these widths (k = 4096 products per element)
    assert rep.rows_compared >= 10 and rep.trigger_steps >= 1 and rep.copied_accepted >= 4
    assert rep.tokens[:10] == y_star or rep.near_ties > 0
    eng.llma_reset(0)
    free = step_parity(eng, OM.OracleModel(shape, w, max_seq=max_seq), prompt, ref, None, 1, 8, 10, "bf16",
                       check_logits=False)
    assert free.tokens[:10] == y_star or free.near_ties > 0
    assert free.max_logit_err <= 5e-2                                     # a gross error would not hide behind the drift
    print(f"7B-shape parity: rows {rep.rows_compared}; cache codes prescribed: max |dlogit| {rep.max_logit_err:.2e}, "
          f"{rep.code_flips} of {rep.codes_seen} codes differ ({rep.code_boundary_dist:.2f} of the code tolerance used); "
          f"free-running: max |dlogit| {free.max_logit_err:.2e}, near ties {free.near_ties}")
    _cache.clear()                                                        # 13 GB of host weights

"""Pins for the CPU oracle: everything here checks the oracle against something
other than itself (closed forms, invariants, brute force, the paper's printed
numbers, an independent library implementation).  No GPU involved."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import decoding as D
from oracle import model as OM
from workloads import ModelShape, make_weights, make_prompt, bf16_bits_from_f32, f32_from_bf16_bits

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

MICRO = ModelShape("micro-fp32", 2, 64, 2, 32, 128, 97, "fp32")
MICRO_BF16 = ModelShape("micro-bf16", 2, 64, 2, 32, 128, 97, "bf16")


# --------------------------------------------------------------------------------------
# scripted models: look-up tables instead of a network
# --------------------------------------------------------------------------------------
class ScriptedModel:
    """Emits target[j] at position base+j if the token fed there is the true
    previous token (the last prompt token for j = 0, else target[j-1]); any other
    input yields the junk id, as a real model conditioned on a wrong token would
    produce an unrelated output."""

    def __init__(self, target, base, first_input, vocab, junk=0):
        self.target, self.base, self.first, self.vocab, self.junk = list(target), base, first_input, vocab, junk
        self.calls = []

    def forward(self, token, pos, want_logits=True):
        self.calls.append((token, pos))
        if not want_logits:
            return None
        j = pos - self.base
        lg = np.zeros(self.vocab, np.float32)
        if 0 <= j < len(self.target):
            expect = self.first if j == 0 else self.target[j - 1]
            lg[self.target[j] if token == expect else self.junk] = 1.0
        else:
            lg[self.junk] = 1.0
        return lg


def scripted_run(target, ref, offs, n, k, vocab=50):
    prompt = [7, 8, 9]
    m = ScriptedModel(target, len(prompt) - 1, prompt[-1], vocab)
    return D.llma_decode(m, prompt, ref, offs, n, k, len(target)), m


# --------------------------------------------------------------------------------------
# P5: the worked example of Figure 2
# --------------------------------------------------------------------------------------
def test_fig2_worked_example():
    # ids stand for words: 11 "from", 12 "the", 21.. "pancreases cows or pigs .", 30 "Pork", 31 "Until"
    span = [21, 22, 23, 24, 25]
    target = [40, 41, 11, 12] + span + [31, 42, 43]
    ref = [60, 61, 11, 12] + span + [30, 62, 63]
    res, _ = scripted_run(target, ref, None, n=2, k=6)
    assert res.tokens == target
    # steps: 4 plain ones ("from the" must first be generated), then the copy step
    copy = res.trace[4]
    assert [r.emitted for r in res.trace[:4]] == [1, 1, 1, 1]
    assert copy.matched and copy.pos == 4 and copy.k_eff == 6
    assert copy.accepted == 5           # "pancreases cows or pigs ." accepted, "Pork" rejected
    assert copy.emitted == 6            # five accepted copies + the model's own "Until"


# --------------------------------------------------------------------------------------
# P7: trigger search against brute force over the definition
# --------------------------------------------------------------------------------------
def brute_match(y, ref, offs, n):
    i = len(y)
    docs = [(0, len(ref))] if offs is None else [(offs[j], offs[j + 1]) for j in range(len(offs) - 1)]
    cands = []
    for (s, e) in docs:
        for pos in range(s, e):
            for t in range(n, i + 1):
                if pos - t >= s and list(ref[pos - t:pos]) == list(y[i - t:i]):
                    cands.append((t, -pos))
    if not cands:
        return False, -1, 0
    t, negpos = max(cands)
    return True, -negpos, t


def test_match_ngrams_bruteforce():
    rng = np.random.default_rng(5)
    n_match = 0
    for trial in range(400):
        alpha = int(rng.integers(2, 5))
        R = int(rng.integers(0, 30))
        ref = rng.integers(0, alpha, R).tolist()
        if rng.random() < 0.5 and R > 2:
            cuts = sorted(set(rng.integers(0, R + 1, int(rng.integers(1, 4))).tolist()))
            offs = [0] + [c for c in cuts if 0 < c < R] + [R]
        else:
            offs = None
        y = rng.integers(0, alpha, int(rng.integers(0, 12))).tolist()
        n = int(rng.integers(1, 4))
        got = D.match_ngrams(y, ref, offs, n)
        want = brute_match(y, ref, offs, n)
        assert got == want, (y, ref, offs, n)
        n_match += got[0]
    assert n_match > 100  # the small alphabets really do produce matches and ties


def test_match_ngrams_edges():
    assert D.match_ngrams([], [1, 2, 3], None, 1) == (False, -1, 0)
    assert D.match_ngrams([1], [1, 2, 3], None, 2) == (False, -1, 0)        # fewer than n generated
    assert D.match_ngrams([3], [1, 2, 3], None, 1) == (False, -1, 0)        # nothing follows the match
    assert D.match_ngrams([2], [1, 2, 3], None, 1) == (True, 2, 1)
    assert D.match_ngrams([1, 2], [1, 2, 3, 9, 2, 5], None, 1) == (True, 2, 2)   # longer backward agreement wins
    assert D.match_ngrams([2], [2, 3, 2, 5], None, 1) == (True, 1, 1)       # tie -> smallest position
    # spans do not cross documents: "1 2" straddles the boundary between the two docs
    assert D.match_ngrams([1, 2], [0, 1, 2, 3], [0, 2, 4], 2) == (False, -1, 0)
    assert D.match_ngrams([1, 2], [0, 1, 2, 3], [0, 2, 4], 1) == (True, 3, 1)


def test_copy_length_by_hand():
    """k_eff = min(k, tokens left in the matched document, tokens still to emit - 1): every
    expectation below is worked out by hand from that sentence (Section 2.2: the copied span
    lies inside one reference document; Algorithm 1 emits exactly N tokens)."""
    offs = [0, 6, 10]                                   # documents [0, 6) and [6, 10)
    assert D.copy_length(4, 10, offs, 8, 100) == 2      # positions 4, 5 are left in the first document
    assert D.copy_length(5, 10, offs, 8, 100) == 1
    assert D.copy_length(6, 10, offs, 8, 100) == 4      # first position of the second document: 6..9
    assert D.copy_length(9, 10, offs, 8, 100) == 1
    assert D.copy_length(1, 10, offs, 3, 100) == 3      # k is the binding term
    assert D.copy_length(1, 10, offs, 8, 3) == 2        # three tokens to go: one comes from the model anyway
    assert D.copy_length(1, 10, offs, 8, 1) == 0        # last token: nothing to copy
    assert D.copy_length(4, 10, None, 8, 100) == 6      # a single document runs to the end
    assert D.copy_length(0, 10, [0, 0, 10], 20, 100) == 10   # an empty document in front changes nothing
    assert D.copy_length(10, 10, offs, 8, 100) == 0     # past the end: no document holds the position


def test_copy_stops_at_document_boundary_scripted():
    """The reference continues with the CORRECT next tokens across a document boundary; a copy
    that ran on into the second document would be accepted whole (and would still be lossless),
    so only the hand-written trace below can tell the two readings apart."""
    target = [11, 12, 13, 14, 15, 16, 17, 18, 19, 20]
    ref = [11, 12, 13, 14] + [15, 16, 17, 18, 19, 20]   # same text, cut into two documents after 14
    offs = [0, 4, 10]
    res, model = scripted_run(target, ref, offs, n=1, k=8)
    assert res.tokens == target
    # step 1: y empty, no trigger: emits 11.  step 2: "11" matches at pos 1; three tokens (12, 13, 14)
    # are left in document one: k_eff = 3, all accepted, plus the model's own 15.  step 3: "15" matches
    # at pos 5 in document two; five tokens left there but only 10 - 5 - 1 = 4 may be copied: 16..19
    # accepted, plus the model's own 20.
    assert [(r.pos, r.k_eff, r.accepted, r.emitted) for r in res.trace] == [(-1, 0, 0, 1), (1, 3, 3, 4), (5, 4, 4, 5)]
    assert D.simulate_decoding_sequence(target, ref, offs, 1, 8) == [(1, 1), (4, 4), (5, 5)]
    # the model saw exactly those inputs, one position at a time, in order (prompt [7, 8, 9]: base 2)
    assert model.calls[2:] == [(9, 2), (11, 3), (12, 4), (13, 5), (14, 6), (15, 7), (16, 8), (17, 9), (18, 10), (19, 11)]
    # the same text as ONE document is copied straight through: 1 + min(8, 9, 8) + ... = two steps
    res1, _ = scripted_run(target, ref, None, n=1, k=8)
    assert [(r.pos, r.k_eff, r.accepted, r.emitted) for r in res1.trace] == [(-1, 0, 0, 1), (1, 8, 8, 9)]


# --------------------------------------------------------------------------------------
# P1/P2/P3/P4/P6 on scripted models (any target, any reference)
# --------------------------------------------------------------------------------------
def ngram_absent_count(y, ref, offs, n):
    """# of i with y[i-n:i] not an n-gram (inside one doc) of the reference, i < n included."""
    docs = [(0, len(ref))] if offs is None else [(offs[j], offs[j + 1]) for j in range(len(offs) - 1)]
    grams = set()
    for (s, e) in docs:
        for p in range(s + n, e + 1):
            grams.add(tuple(ref[p - n:p]))
    return sum(1 for i in range(len(y)) if i < n or tuple(y[i - n:i]) not in grams)


@pytest.mark.parametrize("seed", range(6))
def test_loop_invariants_scripted(seed):
    rng = np.random.default_rng(seed)
    N = 60
    target = rng.integers(1, 6, N).tolist()                    # small alphabet: many matches
    pieces = []
    for _ in range(6):
        a = int(rng.integers(0, N - 8)); pieces += target[a:a + int(rng.integers(3, 12))]
        pieces += rng.integers(1, 6, int(rng.integers(0, 4))).tolist()
    ref = pieces
    offs = [0, len(ref) // 3, len(ref)]
    base_nontrigger = {}
    for n, k in itertools.product((1, 2, 3), (0, 1, 2, 4, 7, 18)):
        res, m = scripted_run(target, ref, offs, n, k, vocab=8)
        assert res.tokens == target                                            # P1 lossless
        assert len(res.tokens) == res.steps + res.copied_accepted               # P2
        assert all(1 <= r.emitted <= k + 1 and r.emitted == r.accepted + 1 for r in res.trace)
        assert all(r.k_eff <= k for r in res.trace)
        sim = D.simulate_decoding_sequence(target, ref, offs, n, k)             # P4
        assert sim == [(1 + r.k_eff, r.emitted) for r in res.trace]
        if k == 0:
            assert res.steps == N and res.trigger_steps == 0                   # P6: k = 0 is greedy
        else:
            # P3: a step that does not trigger starts where the preceding n-gram has no usable
            # occurrence in the reference (or at the very last token, where nothing may be copied),
            # and every such position does start a step -- whatever k is.
            docs = [(offs[j], offs[j + 1]) for j in range(len(offs) - 1)]
            usable = {tuple(ref[p - n:p]) for (s_, e_) in docs for p in range(s_ + n, e_)}
            starts, i = [], 0
            for r in res.trace:
                starts.append((i, r.matched)); i += r.emitted
            for i, matched in starts:
                absent = i < n or tuple(target[i - n:i]) not in usable
                assert matched == (not absent and i < N - 1), (n, k, i)
            present = {tuple(ref[p - n:p]) for (s_, e_) in docs for p in range(s_ + n, e_ + 1)}
            must_start = {i for i in range(N) if i < n or tuple(target[i - n:i]) not in present}
            assert must_start <= {i for i, _ in starts}
            base_nontrigger.setdefault(n, must_start)
            assert base_nontrigger[n] == must_start
        # the model was called once per fed token at consecutive positions
        pos_calls = [p for (_, p) in m.calls[2:]]
        assert pos_calls[0] == 2


# --------------------------------------------------------------------------------------
# the adaptive copy length (a variant beyond the paper) and the trigger fall-back identity
# --------------------------------------------------------------------------------------
def test_next_copy_request_by_hand():
    f = D.next_copy_request
    assert f(4, 0, 0, 1, 16) == 4        # nothing copied: unchanged
    assert f(4, 4, 4, 1, 16) == 8        # accepted in full: doubled
    assert f(4, 2, 2, 1, 16) == 8        # ... also when the document end had cut the copy short
    assert f(12, 12, 12, 1, 16) == 16    # capped
    assert f(5, 5, 1, 1, 16) == 3        # cut short: halved, rounding up
    assert f(3, 3, 0, 2, 16) == 2
    assert f(2, 2, 1, 2, 16) == 2        # never below k_min
    assert f(1, 1, 0, 1, 16) == 1


def test_adaptive_copy_length_trace_by_hand():
    # the reference repeats the target except for one token (index 6: 40 instead of 16)
    target = list(range(10, 26))
    ref = target[:6] + [40] + target[7:]
    prompt = [7, 8, 9]
    m = ScriptedModel(target, len(prompt) - 1, prompt[-1], 50)
    res = D.llma_decode(m, prompt, ref, None, 1, 8, len(target), adaptive=(1, 2, 8))
    assert res.tokens == target
    # step by step: nothing generated yet; 2 asked, both accepted (-> 4); 4 asked, the third is the changed
    # token (-> 2); "16" is nowhere in the reference; 2 asked, both accepted (-> 4); 4 asked and accepted
    assert [(r.pos, r.k_eff, r.accepted) for r in res.trace] == [
        (-1, 0, 0), (1, 2, 2), (4, 4, 2), (-1, 0, 0), (8, 2, 2), (11, 4, 4)]
    # the same run at the fixed k = 8 needs fewer steps but feeds more rows
    fixed, _ = scripted_run(target, ref, None, 1, 8, vocab=50)
    assert [(r.k_eff, r.accepted) for r in fixed.trace] == [(0, 0), (8, 5), (0, 0), (7, 7)]


@pytest.mark.parametrize("seed", range(4))
def test_adaptive_copy_length_invariants(seed):
    rng = np.random.default_rng(100 + seed)
    N = 70
    target = rng.integers(1, 6, N).tolist()
    ref = []
    for _ in range(6):
        a = int(rng.integers(0, N - 10)); ref += target[a:a + int(rng.integers(3, 14))]
        ref += rng.integers(1, 6, int(rng.integers(0, 3))).tolist()
    offs = [0, len(ref) // 2, len(ref)]
    prompt = [7, 8, 9]
    for n, (k_min, k_start, k_cap) in itertools.product((1, 2), ((1, 1, 8), (2, 4, 8), (1, 8, 8), (3, 3, 12))):
        m = ScriptedModel(target, len(prompt) - 1, prompt[-1], 8)
        res = D.llma_decode(m, prompt, ref, offs, n, k_cap, N, adaptive=(k_min, k_start, k_cap))
        assert res.tokens == target                                   # still the greedy output
        k_cur = k_start
        for r in res.trace:
            assert r.k_eff <= k_cur and k_min <= k_cur <= k_cap      # never more than was asked for
            k_cur = D.next_copy_request(k_cur, r.k_eff, r.accepted, k_min, k_cap)
    # pinned at one value the variant is the fixed-k algorithm
    for k in (1, 5):
        m = ScriptedModel(target, len(prompt) - 1, prompt[-1], 8)
        res = D.llma_decode(m, prompt, ref, offs, 1, k, N, adaptive=(k, k, k))
        fixed, _ = scripted_run(target, ref, offs, 1, k, vocab=8)
        assert res.trace == fixed.trace


def test_trigger_fallback_is_the_shorter_trigger():
    """Trying triggers of length n, n-1, ..., n_lo in turn finds what a trigger of length n_lo finds."""
    rng = np.random.default_rng(5)
    for _ in range(300):
        ref = rng.integers(1, 4, int(rng.integers(4, 30))).tolist()
        y = rng.integers(1, 4, int(rng.integers(0, 12))).tolist()
        offs = [0, int(rng.integers(1, len(ref))), len(ref)]
        for n, n_lo in ((3, 1), (3, 2), (2, 1)):
            chain = (False, -1, 0)
            for nn in range(n, n_lo - 1, -1):
                chain = D.match_ngrams(y, ref, offs, nn)
                if chain[0]:
                    break
            assert chain == D.match_ngrams(y, ref, offs, n_lo)


def test_nontrigger_steps_match_bruteforce_count():
    rng = np.random.default_rng(11)
    N = 80
    target = rng.integers(1, 9, N).tolist()
    # reference ends with ids that never occur in the target so "no room after the match" cannot happen
    ref = target[5:30] + [20, 21] + target[40:70] + [22, 23]
    for n in (1, 2, 3):
        for k in (2, 5, 9):
            # make N unreachable by the last-token cap: extend the target's tail with unmatched ids
            tgt = target + [30, 31, 32, 33]
            res, _ = scripted_run(tgt, ref, None, n, k, vocab=40)
            assert res.steps - res.trigger_steps == ngram_absent_count(tgt, ref, None, n)


def test_special_references():
    rng = np.random.default_rng(3)
    target = rng.permutation(np.arange(1, 41)).tolist()        # all tokens distinct
    # reference = the output itself, n = 1: every triggered step accepts everything it copied
    res, _ = scripted_run(target, target, None, 1, 4)
    assert res.tokens == target
    assert all(r.accepted == r.k_eff for r in res.trace if r.matched)
    assert res.trace[0].matched is False and all(r.matched for r in res.trace[1:] if r.k_eff > 0)
    assert res.steps == 1 + math.ceil((len(target) - 1) / 5)
    # reference of ids that are never generated: no trigger at all
    res, _ = scripted_run(target, [45, 46, 47, 48], None, 1, 4)
    assert res.trigger_steps == 0 and res.steps == len(target)
    # empty reference
    res, _ = scripted_run(target, [], None, 1, 4)
    assert res.trigger_steps == 0 and res.tokens == target
    # never overshoot N even when the copy would run past it
    res, _ = scripted_run(target[:7], target, None, 1, 18)
    assert res.tokens == target[:7]


# --------------------------------------------------------------------------------------
# the paper's printed decode statistics satisfy the two identities the loop implies
# --------------------------------------------------------------------------------------
def test_fig5_identities():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "fig5_rag_decode_stats.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 45
    by_n = {}
    for n, k, trig, acc, steps in rows:
        trig, acc, steps = float(trig), float(acc), float(steps)
        # every emitted token is either a step's own output or an accepted copy (Table 1: 111.2 mean outputs)
        assert abs(steps + acc - 111.23) < 0.011
        by_n.setdefault(int(n), []).append(steps - trig)
    for n, vals in by_n.items():
        assert max(vals) - min(vals) < 0.021, (n, vals)     # non-trigger steps do not depend on k
    assert by_n[1][0] < by_n[2][0] < by_n[3][0]             # longer n-grams are absent more often


# --------------------------------------------------------------------------------------
# P8/P9: the forward's building blocks against closed forms and invariants
# --------------------------------------------------------------------------------------
def test_attention_pins():
    rng = np.random.default_rng(0)
    hd = 16
    q = rng.standard_normal(hd).astype(np.float32)
    K = rng.standard_normal((9, hd)).astype(np.float32)
    V = rng.standard_normal((9, hd)).astype(np.float32)
    # single cached row: the output is that V row whatever q, K are
    np.testing.assert_allclose(OM.attention(q, K[:1], V[:1]), V[0], rtol=0, atol=1e-7)
    # equal scores (q = 0): plain mean of the V rows
    np.testing.assert_allclose(OM.attention(np.zeros(hd), K, V), V.mean(0), rtol=0, atol=1e-6)
    # library softmax in float64 (scipy), a different code path for the same definition
    from scipy.special import softmax
    w = softmax((K.astype(np.float64) @ q.astype(np.float64)) / math.sqrt(hd))
    np.testing.assert_allclose(OM.attention(q, K, V), w @ V.astype(np.float64), rtol=1e-6, atol=1e-7)
    # shift invariance: adding a multiple of q-orthogonal... simpler: scaling all keys' projection by a constant offset
    K2 = K + 0.0
    q_unit = q / np.linalg.norm(q)
    K2 = K + 3.0 * q_unit[None, :]                         # adds the same constant to every score
    np.testing.assert_allclose(OM.attention(q, K2, V), OM.attention(q, K, V), rtol=1e-5, atol=1e-6)
    # a dominant score selects its row
    K3 = K.copy(); K3[4] = 50.0 * q
    np.testing.assert_allclose(OM.attention(q, K3, V), V[4], rtol=0, atol=1e-5)


def test_rope_pins():
    rng = np.random.default_rng(1)
    hd, theta = 32, 10000.0
    v = rng.standard_normal(hd).astype(np.float32)
    np.testing.assert_array_equal(OM.rope(v, 0, theta), v)                       # position 0 is the identity
    for p in (1, 7, 500):
        assert abs(np.linalg.norm(OM.rope(v, p, theta)) - np.linalg.norm(v)) < 1e-5   # rotations preserve norm
    q = rng.standard_normal(hd).astype(np.float32)
    k = rng.standard_normal(hd).astype(np.float32)
    d1 = float(OM.rope(q, 13, theta).astype(np.float64) @ OM.rope(k, 6, theta).astype(np.float64))
    d2 = float(OM.rope(q, 107, theta).astype(np.float64) @ OM.rope(k, 100, theta).astype(np.float64))
    assert abs(d1 - d2) < 1e-4                                                   # depends on p - s only
    # pairing (i, i + hd/2) and frequencies: a unit vector on pair i turns by pos * theta^(-2i/hd)
    for i in (0, 3, 15):
        e = np.zeros(hd, np.float32); e[i] = 1.0
        r = OM.rope(e, 5, theta)
        ang = 5.0 * theta ** (-2.0 * i / hd)
        assert abs(r[i] - math.cos(ang)) < 1e-6 and abs(r[i + hd // 2] - math.sin(ang)) < 1e-6
        assert np.abs(np.delete(r, [i, i + hd // 2])).max() == 0.0


def test_rmsnorm_silu_matvec_pins():
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(200) * 3).astype(np.float32)
    out = OM.rmsnorm(x, np.ones(200, np.float32), 0.0)
    assert abs(math.sqrt(float(np.mean(out.astype(np.float64) ** 2))) - 1.0) < 1e-6   # unit RMS with unit gain
    g = rng.standard_normal(200).astype(np.float32)
    np.testing.assert_allclose(OM.rmsnorm(x, g, 0.0), out * g, rtol=1e-6)
    np.testing.assert_allclose(OM.rmsnorm(4 * x, g, 0.0), OM.rmsnorm(x, g, 0.0), rtol=1e-6)   # scale invariant
    big_eps = OM.rmsnorm(np.full(4, 2.0, np.float32), np.ones(4, np.float32), 12.0)    # 2/sqrt(4+12) = 0.5
    np.testing.assert_allclose(big_eps, 0.5, rtol=1e-7)
    # SiLU closed-form values: silu(0)=0, silu(x) - silu(-x) = x, large x -> x
    gv = np.array([0.0, 1.0, -1.0, 20.0, -20.0], np.float32)
    s = OM.silu_mul(gv, np.ones(5, np.float32))
    assert s[0] == 0.0 and abs((s[1] - s[2]) - 1.0) < 1e-6 and abs(s[1] - 1 / (1 + math.exp(-1))) < 1e-7
    assert abs(s[3] - 20.0) < 1e-6 and abs(s[4]) < 1e-7
    np.testing.assert_allclose(OM.silu_mul(gv, np.full(5, -2.5, np.float32)), -2.5 * s, rtol=1e-6)
    # matvec against numpy float64, both storage types; a transposed operand would fail on the shape mix
    W = rng.standard_normal((7, 13)).astype(np.float32)
    xv = rng.standard_normal(13).astype(np.float32)
    np.testing.assert_allclose(OM.matvec(W, xv), W.astype(np.float64) @ xv.astype(np.float64), rtol=1e-6)
    Wb = bf16_bits_from_f32(W)
    np.testing.assert_allclose(OM.matvec(Wb, xv), f32_from_bf16_bits(Wb).astype(np.float64) @ xv.astype(np.float64),
                               rtol=1e-6)


def test_bf16_rounding_matches_torch():
    import torch
    rng = np.random.default_rng(4)
    x = np.concatenate([rng.standard_normal(5000).astype(np.float32) * 10.0 ** rng.integers(-6, 6, 5000),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38], np.float32)]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([OM.round_bf16(v) for v in x], np.float32)
    np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))
    np.testing.assert_array_equal(f32_from_bf16_bits(bf16_bits_from_f32(x)).view(np.uint32), want.view(np.uint32))


# --------------------------------------------------------------------------------------
# the whole forward against an independent implementation of the same decoder family
# --------------------------------------------------------------------------------------
def _hf_model(shape, weights):
    import torch
    from transformers import LlamaConfig, LlamaForCausalLM
    kw = dict(vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.d_ffn,
              num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_heads,
              num_key_value_heads=shape.n_heads, head_dim=shape.head_dim, rms_norm_eps=shape.rms_eps,
              max_position_embeddings=512, attention_bias=False, mlp_bias=False, tie_word_embeddings=False,
              hidden_act="silu")
    try:
        cfg = LlamaConfig(rope_theta=shape.rope_theta, **kw)
    except TypeError:
        cfg = LlamaConfig(rope_parameters={"rope_type": "default", "rope_theta": shape.rope_theta}, **kw)
    cfg._attn_implementation = "eager"
    hf = LlamaForCausalLM(cfg).double().eval()

    def t(name):
        a = weights[name]
        if a.dtype == np.uint16:
            a = f32_from_bf16_bits(a)
        return torch.from_numpy(np.asarray(a, np.float64))

    sd = {"model.embed_tokens.weight": t("tok_emb"), "lm_head.weight": t("lm_head"), "model.norm.weight": t("final_norm")}
    for l in range(shape.n_layers):
        p = f"model.layers.{l}."
        sd[p + "input_layernorm.weight"] = t(f"attn_norm.{l}")
        sd[p + "post_attention_layernorm.weight"] = t(f"ffn_norm.{l}")
        for a, b in (("q_proj", "wq"), ("k_proj", "wk"), ("v_proj", "wv"), ("o_proj", "wo")):
            sd[p + f"self_attn.{a}.weight"] = t(f"{b}.{l}")
        for a, b in (("gate_proj", "w_gate"), ("up_proj", "w_up"), ("down_proj", "w_down")):
            sd[p + f"mlp.{a}.weight"] = t(f"{b}.{l}")
    missing, unexpected = hf.load_state_dict(sd, strict=False)
    assert not [m for m in missing if "rotary" not in m and "inv_freq" not in m], missing
    assert not unexpected, unexpected
    return hf


def test_forward_matches_library_llama():
    """The paper ran LLaMA through the Huggingface Transformers library; the same
    library's LLaMA (float64, eager attention, full-sequence causal pass) must give
    the logits that the oracle produces one cached position at a time."""
    import torch
    shape = MICRO
    w = make_weights(shape, seed=7, std=0.2)                 # larger std: attention and gating are far from trivial
    for name in list(w):
        if w[name].ndim == 1:
            w[name] = (1.0 + 0.3 * np.random.default_rng(len(name)).standard_normal(w[name].shape)).astype(np.float32)
    toks = make_prompt(24, shape.vocab, seed=9)
    hf = _hf_model(shape, w)
    with torch.no_grad():
        want = hf(torch.from_numpy(toks.astype(np.int64))[None]).logits[0].numpy()
    om = OM.OracleModel(shape, w, max_seq=64)
    got = np.stack([om.forward(int(t), p) for p, t in enumerate(toks)])
    scale = np.abs(want).max()
    assert np.abs(got - want).max() <= 2e-5 * scale, (np.abs(got - want).max(), scale)
    assert (got.argmax(1) == want.argmax(1)).all()
    # rollback: overwrite positions 10.. with other tokens, then redo the originals -> same logits again
    for p in range(10, 16):
        om.forward(int((toks[p] + 1) % shape.vocab), p)
    redo = np.stack([om.forward(int(toks[p]), p) for p in range(10, 24)])
    np.testing.assert_array_equal(redo, got[10:])


def test_bf16_storage_reading():
    """bf16 shapes: weights are widened exactly and K/V rows are rounded on entering the cache."""
    shape = MICRO_BF16
    w = make_weights(shape, seed=3, std=0.2)
    toks = make_prompt(6, shape.vocab, seed=2)
    om = OM.OracleModel(shape, w, max_seq=16)
    wf = {k: (f32_from_bf16_bits(v) if v.dtype == np.uint16 else v) for k, v in w.items()}
    of = OM.OracleModel(ModelShape("micro-f", 2, 64, 2, 32, 128, 97, "fp32"), wf, max_seq=16, kv_round_bf16=False)
    a = om.forward(int(toks[0]), 0); b = of.forward(int(toks[0]), 0)
    # with a single position softmax is 1 and V passes through: only V's rounding separates the two
    assert 0 < np.abs(a - b).max() < 0.05 * np.abs(b).max()
    krow = om.read_cache(0, 0, 0)
    np.testing.assert_array_equal(krow, f32_from_bf16_bits(bf16_bits_from_f32(krow)))   # cached rows are bf16 values
    kf = of.read_cache(0, 0, 0)
    np.testing.assert_array_equal(krow, f32_from_bf16_bits(bf16_bits_from_f32(kf)))     # = rounding of the fp32 row


# --------------------------------------------------------------------------------------
# P1/P4/P10 with the real forward
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape", [MICRO, MICRO_BF16], ids=lambda s: s.name)
def test_llma_equals_greedy_real_model(shape):
    w = make_weights(shape, seed=0, std=0.3)
    prompt = make_prompt(12, shape.vocab, seed=1)
    N = 40
    g = D.greedy_decode(OM.OracleModel(shape, w, max_seq=80), prompt, N)
    y = g.tokens
    refs = {
        "self": (y, None),
        "spliced": (y[3:14] + [1, 2] + y[20:33] + [5], [0, 13, 27]),
        "random": (make_prompt(50, shape.vocab, seed=8).tolist(), None),
        "empty": ([], None),
    }
    for name, (ref, offs) in refs.items():
        for n, k in ((1, 4), (2, 3), (1, 18), (3, 7), (1, 0)):
            r = D.llma_decode(OM.OracleModel(shape, w, max_seq=80), prompt, ref, offs, n, k, N)
            assert r.tokens == y, (name, n, k)
            assert D.simulate_decoding_sequence(y, ref, offs, n, k) == [(1 + s.k_eff, s.emitted) for s in r.trace]
    r = D.llma_decode(OM.OracleModel(shape, w, max_seq=80), prompt, y, None, 1, 4, N)
    assert r.steps < N / 2       # with the output itself as reference most steps emit several tokens


def test_prescribed_cache_codes_are_checked():
    """oracle_prescribe_kv: a prescribed bf16 code g is adopted for an unrounded value x iff
    |g - x| <= step / 2 + tol * max(1, max|row|); the rule is restated here in numpy and compared element by element.
    The oracle's own codes change nothing; refused codes leave the oracle's own in place."""
    shape, w = MICRO_BF16, make_weights(MICRO_BF16, seed=3, std=0.3)
    HD = shape.n_heads * shape.head_dim
    tok, pos, tol = 5, 0, 4e-4
    exact = OM.OracleModel(shape, w, max_seq=4, kv_round_bf16=False)      # cache rows unrounded
    exact.forward(tok, pos)
    own = OM.OracleModel(shape, w, max_seq=4)
    base = own.forward(tok, pos)
    # layer 0's unrounded rows are the same in both models (nothing upstream of them is rounded)
    k_un = exact.read_cache(0, pos, 0)
    k_own = np.stack([own.read_cache(l, pos, 0) for l in range(shape.n_layers)])
    v_own = np.stack([own.read_cache(l, pos, 1) for l in range(shape.n_layers)])
    assert np.array_equal(bf16_bits_from_f32(k_un), bf16_bits_from_f32(k_own[0]))

    def neighbour(codes_f32, towards):                                    # the bf16 value next to each code, on the side of `towards`
        bits = bf16_bits_from_f32(codes_f32).astype(np.int32)
        step = np.where(codes_f32 >= 0, 1, -1) * np.where(towards > codes_f32, 1, -1)
        return f32_from_bf16_bits((bits + step).astype(np.uint16))

    def rule(g, x):                                                       # the acceptance rule, restated
        big = np.maximum(np.abs(g.astype(np.float64)), np.abs(x.astype(np.float64)))
        step = 2.0 ** (np.floor(np.log2(big)) + 1 - 8)
        return np.abs(g.astype(np.float64) - x) - 0.5 * step <= tol * max(1.0, float(np.abs(x).max()))

    # (1) the oracle's own codes: nothing differs, same logits
    m = OM.OracleModel(shape, w, max_seq=4)
    got = m.forward(tok, pos, given_kv=(k_own, v_own), code_tol=tol)
    assert np.array_equal(got, base) and m.code_stats[0] == 0 and m.code_stats[3] == 2 * shape.n_layers * HD
    # (2) layer 0: every K element replaced by the code on the other side of its unrounded value, then (3) by the
    # neighbouring code on the wrong side: adopted exactly where the rule says so
    sel = k_un != k_own[0]
    for towards in (k_un, 2 * k_own[0] - k_un):
        given = k_own.copy()
        given[0] = np.where(sel, neighbour(k_own[0], towards), k_own[0])
        want_accept = rule(given[0], k_un) & sel
        m = OM.OracleModel(shape, w, max_seq=4)
        m.forward(tok, pos, given_kv=(given, v_own), code_tol=tol)
        assert np.array_equal(m.read_cache(0, pos, 0), np.where(want_accept, given[0], k_own[0]))
        assert m.code_stats[1] >= (sel & ~want_accept).sum() and m.code_stats[2] <= 1.0
    given = k_own.copy()
    given[0] = np.where(sel, neighbour(k_own[0], k_un), k_own[0])
    assert 5 < (rule(given[0], k_un) & sel).sum() < sel.sum() - 5          # both branches of the rule were exercised

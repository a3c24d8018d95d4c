"""Greedy decoding, LLMA decoding and the target-guided simulation, step by step
as the paper states them (test infrastructure only).

``model`` is anything with ``forward(token, pos, want_logits=True)`` returning the
next-token logits after ``token`` is placed at position ``pos`` (see
``oracle.model.OracleModel``; the tests also pass scripted look-up models).

Readings of the paper taken here (each is a choice where the text is silent):
  * The prompt's first P-1 tokens are cached without emitting anything and the
    last prompt token is the first "pending" input, so every output token comes
    from a decoding step and greedy takes exactly N steps (Algorithm 1 starts
    with y empty and calls the model inside the loop).
  * The trigger looks at generated tokens only; with fewer than n of them there
    is no match (Section 2.2 matches the n tokens generated last).
  * Section 2.2 prefers, among several matches, the one that agrees with the
    generated text for longest: read as how far the match extends backwards, bounded
    by the start of the document and the start of y.
  * Ties go to the smallest flattened reference position (one valid instance of
    the paper's random tie-break; it cannot change y, only the trace).
  * Trigger span and copied span stay inside one document; a candidate needs at
    least one token after it.  The copy length actually used is
    k_eff = min(k, tokens left in the document, N - len(y) - 1), so y never
    overshoots N; k_eff = 0 is an ordinary one-token step.

One variant beyond the paper (which fixes n and k for a run and sweeps them, Section 3.5):
``adaptive=(k_min, k_start, k_cap)`` lets the copy length follow the last copy's fate, see
``next_copy_request``.  A fall-back from n to a shorter trigger needs no code of its own: with the
longest-agreement rule above, trying n, n-1, ..., n_lo in turn finds exactly what a trigger of
length n_lo finds, since the candidate that agrees for longest is the same for both.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np


def _docs(ref_len: int, doc_offsets: Optional[Sequence[int]]) -> List[Tuple[int, int]]:
    if doc_offsets is None:
        return [(0, ref_len)]
    return [(int(doc_offsets[i]), int(doc_offsets[i + 1])) for i in range(len(doc_offsets) - 1)]


def match_ngrams(y: Sequence[int], ref: Sequence[int], doc_offsets: Optional[Sequence[int]], n: int
                 ) -> Tuple[bool, int, int]:
    """Section 2.2, trigger: does y[i-n:i] equal some span ref[pos-n:pos] inside one
    document with at least one token following?  Among all such ``pos`` pick the
    one whose agreement with y extends furthest backwards; ties -> smallest pos.

    Returns (matched, pos, ext) with ``pos`` a flattened reference index (the first
    token to copy) and ``ext`` >= n the backward agreement length.
    """
    i = len(y)
    if n < 1 or i < n:
        return False, -1, 0
    best_pos, best_ext = -1, 0
    for (s, e) in _docs(len(ref), doc_offsets):
        for pos in range(s + n, e):  # pos < e: at least one token follows
            t = 0
            while t < i and pos - t - 1 >= s and ref[pos - t - 1] == y[i - t - 1]:
                t += 1
            if t >= n and t > best_ext:  # strict: the first (smallest) pos keeps a tie
                best_pos, best_ext = pos, t
    return best_pos >= 0, best_pos, best_ext


def copy_length(pos: int, ref_len: int, doc_offsets: Optional[Sequence[int]], k: int, remaining: int) -> int:
    """k_eff = min(k, tokens left in pos's document, remaining - 1)."""
    for (s, e) in _docs(ref_len, doc_offsets):
        if s <= pos < e:
            return max(0, min(k, e - pos, remaining - 1))
    return 0


def next_copy_request(k_cur: int, k_eff: int, accepted: int, k_min: int, k_cap: int) -> int:
    """Adaptive copy length (variant): the number of tokens to ask for next.  Unchanged by a step
    that copied nothing; doubled (up to k_cap) after a copy accepted in full; halved, rounding up
    (down to k_min), after a copy the model cut short."""
    if k_eff <= 0:
        return k_cur
    if accepted == k_eff:
        return min(2 * k_cur, k_cap)
    return max(k_min, (k_cur + 1) // 2)


@dataclass
class StepRecord:
    matched: bool      # a copy was applied (k_eff > 0)
    pos: int           # first copied reference index, -1 if none
    k_eff: int         # number of copied tokens fed to the model
    accepted: int      # copied tokens that survived verification
    emitted: int       # tokens appended to y this step (accepted + 1)


@dataclass
class DecodeResult:
    tokens: List[int]
    trace: List[StepRecord] = field(default_factory=list)
    logits: List[np.ndarray] = field(default_factory=list)  # one row per *emitted* token when kept

    @property
    def steps(self) -> int:
        return len(self.trace)

    @property
    def trigger_steps(self) -> int:
        return sum(1 for r in self.trace if r.matched)

    @property
    def copied_accepted(self) -> int:
        return sum(r.accepted for r in self.trace)


def prefill(model, prompt: Sequence[int]) -> Tuple[int, int]:
    """Cache prompt[0..P-2]; return (kv_len, pending) = (P-1, prompt[P-1])."""
    if len(prompt) < 1:
        raise ValueError("prompt must hold at least one token")
    for p, tok in enumerate(prompt[:-1]):
        model.forward(int(tok), p, want_logits=False)
    return len(prompt) - 1, int(prompt[-1])


def greedy_decode(model, prompt: Sequence[int], n_new: int, keep_logits: bool = False) -> DecodeResult:
    """Eq. 2: one token per step, y_i = argmax P(y | x, y_<i) (lowest id on ties)."""
    L, pending = prefill(model, prompt)
    res = DecodeResult(tokens=[])
    for _ in range(n_new):
        lg = model.forward(pending, L)
        o = int(np.argmax(lg))
        res.tokens.append(o)
        res.trace.append(StepRecord(False, -1, 0, 0, 1))
        if keep_logits:
            res.logits.append(lg)
        L += 1
        pending = o
    return res


def llma_decode(model, prompt: Sequence[int], ref: Sequence[int], doc_offsets: Optional[Sequence[int]],
                n: int, k: int, n_new: int, keep_logits: bool = False,
                adaptive: Optional[Tuple[int, int, int]] = None) -> DecodeResult:
    """Algorithm 1.  The k+1 outputs of a copy step (Eq. 3) are computed one position
    at a time, in order, on the inputs [pending, d_pos, ..., d_pos+k_eff-1].
    ``adaptive=(k_min, k_start, k_cap)``: the variant of ``next_copy_request``; a step then asks
    for min(k_cur, k) tokens."""
    L, pending = prefill(model, prompt)
    y: List[int] = []
    res = DecodeResult(tokens=y)
    ref = [int(t) for t in ref]
    k_cur = adaptive[1] if adaptive else 0
    while len(y) < n_new:
        matched, pos, _ = match_ngrams(y, ref, doc_offsets, n)
        k_ask = min(k_cur, k) if adaptive else k
        k_eff = copy_length(pos, len(ref), doc_offsets, k_ask, n_new - len(y)) if matched else 0
        inputs = [pending] + ref[pos:pos + k_eff] if k_eff > 0 else [pending]
        outs, rows = [], []
        for j, tok in enumerate(inputs):
            lg = model.forward(tok, L + j)
            outs.append(int(np.argmax(lg)))
            rows.append(lg)
        # o_0 is always valid; o_{i+1} is valid while o_i equals the copied d_{pos+i}
        a = 0
        while a < k_eff and outs[a] == ref[pos + a]:
            a += 1
        y.extend(outs[:a + 1])
        if keep_logits:
            res.logits.extend(rows[:a + 1])
        res.trace.append(StepRecord(k_eff > 0, pos if k_eff > 0 else -1, k_eff, a, a + 1))
        if adaptive:
            k_cur = next_copy_request(k_cur, k_eff, a, adaptive[0], adaptive[2])
        L += a + 1          # rows past L are stale and get overwritten by later steps
        pending = outs[a]
    return res


def simulate_decoding_sequence(y: Sequence[int], ref: Sequence[int], doc_offsets: Optional[Sequence[int]],
                               n: int, k: int) -> List[Tuple[int, int]]:
    """Algorithm 2: from a target output y and the references alone, the number of
    (input, output) tokens of every decoding step.  Inputs are reported as
    1 + k_eff (equal to the paper's 1 + k whenever k tokens are available)."""
    y = [int(t) for t in y]
    ref = [int(t) for t in ref]
    s: List[Tuple[int, int]] = []
    step = 0
    while step < len(y):
        matched, pos, _ = match_ngrams(y[:step], ref, doc_offsets, n)
        k_eff = copy_length(pos, len(ref), doc_offsets, k, len(y) - step) if matched else 0
        if k_eff == 0:
            step += 1
            s.append((1, 1))
            continue
        num_valid = 0  # get_matched_tokens: how far the reference keeps agreeing with the target
        while num_valid < k_eff and ref[pos + num_valid] == y[step + num_valid]:
            num_valid += 1
        step += num_valid + 1
        s.append((1 + k_eff, num_valid + 1))
    return s

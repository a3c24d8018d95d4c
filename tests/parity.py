"""Step-by-step parity harness: CUDA engine vs CPU oracle on the same seeded inputs.

Integer results (match position, copy length, accepted count, tokens) must be equal;
logits must agree within the stated tolerance on every row of every step.  Where the
two argmaxes differ, the oracle's top-1/top-2 margin at that row must be below
``tie_margin`` (the decision is then legitimately ambiguous across precisions): the event
is counted and both sides continue from the GPU's tokens, which the oracle's
position-indexed cache allows without any special handling.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

from oracle import decoding as D


@dataclass
class ParityReport:
    steps: int = 0
    tokens: List[int] = field(default_factory=list)
    near_ties: int = 0
    max_logit_err: float = 0.0
    max_logit_scale: float = 0.0
    trigger_steps: int = 0
    copied_accepted: int = 0
    rows_compared: int = 0
    code_flips: int = 0            # cache elements where the engine's bf16 code was adopted over the oracle's own
    code_violations: int = 0       # ... where the engine's code was not one of the two bracketing codes
    code_boundary_dist: float = 0.0   # largest share of the tolerance an adopted code needed (<= 1)
    codes_seen: int = 0


BF16_LOGIT_TOL = 2e-2      # absolute, at every depth


def logits_close(got: np.ndarray, want: np.ndarray, mode: str, check: bool = True) -> float:
    """Returns the error measure and (with ``check``) asserts the tolerance.
    fp32: |d| <= 1e-4 * max(1, max|want|) per row.  bf16: |d| <= 2e-2."""
    err = float(np.abs(got - want).max())
    tol = 1e-4 * max(1.0, float(np.abs(want).max())) if mode == "fp32" else BF16_LOGIT_TOL
    if check:
        assert err <= tol, f"logit error {err:.3e} above tolerance {tol:.3e} ({mode})"
    return err


def gpu_kv_rows(eng, seq: int, pos: int):
    """K and V cache rows of one position in every layer, as the engine stored them: float32 [n_layers, H*hd]."""
    L = eng.shape.n_layers
    return (np.stack([eng.llma_debug_kv_row(l, seq, pos, 0) for l in range(L)]),
            np.stack([eng.llma_debug_kv_row(l, seq, pos, 1) for l in range(L)]))


def step_parity(eng, oracle_model, prompt: Sequence[int], ref: Sequence[int], offs: Optional[Sequence[int]],
                n: int, k: int, n_new: int, mode: str, seq: int = 0, tie_margin: float = 1e-3,
                prescribe_kv: bool = False, check_logits: bool = True, adaptive=None) -> ParityReport:
    """Drive ``eng.llma_step`` and the oracle side by side for ``n_new`` tokens of one sequence."""
    assert seq == 0
    return step_parity_batch(eng, [oracle_model], [prompt], [ref], [offs], n, k, n_new, mode, tie_margin,
                             prescribe_kv, check_logits, adaptive)[0]


def step_parity_batch(eng, oracle_models, prompts, refs, offs_list, n: int, k: int, n_new: int, mode: str,
                      tie_margin: float = 1e-3, prescribe_kv: bool = False, check_logits: bool = True,
                      adaptive=None) -> List[ParityReport]:
    """Several sequences decoded together by ``eng.llma_step`` (one forward pass per step for all of
    them), each compared with its own oracle run: integer results per step, every logits row, tokens.
    Runs until every sequence has at least ``n_new`` tokens.

    ``prescribe_kv``: the cache is bf16, so every cached element is a quantised code; where the engine's code
    and the oracle's differ, the oracle adopts the engine's IF rounding some value within the projection's own
    tolerance (1e-4 of the row scale) of the oracle's unrounded value gives that code (counted in ``code_flips``;
    anything else is counted in ``code_violations`` and must not happen).  Both sides then take that decision
    alike and the logits compare the arithmetic instead of the butterfly effect of single rounding flips.
    Prompt rows are prescribed too.

    ``adaptive = (k_min, k_start)``: the adaptive copy length is switched on for every sequence and the plan the
    engine must follow comes from ``oracle.decoding.next_copy_request``."""
    B = len(prompts)
    reps = [ParityReport() for _ in range(B)]
    refs = [[int(t) for t in r] for r in refs]
    kp1 = eng.max_k + 1
    L, pending, ys = [0] * B, [0] * B, [[] for _ in range(B)]
    for s in range(B):
        eng.llma_prefill(s, prompts[s])
        eng.llma_set_reference(s, refs[s], offs_list[s])
        if prescribe_kv:
            for p, tok in enumerate(prompts[s][:-1]):
                oracle_models[s].forward(int(tok), p, want_logits=False, given_kv=gpu_kv_rows(eng, s, p))
            L[s], pending[s] = len(prompts[s]) - 1, int(prompts[s][-1])
        else:
            L[s], pending[s] = D.prefill(oracle_models[s], prompts[s])
        assert eng.llma_kv_len(s) == L[s]
        if adaptive:
            eng.llma_set_adaptive_k(s, adaptive[0], adaptive[1])
    k_cur = [adaptive[1] if adaptive else 0] * B
    while min(len(y) for y in ys) < n_new:
        want = []
        for s in range(B):
            ref, offs, y = refs[s], offs_list[s], ys[s]
            matched, pos, _ = D.match_ngrams(y, ref, offs, n)
            k_ask = min(k_cur[s], k) if adaptive else k
            k_eff = D.copy_length(pos, len(ref), offs, k_ask, eng.max_seq - L[s]) if matched else 0
            want.append((pos, k_eff, [pending[s]] + (ref[pos:pos + k_eff] if k_eff > 0 else [])))
        # the integer plan above needs no model, so the engine can go first and its cache rows (also those of
        # copied tokens that will be rejected: they stay in the cache until overwritten) can be prescribed
        got_all = eng.llma_step(n, k)
        infos = eng.llma_last_step_info()
        logits = eng.llma_debug_logits()
        for s in range(B):
            pos, k_eff, inputs = want[s]
            rows = np.stack([oracle_models[s].forward(tok, L[s] + j,
                                                      given_kv=gpu_kv_rows(eng, s, L[s] + j) if prescribe_kv else None)
                             for j, tok in enumerate(inputs)])
            want[s] = (pos, k_eff, rows)
        for s in range(B):
            rep, ref = reps[s], refs[s]
            pos, k_eff, want_rows = want[s]
            outs = want_rows.argmax(1).tolist()
            a = 0
            while a < k_eff and outs[a] == ref[pos + a]:
                a += 1
            want_tokens = outs[:a + 1]
            got_tokens, info = got_all[s], infos[s]
            assert info.k_eff == k_eff, (s, rep.steps, info.k_eff, k_eff)
            assert info.pos == (pos if k_eff > 0 else -1), (s, rep.steps, info.pos, pos)
            got_rows = logits[s * kp1: s * kp1 + k_eff + 1]
            for j in range(k_eff + 1):
                rep.max_logit_err = max(rep.max_logit_err, logits_close(got_rows[j], want_rows[j], mode, check_logits))
                rep.max_logit_scale = max(rep.max_logit_scale, float(np.abs(want_rows[j]).max()))
            rep.rows_compared += k_eff + 1
            # the engine's acceptance must be Algorithm 1 applied to its own argmaxes
            gouts = got_rows.argmax(1).tolist()
            ga = 0
            while ga < k_eff and gouts[ga] == ref[pos + ga]:
                ga += 1
            assert got_tokens == gouts[:ga + 1], (s, rep.steps, got_tokens, gouts, ga)
            assert info.accepted == ga and info.emitted == ga + 1
            if adaptive:
                k_cur[s] = D.next_copy_request(k_cur[s], k_eff, ga, adaptive[0], eng.max_k)
            if got_tokens != want_tokens:
                common = min(len(got_tokens), len(want_tokens))
                diff = [i for i in range(common) if got_tokens[i] != want_tokens[i]]
                # both sides apply Algorithm 1's acceptance rule to their own argmaxes on the same copied
                # tokens, so two token lists that agree on their common prefix have the same length
                assert diff, f"seq {s} step {rep.steps}: equal prefixes but {len(got_tokens)} vs {len(want_tokens)} tokens"
                j = diff[0]
                srt = np.sort(want_rows[j])
                margin = float(srt[-1] - srt[-2])
                assert margin < tie_margin, f"seq {s}: tokens differ at step {rep.steps} row {j} with oracle margin {margin:.3e}"
                rep.near_ties += 1
            ys[s].extend(got_tokens)
            L[s] += len(got_tokens)
            pending[s] = got_tokens[-1]
            assert eng.llma_kv_len(s) == L[s]
            rep.steps += 1
            rep.trigger_steps += int(k_eff > 0)
            rep.copied_accepted += len(got_tokens) - 1
    for s in range(B):
        reps[s].tokens = ys[s]
        st = getattr(oracle_models[s], "code_stats", None)
        if st is not None:
            reps[s].code_flips, reps[s].code_violations = int(st[0]), int(st[1])
            reps[s].code_boundary_dist, reps[s].codes_seen = float(st[2]), int(st[3])
    return reps

"""GPU tests of the C ABI's argument checking and edge cases (host-side failures only)."""
import numpy as np
import pytest

from workloads import SHAPES, make_prompt, make_weights

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def setup():
    from paper_2304_04487_b200 import Engine
    shape = SHAPES["tiny-fp32"]
    w = make_weights(shape, seed=0)
    return Engine, shape, w


def test_argument_errors_leave_engine_usable(setup):
    from paper_2304_04487_b200 import LlmaError
    Engine, shape, w = setup
    eng = Engine(shape, w, max_seq=48, max_ref=16, max_k=4)
    with pytest.raises(LlmaError) as ei:
        eng.llma_step(1, 2)                              # nothing prefilled
    assert ei.value.status == -6
    prompt = make_prompt(20, shape.vocab, seed=1)
    for bad, code in ((list(prompt[:5]) + [shape.vocab], -3), ([-1], -3), (list(range(49)), -4), ([], -9)):
        with pytest.raises(LlmaError) as ei:
            eng.llma_prefill(0, bad)
        assert ei.value.status == code
    with pytest.raises(LlmaError) as ei:
        eng.llma_prefill(1, prompt)                      # only one slot
    assert ei.value.status == -4
    eng.llma_prefill(0, prompt)
    for (n, k) in ((0, 2), (1, 5), (1, -1)):
        with pytest.raises(LlmaError) as ei:
            eng.llma_step(n, k)
        assert ei.value.status == -9
    with pytest.raises(LlmaError) as ei:
        eng.llma_set_reference(0, list(range(17)))
    assert ei.value.status == -5
    with pytest.raises(LlmaError) as ei:
        eng.llma_set_reference(0, [1, 2, 3, 4], [0, 3, 2, 4])
    assert ei.value.status == -5
    with pytest.raises(LlmaError) as ei:
        eng.llma_set_reference(0, [1, 2, shape.vocab])
    assert ei.value.status == -3
    with pytest.raises(LlmaError) as ei:
        eng.llma_generate(30, 1, 2)                      # 19 cached + 30 > 48
    assert ei.value.status == -4
    with pytest.raises(LlmaError) as ei:
        eng.llma_debug_logits()                          # keep_logits was not requested
    assert ei.value.status == -6
    (toks,), st = eng.llma_generate(29, 1, 2)            # exactly fills the cache
    assert len(toks) == 29 and eng.llma_kv_len(0) == 48
    with pytest.raises(LlmaError) as ei:
        eng.llma_step(1, 2)                              # cache is full
    assert ei.value.status == -4
    eng.llma_rewind(0)
    (again,), _ = eng.llma_generate(29, 1, 0)
    assert again == toks
    eng.llma_reset(0)
    with pytest.raises(LlmaError):
        eng.llma_kv_len(0)


def test_unsupported_configs_rejected(setup):
    from paper_2304_04487_b200 import LlmaError
    Engine, shape, w = setup
    with pytest.raises(LlmaError) as ei:
        Engine(shape, w, max_seq=32, max_ref=8, max_k=16, max_batch=16)  # 16 * 17 rows > 256
    assert ei.value.status == -2
    with pytest.raises(LlmaError) as ei:
        Engine(shape, w, max_seq=32, max_ref=8, max_k=2, gemm_impl=2)    # tensor-core GEMM needs bf16
    assert ei.value.status == -2


def test_edge_cases(setup):
    Engine, shape, w = setup
    eng = Engine(shape, w, max_seq=64, max_ref=32, max_k=8, eos_id=-1)
    # one-token prompt: nothing to cache, first step runs at position 0
    eng.llma_prefill(0, [5])
    assert eng.llma_kv_len(0) == 0
    (g,), st = eng.llma_generate(20, 1, 0)
    assert len(g) == 20
    # zero new tokens is a no-op
    (z,), st0 = eng.llma_generate(0, 1, 4)
    assert z == [] and st0.steps == 0
    # a match right at the end of a document copies nothing; a copy longer than what is left to
    # emit is cut so that exactly max_new tokens come out
    eng.llma_set_reference(0, g[:6] + g[10:14], [0, 6, 10])
    eng.llma_rewind(0)
    (t,), st = eng.llma_generate(7, 1, 8)
    assert t == g[:7] and st.tokens == 7
    eng.llma_rewind(0)
    (t,), st = eng.llma_generate(20, 1, 8)
    assert t == g
    # EOS: generation stops right after the first occurrence of eos_id
    eos = g[9]
    first = g.index(eos)
    e2 = Engine(shape, w, max_seq=64, max_ref=32, max_k=8, eos_id=eos)
    e2.llma_prefill(0, [5])
    e2.llma_set_reference(0, g[:20])
    (t,), st = e2.llma_generate(20, 1, 8)
    assert t == g[:first + 1]


def test_microbench_mma_runs_and_rejects_bad_arguments():
    """The tensor-core timing probe: a plausible figure for a legal shape, LLMA_ERR_ARG for the rest."""
    from paper_2304_04487_b200 import LlmaError, llma_microbench_mma
    t32 = llma_microbench_mma(32, 1, 256, 0)
    t256 = llma_microbench_mma(256, 2, 256, 1)
    assert 10.0 < t32 < 1000.0 and 10.0 < t256 < 1000.0, (t32, t256)
    for bad in ((24, 1, 256, 0), (272, 1, 256, 0), (256, 3, 256, 0), (32, 1, 0, 0), (32, 1, 256, 5), (0, 1, 1, 0)):
        with pytest.raises(LlmaError):
            llma_microbench_mma(*bad)

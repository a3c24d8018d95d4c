"""Micro-benchmark of the projection GEMM on its own (weight streaming at 32 activation rows).

    python -m paper_2304_04487_b200.microbench --n-out 22016 --k-in 4096 --iters 40
    python -m paper_2304_04487_b200.microbench --mma      # tensor-core time per MMA against N, regions, commits
    python -m paper_2304_04487_b200.microbench --attention --batch 16 --history 4096 --k 8
                                                          # one 7B-shaped layer, B sequences: per-kernel-class times of
                                                          # a one-row and a (k+1)-row step; prints how many attention
                                                          # launches precede them (for a profiler's launch-skip)

Cycles through several weight buffers so that every launch streams its matrix from HBM
(one matrix may fit in the 126 MB L2), times the launches with CUDA events on the launching
stream and prints achieved GB/s of weight bytes.
"""
from __future__ import annotations

import argparse
import json


def main():
    import torch
    from . import llma_gemm_rows32_bf16_noalloc
    ap = argparse.ArgumentParser()
    ap.add_argument("--n-out", type=int, default=22016)
    ap.add_argument("--k-in", type=int, default=4096)
    ap.add_argument("--iters", type=int, default=40)
    ap.add_argument("--buffers", type=int, default=4)
    ap.add_argument("--mma", action="store_true")
    ap.add_argument("--attention", action="store_true")
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--history", type=int, default=4096)
    ap.add_argument("--k", type=int, default=8)
    a = ap.parse_args()
    if a.attention:
        from workloads import SHAPES, make_prompt, make_weights
        from . import Engine
        shape = SHAPES["llama7b-1layer"]
        eng = Engine(shape, make_weights(shape, seed=0), max_seq=a.history + 100, max_ref=64, max_k=a.k, max_batch=a.batch)
        for s_ in range(a.batch):
            eng.llma_prefill(s_, make_prompt(a.history, shape.vocab, seed=100 + s_))
        ys, _ = eng.llma_generate(24, 1, 0)
        for s_ in range(a.batch):
            eng.llma_set_reference(s_, ys[s_], None)     # every sequence then copies k tokens per step
            eng.llma_rewind(s_)
        before = a.batch * ((a.history - 1 + 127) // 128) + 24     # prompt passes + the greedy steps above (one layer)
        out = {"attention_tiles_per_cta": eng.llma_debug_attention_tiles(), "attention_launches_before": before}
        for kk in (0, a.k):
            eng.llma_step(1, kk); eng.llma_step(1, kk)
            pr = eng.llma_profile_steps(1, kk, 3)
            out[f"k={kk}"] = {n: round(1e3 * v["ms_per_step"], 1) for n, v in pr.items()}
        print(json.dumps(out))
        return
    if a.mma:
        from . import llma_microbench_mma
        rows = []
        for n in (16, 32, 64, 96, 128, 144, 192, 256):
            for regions in (1, 2):
                if regions * n <= 512:
                    rows.append({"n": n, "regions": regions, "commits_per_group": 0,
                                 "ns_per_mma": round(llma_microbench_mma(n, regions, 512, 0), 1)})
        for commits in (1, 2):
            rows.append({"n": 32, "regions": 1, "commits_per_group": commits,
                         "ns_per_mma": round(llma_microbench_mma(32, 1, 512, commits), 1)})
        print(json.dumps({"mma_m128_k16_bf16": rows}))
        return
    torch.manual_seed(0)
    Ws = [(torch.randn(a.n_out, a.k_in, device="cuda") * 0.02).to(torch.bfloat16) for _ in range(a.buffers)]
    act = torch.randn(32, a.k_in, device="cuda").to(torch.bfloat16)
    out = torch.empty(32, a.n_out, device="cuda")
    st = torch.cuda.current_stream()
    for i in range(3):
        llma_gemm_rows32_bf16_noalloc(Ws[i % a.buffers], act, out)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(a.iters + 1)]
    # each call is synchronous (it reads back its error word), so the event pairs bracket
    # exactly one launch plus its small clears; the clears are a few microseconds
    times = []
    for i in range(a.iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        llma_gemm_rows32_bf16_noalloc(Ws[i % a.buffers], act, out)
        e1.record(st)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    times.sort()
    med = times[len(times) // 2]
    nbytes = a.n_out * a.k_in * 2
    print(json.dumps({"n_out": a.n_out, "k_in": a.k_in, "bytes": nbytes, "median_us": 1e3 * med,
                      "min_us": 1e3 * times[0], "gbs_median": nbytes / (med / 1e3) / 1e9,
                      "gbs_best": nbytes / (times[0] / 1e3) / 1e9}))


if __name__ == "__main__":
    main()

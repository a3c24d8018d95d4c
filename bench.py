#!/usr/bin/env python
"""Benchmark of the LLMA reference-copy decode loop on B200.

One "step" of this benchmark is one whole decode of the workload: llma_generate of
``n_new`` tokens (trigger search, copy, (k+1)-row forward, argmax, accept, K/V commit for
every decoding step) from the state right after prefill.  The workload is the LLaMA-7B-shaped
bf16 decoder with random-init weights, a 1536-token prompt, a reference of three 480-token
documents spliced from the engine's own greedy continuation at 80 % overlap, n = 1, k = 8,
256 new tokens, batch 1.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

N > 1 (under torchrun) runs N independent replicas, one per GPU: the path is a single
dependent chain per sequence and has nothing to shard or exchange.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import SHAPES, build_reference, make_prompt, make_weights  # noqa: E402

WORKLOADS = {
    # name: (shape, prompt_len, doc_lengths, overlap, n, k, n_new)
    "llama7b-rag": ("llama7b-shape", 1536, [480, 480, 480], 0.8, 1, 8, 256),
    "llama13b-rag": ("llama13b-shape", 2048, [1024], 0.8, 1, 8, 256),
    "llama7b-2layer-rag": ("llama7b-2layer", 1536, [480, 480, 480], 0.8, 1, 8, 256),   # small case for profiler captures
    "mid-rag": ("mid-bf16", 256, [128, 128], 0.8, 1, 8, 128),
    "tiny-fp32": ("tiny-fp32", 128, [256], 0.6, 2, 4, 64),
}
METRIC = "tokens_per_s_llma_b1"
UNIT = "tokens/s"


def measured_traffic_ratio():
    """DRAM traffic / algorithmic bytes of the GEMM kernel from the committed ncu summary, or None
    when the kernel's sources have changed since those counters were taken."""
    import hashlib
    prof = os.path.join(ROOT, "profiles", "gemm_ws_kernel_ncu_full_22016x4096.md")
    src = [os.path.join(ROOT, "paper_2304_04487_b200", "csrc", f)
           for f in ("gemm_tcgen05.cu", "gemm_epilogue.cuh", "gemm_tcgen05.cuh", "ptx_sm100.cuh")]
    try:
        h = hashlib.sha256(b"".join(open(f, "rb").read() for f in src)).hexdigest()[:16]
        kv = dict(l.strip().split("=", 1) for l in open(prof) if "=" in l and not l.startswith("|") and " " not in l.strip())
        if kv.get("kernel_sources_sha256_16") == h:
            return float(kv["traffic_ratio"])
    except Exception:
        pass
    return None


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks of the default process group
    (identity without one): multi-GPU numbers are timed per rank and reported as the slowest."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def replica_throughput(tokens_per_replica: int, world: int, slowest_seconds: float) -> float:
    """Whole-job tokens/s of `world` independent replicas (weak scaling: same work per GPU)."""
    return tokens_per_replica * world / slowest_seconds


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


def cpu_oracle_sample(shape, weights, n, k, budget_s=20.0):
    """Times the CPU oracle as it stands on a bounded sample of the same decoder: after a
    4-token prompt, greedy tokens are decoded until ~40 % of the budget is used; then LLMA
    decoding (same n, k) of those tokens with an 80 %-overlap reference built from them."""
    from oracle import decoding as D
    from oracle import model as OM
    prompt = make_prompt(4, shape.vocab, seed=1).tolist()
    om = OM.OracleModel(shape, weights, max_seq=96)
    L, pending = D.prefill(om, prompt)
    t0 = time.perf_counter()
    y = []
    while len(y) < 24 and (time.perf_counter() - t0 < 0.4 * budget_s or len(y) < 4):
        o = int(np.argmax(om.forward(pending, L))); y.append(o); L += 1; pending = o
    t_greedy = time.perf_counter() - t0
    ref, offs, _ = build_reference(y, [max(8, 2 * len(y))], 0.8, shape.vocab, span_len=(3, 6), seed=0)
    om2 = OM.OracleModel(shape, weights, max_seq=96)
    D.prefill(om2, prompt)                      # prefill outside the timed part, as on the GPU
    L, pending, out = len(prompt) - 1, prompt[-1], []
    t1 = time.perf_counter()
    refl = ref.tolist()
    steps = 0
    while len(out) < len(y):
        matched, pos, _ = D.match_ngrams(out, refl, offs.tolist(), n)
        k_eff = D.copy_length(pos, len(refl), offs.tolist(), k, len(y) - len(out)) if matched else 0
        inputs = [pending] + refl[pos:pos + k_eff] if k_eff else [pending]
        outs = [int(np.argmax(om2.forward(t, L + j))) for j, t in enumerate(inputs)]
        a = 0
        while a < k_eff and outs[a] == refl[pos + a]:
            a += 1
        out += outs[:a + 1]; L += a + 1; pending = outs[a]; steps += 1
    t_llma = time.perf_counter() - t1
    assert out == y, "CPU oracle: LLMA differs from greedy"
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    return {"value": len(y) / t_llma, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{shape.name}: 4-token prompt, {len(y)} tokens decoded by LLMA (n={n}, k={k}) in {steps} steps "
                      f"({t_llma:.1f} s); same tokens by one-token greedy: {len(y) / t_greedy:.3f} tokens/s",
            "greedy_value": len(y) / t_greedy}


def run_reference(args, rank):
    if rank != 0:
        return
    shape_name, P, docs, f, n, k, n_new = WORKLOADS[args.workload]
    shape = SHAPES[shape_name]
    w = make_weights(shape, seed=0)
    vals = []
    for _ in range(args.warmup + args.steps):
        vals.append(cpu_oracle_sample(shape, w, n, k, budget_s=max(10.0, 150.0 / (args.warmup + args.steps))))
    timed = vals[args.warmup:]
    v = float(np.mean([x["value"] for x in timed]))
    cb = dict(timed[-1]); cb["value"] = v
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * n_new / v, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if shape.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": args.workload, "shape": shape.name, "n": n, "k": k, "n_new": n_new},
            "cpu_baseline": cb,
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b-rag", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-steps", type=int, default=6)
    ap.add_argument("--profile-only", action="store_true",
                    help="short run for profilers: prefill, 32 greedy steps, then --steps LLMA decodes of 32 tokens")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2304_04487_b200 import Engine
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the engine has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    shape_name, P, docs, f, n, k, n_new = WORKLOADS[args.workload]
    shape = SHAPES[shape_name]
    t_gen = time.perf_counter()
    w = make_weights(shape, seed=0)
    t_gen = time.perf_counter() - t_gen
    prompt = make_prompt(P, shape.vocab, seed=1)
    max_seq = P + n_new + 32
    eng = Engine(shape, w, max_seq=max_seq, max_ref=sum(docs), max_k=k, device=f"cuda:{local_rank}")
    t_pre = time.perf_counter()
    eng.llma_prefill(0, prompt)
    t_pre = time.perf_counter() - t_pre
    if args.profile_only:
        n_new = 32
    (y_star,), g0 = eng.llma_generate(n_new, 1, 0)
    if args.profile_only:
        # launches so far: ceil((P-1)/32) prefill passes of (1 + 7 L) kernels (tensor-core path), then
        # n_new greedy steps of g0.launches / n_new kernels each
        eng.llma_set_reference(0, y_star, None)
        tot = 0
        for _ in range(args.steps):
            eng.llma_rewind(0)
            _, st = eng.llma_generate(n_new, n, k)
            tot += st.launches
        print(json.dumps({"profile_only": True, "launches_per_step": g0.launches // n_new,
                          "greedy_launches": int(g0.launches), "llma_launches": int(tot),
                          "llma_steps": int(st.steps), "llma_ms_per_step": st.device_ms / st.steps}))
        return
    ref, offs, ref_info = build_reference(y_star, docs, f, shape.vocab, seed=0)
    ref_host = torch.from_numpy(ref.copy()).pin_memory().numpy()

    def one_llma():
        eng.llma_set_reference(0, ref_host, offs)        # host -> device copy of the step's inputs
        eng.llma_rewind(0)
        toks, st = eng.llma_generate(n_new, n, k)         # device -> host read of the result inside
        return toks[0], st

    def one_greedy():
        eng.llma_rewind(0)
        toks, st = eng.llma_generate(n_new, 1, 0)
        return toks[0], st

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        toks, _ = one_llma()
        assert toks == y_star, "LLMA output differs from the engine's own greedy decode"
        one_greedy()

    sampler = ClockSampler(local_rank)
    sampler.start()
    # ---- timed region: K LLMA decodes; device time from the engine's own CUDA events ----------
    barrier()
    dev_ms, wall0, launches, steps_taken, trig, acc = 0.0, time.perf_counter(), 0, 0, 0, 0
    for _ in range(args.steps):
        toks, st = one_llma()
        dev_ms += st.device_ms; launches += st.launches; steps_taken += st.steps
        trig += st.trigger_steps; acc += st.copied_accepted
    barrier()
    wall_s = time.perf_counter() - wall0
    # ---- same number of greedy decodes on the same engine ----------------------------------------
    g_ms = 0.0
    g_wall0 = time.perf_counter()
    for _ in range(args.steps):
        toks, st = one_greedy()
        g_ms += st.device_ms
    barrier()
    clocks = sampler.stop()
    assert toks == y_star

    dev_ms, wall_s, g_ms = max_over_ranks([dev_ms, wall_s, g_ms], device="cuda")
    value = replica_throughput(args.steps * n_new, world, dev_ms / 1e3)
    e2e_value = replica_throughput(args.steps * n_new, world, wall_s)
    greedy_value = replica_throughput(args.steps * n_new, world, g_ms / 1e3)

    # ---- roofline of the dominant kernel: the weight-streaming GEMM -----------------------------
    peak, peak_kind = load_peaks()
    eng.llma_set_reference(0, y_star, None)              # every profiled step verifies k+1 rows
    eng.llma_rewind(0)
    eng.llma_step(1, 0)
    prof = eng.llma_profile_steps(1, k, args.profile_steps)
    gemm_keys = [x for x in prof if x.startswith("gemm_")]
    gemm_ms = sum(prof[x]["ms_per_step"] for x in gemm_keys)
    gemm_launches = sum(prof[x]["launches_per_step"] for x in gemm_keys)
    wbytes = shape.weight_bytes_per_step()
    kv_len_mid = P + n_new // 2
    kvbytes = shape.kv_bytes_per_position() * kv_len_mid
    achieved = wbytes / (gemm_ms / 1e3) / 1e9
    step_ms = dev_ms / max(steps_taken, 1)
    roofline = {"bound": "hbm", "kernel": "gemm_ws_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                # per launch, scaled from the ncu capture of a 180 MB launch (traffic grows with the matrix size)
                "traffic": (None if measured_traffic_ratio() is None
                            else measured_traffic_ratio() * wbytes / max(gemm_launches, 1)),
                "bytes_per_launch": wbytes / max(gemm_launches, 1), "us_per_launch": 1e3 * gemm_ms / max(gemm_launches, 1),
                "launches_per_step": gemm_launches,
                "whole_step": {"bytes": wbytes + kvbytes, "ms": step_ms,
                               "frac": (wbytes + kvbytes) / (step_ms / 1e3) / 1e9 / peak},
                "per_class_ms_per_step": {x: round(prof[x]["ms_per_step"], 4) for x in prof}}

    # step latency against k: reference = y* itself, so every step feeds k+1 rows.  k <= 8 on the
    # benchmark's engine (16-row MMA shape); k = 16 needs an engine created for 17 rows (32-row shape)
    lat = {}
    for kk in (0, 1, 4, 8):
        if kk > k:
            continue
        eng.llma_rewind(0)
        _, st = eng.llma_generate(n_new, 1, kk)
        lat[str(kk)] = {"ms_per_step": st.device_ms / st.steps, "tokens_per_step": st.tokens / st.steps}
    eng16 = Engine(shape, None, max_seq=max_seq, max_ref=sum(docs), max_k=16, device=f"cuda:{local_rank}",
                   share_weights_with=eng)
    eng16.llma_prefill(0, prompt)
    eng16.llma_set_reference(0, y_star, None)
    for kk in (0, 8, 16):
        eng16.llma_rewind(0)
        _, st = eng16.llma_generate(n_new, 1, kk)
        lat[f"{kk}@32rows"] = {"ms_per_step": st.device_ms / st.steps, "tokens_per_step": st.tokens / st.steps}
    eng16.llma_destroy()

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dev_ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if shape.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": args.workload, "shape": shape.name, "prompt": P, "reference_docs": docs,
                       "overlap": f, "n": n, "k": k, "n_new": n_new, "batch": 1,
                       "l2": "inputs (weights) larger than L2", "replicas": world,
                       "reference_info": ref_info},
            "greedy_tokens_per_s": greedy_value, "speedup_vs_own_greedy": value / greedy_value,
            "decode_ms_per_llma_step": step_ms, "tokens_per_llma_step": n_new * args.steps / max(steps_taken, 1),
            "llma_steps_per_decode": steps_taken / args.steps, "trigger_steps_per_decode": trig / args.steps,
            "accepted_per_decode": acc / args.steps, "step_latency_vs_k": lat,
            "prefill_s": t_pre, "weight_gen_s": t_gen,
            "clocks": clocks, "gpu_launches": int(launches),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(ref.nbytes + offs.nbytes),
                    "d2h_bytes_per_step": int(4 * n_new),
                    "note": "set_reference (host->device) + rewind + generate (tokens device->host), wall clock; "
                            "prefill excluded as in value"},
            "roofline": roofline}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_oracle_sample(shape, w, n, k)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

"""Where the time of a decoding step goes, from timestamps taken inside the kernels.

Needs the measurement build of the library (it records nothing otherwise):

    LLMA_BUILD_STAMPS=1 python -m paper_2304_04487_b200.build
    python -m paper_2304_04487_b200.timeline [--shape llama7b-shape] [--prompt 1536] [--k 0 8] [--batch 1]
    python -m paper_2304_04487_b200.build          # back to the normal library

Prints, per projection of a layer (averaged over the inner layers of the last step of a decode), the
events of its CTAs relative to the end of the projection before it, and what the attention kernels
between the QKV and the output projection do.  All times in microseconds.  With --batch B the B sequences
decode together; beyond 32 rows per step that is the wide GEMM kernel, whose last two words per CTA are the
time its MMA thread spent waiting for ring stages and (unused) zero.
"""
from __future__ import annotations

import argparse

import numpy as np


def main():
    from workloads import SHAPES, make_prompt, make_weights
    from . import Engine
    ap = argparse.ArgumentParser()
    ap.add_argument("--shape", default="llama7b-shape")
    ap.add_argument("--prompt", type=int, default=1536)
    ap.add_argument("--new", type=int, default=64)
    ap.add_argument("--k", type=int, nargs="+", default=[0, 8])
    ap.add_argument("--batch", type=int, default=1)
    a = ap.parse_args()
    shape = SHAPES[a.shape]
    B = a.batch
    eng = Engine(shape, make_weights(shape, seed=0), max_seq=a.prompt + a.new + 32, max_ref=a.new, max_k=max(a.k + [8]),
                 max_batch=B)
    wide = B * (max(a.k + [8]) + 1) > 32
    for s_ in range(B):
        eng.llma_prefill(s_, make_prompt(a.prompt, shape.vocab, seed=1 + s_))
    ys, _ = eng.llma_generate(a.new, 1, 0)
    for s_ in range(B):
        eng.llma_set_reference(s_, ys[s_], None)
    L = shape.n_layers
    names = ["qkv", "o", "gate/up", "down"]
    for k in a.k:
        for s_ in range(B):
            eng.llma_rewind(s_)
        eng.llma_debug_timeline(clear=True)
        _, st = eng.llma_generate(a.new, 1, k)
        t = eng.llma_debug_timeline(clear=False).astype(np.int64)
        sms = int((t[0, :, 0] > 0).sum())
        print(f"k = {k}: {st.device_ms / st.steps:.3f} ms per step, {sms} CTAs per projection")
        g = t[:4 * L + 1, :sms, :7]
        for cls in range(4):
            rows = []
            for l in range(1, L - 1):
                i = 4 * l + cls
                prev_end = g[i - 1, :, 5].max()
                s = g[i] - prev_end
                rows.append([s[:, 0].min(), s[:, 1].min(), s[:, 2].min(), np.median(s[:, 2]), s[:, 3].min(), s[:, 3].max(),
                             s[:, 4].max(), s[:, 5].min(), s[:, 5].max()])
                last = int(np.argmax(s[:, 5]))  # the CTA that ends last: its own accumulator, epilogue start and end
                if wide:  # words 6, 7 hold durations there: the MMA thread's waits
                    rows[-1] += [s[last, 4], g[i, :, 6].mean()]
                else:
                    rows[-1] += [s[last, 4], s[last, 6] if g[i, last, 6] > 0 else s[last, 4]]
            m = np.mean(rows, 0) / 1e3
            print(f"  {names[cls]:8s} after the projection before it ended: first CTA starts {m[0]:6.2f}, dependency released {m[1]:6.2f}, "
                  f"first MMA {m[2]:6.2f} (median {m[3]:6.2f}), last MMA issued {m[4]:6.2f}..{m[5]:6.2f}, "
                  f"last accumulator ready {m[6]:6.2f}, CTAs end {m[7]:6.2f}..{m[8]:6.2f}; the CTA that ends last: "
                  f"accumulator {m[9]:6.2f}, " + (f"MMA thread waited for stages {m[10]:6.2f} in all" if wide else f"partials summed {m[10]:6.2f}"))
        rows = []
        for l in range(1, L - 1):
            qkv_end = g[4 * l, :, 5].max()
            at, mg = t[300 + l, 0] - qkv_end, t[400 + l, 0] - qkv_end
            rows.append([at[1], at[3], at[5], at[7], mg[3], mg[7], g[4 * l + 1, :, 1].min() - qkv_end])
        m = np.mean(rows, 0) / 1e3
        print(f"  attention after the QKV projection ended: last CTA starts {m[0]:.2f}, dependency released {m[1]:.2f}, last K tile landed "
              f"{m[2]:.2f}, last CTA ends {m[3]:.2f}; merge: dependency released {m[4]:.2f}, last warp ends {m[5]:.2f}; "
              f"output projection released {m[6]:.2f}")
        lm = g[4 * L] - g[4 * L - 1, :, 5].max()
        print(f"  lm head: first MMA {lm[:, 2].min() / 1e3:.2f}, last MMA issued {lm[:, 3].min() / 1e3:.2f}..{lm[:, 3].max() / 1e3:.2f}, "
              f"CTAs end {lm[:, 5].min() / 1e3:.2f}..{lm[:, 5].max() / 1e3:.2f}")


if __name__ == "__main__":
    main()

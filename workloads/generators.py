"""Seeded generators for decoder shapes, weights, prompts and reference documents.

Everything here is input data: normal/uniform draws, bf16 storage conversion of
the drawn weights, and the splicing of token spans into reference documents.
No decoding arithmetic lives in this file.

Streams (numpy SFC64 seeded by (seed, tensor index) for weights, Philox keyed by
(seed, stream id) for tokens) so that every tensor can
be regenerated on its own and in parallel:
    weights  seed 0   one stream per tensor (index in ``weight_names``)
    prompt   seed 1
    filler   seed 2   (reference tokens that are not copied from y*)
    layout   seed 3   (span lengths, gaps, filler placement)
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, asdict
from typing import Dict, List, Sequence, Tuple

import numpy as np


@dataclass(frozen=True)
class ModelShape:
    """LLaMA-style decoder shape.  ``dtype`` is how weights are stored."""

    name: str
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    dtype: str  # "fp32" | "bf16"
    rms_eps: float = 1e-6
    rope_theta: float = 10000.0

    def with_layers(self, n_layers: int) -> "ModelShape":
        d = asdict(self)
        d["n_layers"] = n_layers
        d["name"] = f"{self.name}-L{n_layers}"
        return ModelShape(**d)

    def weight_bytes_per_step(self) -> int:
        """Bytes of weights one decode step must stream (embedding rows excluded)."""
        e = 4 if self.dtype == "fp32" else 2
        d, f, v = self.d_model, self.d_ffn, self.vocab
        qkvo = 4 * (self.n_heads * self.head_dim) * d
        per_layer = (qkvo + 3 * f * d) * e
        return self.n_layers * per_layer + v * d * e

    def kv_bytes_per_position(self) -> int:
        e = 4 if self.dtype == "fp32" else 2
        return self.n_layers * 2 * self.n_heads * self.head_dim * e


SHAPES: Dict[str, ModelShape] = {
    # tiny fp32 decoder: the case the CPU oracle finishes in seconds
    "tiny-fp32": ModelShape("tiny-fp32", 2, 256, 4, 64, 1024, 4096, "fp32"),
    # same widths stored in bf16: exercises the tensor-core path at oracle-friendly size
    "tiny-bf16": ModelShape("tiny-bf16", 2, 256, 4, 64, 1024, 4096, "bf16"),
    # head_dim 128 at small width, several row tiles and a ragged vocab tail
    "small-bf16": ModelShape("small-bf16", 3, 512, 4, 128, 1408, 5000, "bf16"),
    # wide enough that every projection is split over several CTAs along k
    "mid-bf16": ModelShape("mid-bf16", 2, 1024, 8, 128, 2816, 8000, "bf16"),
    "llama7b-shape": ModelShape("llama7b-shape", 32, 4096, 32, 128, 11008, 32000, "bf16"),
    # two layers at the 7B widths: the same kernels and tile shapes at a size a profiler capture can hold
    "llama7b-2layer": ModelShape("llama7b-2layer", 2, 4096, 32, 128, 11008, 32000, "bf16"),
    # one layer of the 7B-shaped decoder with a token table too small to matter: what a step costs is the layer
    "llama7b-1layer": ModelShape("llama7b-1layer", 1, 4096, 32, 128, 11008, 256, "bf16"),
    "llama13b-shape": ModelShape("llama13b-shape", 40, 5120, 40, 128, 13824, 32000, "bf16"),
    "llama13b-2layer": ModelShape("llama13b-2layer", 2, 5120, 40, 128, 13824, 32000, "bf16"),
}


def weight_names(shape: ModelShape) -> List[str]:
    names = ["tok_emb", "lm_head", "final_norm"]
    for l in range(shape.n_layers):
        for w in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down"):
            names.append(f"{w}.{l}")
    return names


def _weight_dims(shape: ModelShape, name: str) -> Tuple[int, ...]:
    base = name.split(".")[0]
    d, f, v, hh = shape.d_model, shape.d_ffn, shape.vocab, shape.n_heads * shape.head_dim
    return {
        "tok_emb": (v, d), "lm_head": (v, d), "final_norm": (d,),
        "attn_norm": (d,), "ffn_norm": (d,),
        "wq": (hh, d), "wk": (hh, d), "wv": (hh, d), "wo": (d, hh),
        "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f),
    }[base]


def bf16_bits_from_f32(x: np.ndarray) -> np.ndarray:
    """Storage conversion fp32 -> bf16 bit patterns (round to nearest, ties to even)."""
    u = np.array(x, dtype=np.float32, copy=True, order="C").view(np.uint32)
    shape = u.shape
    u = u.reshape(-1)
    lsb = u >> np.uint32(16)
    lsb &= np.uint32(1)
    u += np.uint32(0x7FFF)
    u += lsb
    return np.ascontiguousarray(u.view(np.uint16)[1::2]).reshape(shape)   # high halves (little endian)


def f32_from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _gen_one(shape: ModelShape, name: str, index: int, seed: int, std: float) -> np.ndarray:
    dims = _weight_dims(shape, name)
    if len(dims) == 1:  # norm gains
        g = np.ones(dims, dtype=np.float32)
        return g
    rng = np.random.Generator(np.random.SFC64(np.random.SeedSequence([seed, index])))
    rows, cols = dims
    out_dtype = np.float32 if shape.dtype == "fp32" else np.uint16
    out = np.empty(dims, dtype=out_dtype)
    step = max(1, (1 << 24) // cols)  # ~64 MB fp32 chunks bound the temporaries
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        blk = rng.standard_normal((r1 - r0, cols), dtype=np.float32)
        blk *= np.float32(std)
        if shape.dtype == "fp32":
            out[r0:r1] = blk
        else:
            out[r0:r1] = bf16_bits_from_f32(blk)
    return out


def make_weights(shape: ModelShape, seed: int = 0, std: float = 0.02, threads: int = 8) -> Dict[str, np.ndarray]:
    """All tensors of the decoder, N(0, std) (norm gains 1).

    fp32 shapes give float32 arrays.  bf16 shapes give uint16 arrays of bf16 bit
    patterns for the matrices (that *is* the stored weight) and float32 gains.
    Layout is row-major ``[out_features, in_features]``.
    """
    names = weight_names(shape)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        arrs = list(ex.map(lambda t: _gen_one(shape, t[1], t[0], seed, std), enumerate(names)))
    return dict(zip(names, arrs))


def make_prompt(n_tokens: int, vocab: int, seed: int = 1) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(key=[seed, 0]))
    return rng.integers(0, vocab, size=n_tokens, dtype=np.int64).astype(np.int32)


def build_reference(
    y_star: Sequence[int],
    doc_lengths: Sequence[int],
    overlap: float,
    vocab: int,
    span_len: Tuple[int, int] = (4, 16),
    seed: int = 0,
) -> Tuple[np.ndarray, np.ndarray, Dict[str, float]]:
    """Splice spans of ``y_star`` with filler tokens into reference documents.

    Walk ``y_star`` left to right marking spans (lengths uniform in ``span_len``)
    separated by at least one unmarked token until a fraction ``overlap`` of its
    tokens is marked.  The marked spans, in order, are laid out over documents of
    the given lengths with filler in between; a span never crosses a document
    boundary.  Filler ids are drawn from ids that do not occur in ``y_star``
    whenever such ids exist, so filler cannot add overlap by accident.

    Returns (tokens int32[R], doc_offsets int32[n_docs+1], info) where info holds
    the realised coverage and span count.
    """
    y = np.asarray(y_star, dtype=np.int64)
    n = len(y)
    lay = np.random.Generator(np.random.Philox(key=[3, seed]))
    fil = np.random.Generator(np.random.Philox(key=[2, seed]))
    lo, hi = span_len

    # --- mark spans on y* ------------------------------------------------------
    spans: List[Tuple[int, int]] = []
    covered, i = 0, 0
    want = overlap * n
    while i < n and covered < want:
        ln = int(lay.integers(lo, hi + 1))
        ln = min(ln, n - i, max(1, int(round(want - covered))))
        spans.append((i, i + ln))
        covered += ln
        # gap sized so that the long-run marked fraction is ``overlap``
        mean_gap = ln * (1.0 - overlap) / max(overlap, 1e-6)
        gap = max(1, int(round(mean_gap * float(lay.uniform(0.5, 1.5)))))
        i += ln + gap

    # --- filler alphabet -----------------------------------------------------------
    present = np.zeros(vocab, dtype=bool)
    present[y[(y >= 0) & (y < vocab)]] = True
    absent = np.nonzero(~present)[0]
    def filler(m: int) -> np.ndarray:
        if m <= 0:
            return np.zeros(0, dtype=np.int64)
        if len(absent) > 0:
            return absent[fil.integers(0, len(absent), size=m)]
        return fil.integers(0, vocab, size=m)

    # --- lay spans out over the documents -----------------------------------------
    total = int(sum(doc_lengths))
    span_tokens = sum(b - a for a, b in spans)
    slack = max(0, total - span_tokens)
    per_gap = slack // (len(spans) + len(doc_lengths)) if spans else 0
    docs: List[np.ndarray] = []
    si = 0
    placed = 0
    for dl in doc_lengths:
        parts: List[np.ndarray] = []
        room = int(dl)
        while si < len(spans):
            a, b = spans[si]
            lead = min(per_gap, max(0, room - (b - a)))
            if (b - a) + lead > room:
                break
            parts.append(filler(lead))
            parts.append(y[a:b])
            room -= lead + (b - a)
            placed += b - a
            si += 1
        parts.append(filler(room))
        doc = np.concatenate(parts) if parts else np.zeros(0, dtype=np.int64)
        assert len(doc) == dl
        docs.append(doc)
    tokens = np.concatenate(docs).astype(np.int32) if docs else np.zeros(0, dtype=np.int32)
    offsets = np.zeros(len(doc_lengths) + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(np.asarray(doc_lengths, dtype=np.int64))
    info = {
        "nominal_overlap": float(overlap),
        "marked_fraction": covered / max(n, 1),
        "placed_fraction": placed / max(n, 1),
        "n_spans": float(si),
    }
    return tokens, offsets, info

"""ctypes view of the C oracle forward (test infrastructure only).

``OracleModel.forward(token, pos)`` returns the next-token logits of the decoder
after ``token`` has been placed at position ``pos`` (its K/V rows overwrite cache
row ``pos``; it attends to rows ``0..pos``).  Eq. 2 of the paper takes the argmax
of exactly these logits; Eq. 3 is the same quantity at k+1 consecutive positions.
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, Optional

import numpy as np

from . import build as _build


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "d_model", "n_heads", "head_dim", "d_ffn", "vocab",
        "weights_bf16", "kv_round_bf16", "max_seq")] + [("rms_eps", C.c_float), ("rope_theta", C.c_float)]


class _Weights(C.Structure):
    _fields_ = [
        ("tok_emb", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
        ("attn_norm", C.POINTER(C.c_void_p)),
        ("wq", C.POINTER(C.c_void_p)), ("wk", C.POINTER(C.c_void_p)), ("wv", C.POINTER(C.c_void_p)),
        ("wo", C.POINTER(C.c_void_p)),
        ("ffn_norm", C.POINTER(C.c_void_p)),
        ("w_gate", C.POINTER(C.c_void_p)), ("w_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p)),
    ]


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.oracle_create.restype = C.c_void_p
        L.oracle_create.argtypes = [C.POINTER(_Cfg), C.POINTER(_Weights)]
        L.oracle_destroy.argtypes = [C.c_void_p]
        L.oracle_forward.restype = C.c_int32
        L.oracle_forward.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.oracle_prescribe_kv.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_double, C.c_void_p]
        L.oracle_read_cache.restype = C.c_int32
        L.oracle_read_cache.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        L.oracle_round_bf16.restype = C.c_float
        L.oracle_round_bf16.argtypes = [C.c_float]
        L.oracle_matvec.argtypes = [C.c_void_p, C.c_int32, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]
        L.oracle_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_float, C.c_void_p]
        L.oracle_rope.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_float]
        L.oracle_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int64, C.c_int32,
                                       C.c_void_p, C.c_void_p]
        L.oracle_silu_mul.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        _lib = L
    return _lib


def _p(a: np.ndarray) -> int:
    return a.ctypes.data


# ---- thin wrappers of the C primitives (used by the pin tests) ---------------------------

def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    x = np.ascontiguousarray(x, np.float32); g = np.ascontiguousarray(g, np.float32)
    out = np.empty_like(x)
    lib().oracle_rmsnorm(_p(x), _p(g), x.size, eps, _p(out))
    return out


def rope(vec: np.ndarray, pos: int, theta: float) -> np.ndarray:
    v = np.array(vec, dtype=np.float32, copy=True)
    lib().oracle_rope(_p(v), v.size, pos, theta)
    return v


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """q [hd], K/V [n_pos, hd] -> softmax(q K^T / sqrt(hd)) V."""
    q = np.ascontiguousarray(q, np.float32)
    K = np.ascontiguousarray(K, np.float32); V = np.ascontiguousarray(V, np.float32)
    n_pos, hd = K.shape
    out = np.empty(hd, np.float32); scores = np.empty(n_pos, np.float64)
    lib().oracle_attention(_p(q), _p(K), _p(V), n_pos, hd, hd, _p(out), _p(scores))
    return out


def matvec(W: np.ndarray, x: np.ndarray) -> np.ndarray:
    """W float32 or uint16 (bf16 bit patterns), row-major [rows, cols]."""
    W = np.ascontiguousarray(W); x = np.ascontiguousarray(x, np.float32)
    out = np.empty(W.shape[0], np.float32)
    lib().oracle_matvec(_p(W), int(W.dtype == np.uint16), W.shape[0], W.shape[1], _p(x), _p(out))
    return out


def silu_mul(g: np.ndarray, u: np.ndarray) -> np.ndarray:
    g = np.ascontiguousarray(g, np.float32); u = np.ascontiguousarray(u, np.float32)
    out = np.empty_like(g)
    lib().oracle_silu_mul(_p(g), _p(u), g.size, _p(out))
    return out


def round_bf16(x: float) -> float:
    return float(lib().oracle_round_bf16(float(x)))


# ---- the model -------------------------------------------------------------

class OracleModel:
    """One-token-at-a-time decoder with a position-indexed K/V cache."""

    def __init__(self, shape, weights: Dict[str, np.ndarray], max_seq: int, kv_round_bf16: Optional[bool] = None):
        self.shape = shape
        self.vocab = shape.vocab
        self.max_seq = max_seq
        bf16 = shape.dtype == "bf16"
        if kv_round_bf16 is None:
            kv_round_bf16 = bf16
        want = np.uint16 if bf16 else np.float32
        self._keep = {}
        for name, arr in weights.items():
            dt = np.float32 if arr.ndim == 1 else want
            a = np.ascontiguousarray(arr, dtype=dt) if arr.dtype != dt else np.ascontiguousarray(arr)
            self._keep[name] = a
        L = shape.n_layers

        def arr_of(prefix):
            t = (C.c_void_p * L)(*[_p(self._keep[f"{prefix}.{l}"]) for l in range(L)])
            self._keep["_ptrs_" + prefix] = t
            return C.cast(t, C.POINTER(C.c_void_p))

        w = _Weights(_p(self._keep["tok_emb"]), _p(self._keep["lm_head"]), _p(self._keep["final_norm"]),
                     arr_of("attn_norm"), arr_of("wq"), arr_of("wk"), arr_of("wv"), arr_of("wo"),
                     arr_of("ffn_norm"), arr_of("w_gate"), arr_of("w_up"), arr_of("w_down"))
        cfg = _Cfg(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn, shape.vocab,
                   int(bf16), int(bool(kv_round_bf16)), max_seq, shape.rms_eps, shape.rope_theta)
        self.code_stats = np.zeros(4, np.float64)
        self._h = lib().oracle_create(C.byref(cfg), C.byref(w))
        if not self._h:
            raise MemoryError("oracle_create failed")

    def forward(self, token: int, pos: int, want_logits: bool = True, given_kv=None, code_tol: float = 1e-4
                ) -> Optional[np.ndarray]:
        """``given_kv = (K, V)``, float32 [n_layers, H*hd]: prescribed bf16 cache codes of this position.  A code
        is adopted only if rounding some value within ``code_tol * max(1, max|row|)`` of the oracle's own unrounded
        value gives it; ``self.code_stats`` = differing elements, violations, largest share of the tolerance used,
        elements seen."""
        out = np.empty(self.vocab, np.float32) if want_logits else None
        if given_kv is not None:
            gk = np.ascontiguousarray(given_kv[0], np.float32); gv = np.ascontiguousarray(given_kv[1], np.float32)
            assert gk.shape == gv.shape == (self.shape.n_layers, self.shape.n_heads * self.shape.head_dim)
            self._given = (gk, gv)                      # kept alive across the call
            lib().oracle_prescribe_kv(self._h, _p(gk), _p(gv), float(code_tol), _p(self.code_stats))
        rc = lib().oracle_forward(self._h, int(token), int(pos), _p(out) if want_logits else None, None)
        if rc != 0:
            raise ValueError(f"oracle_forward({token}, {pos}) rejected its arguments")
        return out

    def hidden(self, token: int, pos: int) -> np.ndarray:
        out = np.empty(self.shape.d_model, np.float32)
        rc = lib().oracle_forward(self._h, int(token), int(pos), None, _p(out))
        if rc != 0:
            raise ValueError("oracle_forward rejected its arguments")
        return out

    def read_cache(self, layer: int, pos: int, which: int) -> np.ndarray:
        out = np.empty(self.shape.n_heads * self.shape.head_dim, np.float32)
        if lib().oracle_read_cache(self._h, layer, pos, which, _p(out)) != 0:
            raise ValueError("bad cache index")
        return out

    def close(self) -> None:
        if self._h:
            lib().oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

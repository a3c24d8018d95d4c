"""ctypes binding of include/llma.h (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libllma_b200.so")

LLMA_DTYPE_F32, LLMA_DTYPE_BF16 = 0, 1
LLMA_GEMM_AUTO, LLMA_GEMM_SIMT, LLMA_GEMM_TCGEN05 = 0, 1, 2


class LlmaConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ffn", "vocab", "dtype",
                                         "max_batch", "max_seq", "max_ref", "max_k")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("eos_id", C.c_int32),
                ("gemm_impl", C.c_int32), ("keep_logits", C.c_int32)]


class LlmaWeights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm",
                                                     "w_gate", "w_up", "w_down")]


class LlmaStats(C.Structure):
    _fields_ = [("steps", C.c_int64), ("trigger_steps", C.c_int64), ("copied_accepted", C.c_int64),
                ("tokens", C.c_int64), ("launches", C.c_int64), ("device_ms", C.c_float)]


class LlmaStepInfo(C.Structure):
    _fields_ = [("pos", C.c_int32), ("k_eff", C.c_int32), ("accepted", C.c_int32), ("emitted", C.c_int32)]


K_NAMES = ("plan", "embed", "norm", "gemm_qkv", "attn", "gemm_o", "gemm_gateup", "gemm_down", "gemm_lmhead",
           "argmax", "accept", "epilogue")


class LlmaProfile(C.Structure):
    _fields_ = [("ms", C.c_double * len(K_NAMES)), ("launches", C.c_int64 * len(K_NAMES)),
                ("steps", C.c_int64), ("total_ms", C.c_double)]


class LlmaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().llma_strerror(status).decode()
        extra = f" (CUDA error {lib().llma_last_cuda_error()})" if status == -7 else ""
        super().__init__(f"{where}: {msg}{extra} [{status}]")


_lib = None

EXPORTS = ("llma_create", "llma_destroy", "llma_prefill", "llma_set_reference", "llma_step", "llma_generate",
           "llma_rewind", "llma_set_adaptive_k", "llma_reset", "llma_last_step_info", "llma_debug_logits", "llma_debug_kv_row",
           "llma_kv_len", "llma_debug_buffer", "llma_gemm_impl", "llma_profile_steps", "llma_gemm_rows32_bf16", "llma_microbench_mma",
           "llma_gemm_rows32_bf16_noalloc", "llma_generate_forced", "llma_debug_set_device_error", "llma_row_capacity", "llma_debug_attention_tiles", "llma_debug_timeline",
           "llma_last_cuda_error", "llma_strerror")


def lib() -> C.CDLL:
    """Load the CUDA library.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2304_04487_b200.build` "
                              "(nvcc, sm_100a); there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, pi32 = C.c_void_p, C.c_int32, C.POINTER(C.c_int32)
        L.llma_create.argtypes = [C.POINTER(LlmaConfig), C.POINTER(LlmaWeights), vp, C.POINTER(vp)]
        L.llma_destroy.argtypes = [vp]
        L.llma_prefill.argtypes = [vp, i32, pi32, i32]
        L.llma_set_reference.argtypes = [vp, i32, pi32, i32, pi32, i32]
        L.llma_step.argtypes = [vp, i32, i32, pi32, pi32]
        L.llma_generate.argtypes = [vp, i32, i32, i32, pi32, pi32, C.POINTER(LlmaStats)]
        L.llma_rewind.argtypes = [vp, i32]
        L.llma_microbench_mma.argtypes = [i32, i32, i32, i32, C.POINTER(C.c_double)]
        L.llma_set_adaptive_k.argtypes = [vp, i32, i32, i32]
        L.llma_reset.argtypes = [vp, i32]
        L.llma_last_step_info.argtypes = [vp, C.POINTER(LlmaStepInfo)]
        L.llma_debug_logits.argtypes = [vp, C.POINTER(C.c_float)]
        L.llma_debug_kv_row.argtypes = [vp, i32, i32, i32, i32, C.POINTER(C.c_float)]
        L.llma_kv_len.argtypes = [vp, i32]
        L.llma_gemm_impl.argtypes = [vp]
        L.llma_row_capacity.argtypes = [vp]
        L.llma_debug_attention_tiles.argtypes = [vp]
        L.llma_debug_timeline.argtypes = [vp, i32, vp]
        L.llma_debug_set_device_error.argtypes = [vp, i32]
        L.llma_generate_forced.argtypes = [vp, i32, pi32, i32, pi32, i32, C.POINTER(LlmaStats)]
        L.llma_debug_buffer.argtypes = [vp, i32, C.POINTER(C.c_float), C.c_int64]
        L.llma_gemm_rows32_bf16.argtypes = [vp, vp, vp, i32, i32, vp]
        L.llma_gemm_rows32_bf16_noalloc.argtypes = [vp, vp, vp, i32, i32, vp]
        L.llma_profile_steps.argtypes = [vp, i32, i32, i32, C.POINTER(LlmaProfile)]
        L.llma_last_cuda_error.argtypes = []
        L.llma_strerror.argtypes = [C.c_int]
        L.llma_strerror.restype = C.c_char_p
        for name in EXPORTS:
            if name != "llma_strerror":
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _pi32(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def llma_gemm_rows32_bf16(W, a, out, stream=None) -> None:
    """W [n_out, k_in] bf16, a [32, k_in] bf16, out [32, n_out] fp32: CUDA torch tensors (device memory only)."""
    import torch
    assert W.dtype == torch.bfloat16 and a.dtype == torch.bfloat16 and out.dtype == torch.float32
    assert W.is_contiguous() and a.is_contiguous() and out.is_contiguous() and a.shape[0] == 32
    n_out, k_in = W.shape
    assert a.shape[1] == k_in and tuple(out.shape) == (32, n_out)
    st = stream if stream is not None else torch.cuda.current_stream(W.device)
    rc = lib().llma_gemm_rows32_bf16(W.data_ptr(), a.data_ptr(), out.data_ptr(), n_out, k_in, st.cuda_stream)
    if rc != 0:
        raise LlmaError(rc, "llma_gemm_rows32_bf16")


def llma_gemm_rows32_bf16_noalloc(W, a, out, stream=None) -> None:
    """Same product as ``llma_gemm_rows32_bf16`` through the entry point that allocates nothing
    (its scratch is a fixed array inside the library).  For callers that may not call
    cudaMalloc; calls on one device must not overlap."""
    import torch
    assert W.dtype == torch.bfloat16 and a.dtype == torch.bfloat16 and out.dtype == torch.float32
    assert W.is_contiguous() and a.is_contiguous() and out.is_contiguous() and a.shape[0] == 32
    n_out, k_in = W.shape
    assert a.shape[1] == k_in and tuple(out.shape) == (32, n_out)
    st = stream if stream is not None else torch.cuda.current_stream(W.device)
    rc = lib().llma_gemm_rows32_bf16_noalloc(W.data_ptr(), a.data_ptr(), out.data_ptr(), n_out, k_in, st.cuda_stream)
    if rc != 0:
        raise LlmaError(rc, "llma_gemm_rows32_bf16_noalloc")


def llma_microbench_mma(n: int, regions: int = 1, groups: int = 512, commits_per_group: int = 0) -> float:
    """Nanoseconds one M128 x n x K16 bf16 tcgen05.mma occupies the tensor core (see include/llma.h)."""
    ns = C.c_double(0.0)
    rc = lib().llma_microbench_mma(n, regions, groups, commits_per_group, C.byref(ns))
    if rc != 0:
        raise LlmaError(rc, "llma_microbench_mma")
    return float(ns.value)


class Engine:
    """Owns the device copies of the weights (torch tensors: device memory only) and one
    ``llma_engine``.  Method names follow the C entry points."""

    def __init__(self, shape, weights: Dict[str, np.ndarray], max_seq: int, max_ref: int, max_k: int,
                 max_batch: int = 1, eos_id: int = -1, gemm_impl: int = LLMA_GEMM_AUTO, keep_logits: bool = False,
                 device: str = "cuda:0", stream=None, share_weights_with: "Engine" = None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the LLMA engine has no CPU path")
        self._torch = torch
        self.shape = shape
        self.max_k, self.max_batch, self.max_seq = max_k, max_batch, max_seq
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        bf16 = shape.dtype == "bf16"
        self._dev: Dict[str, "torch.Tensor"] = {}
        if share_weights_with is not None:        # a second engine over the same device copies of the weights
            self._dev = share_weights_with._dev
            weights = {}
        for name, arr in weights.items():
            if arr.ndim == 1:
                t = torch.from_numpy(np.ascontiguousarray(arr, np.float32)).to(self.device)
            elif bf16:
                assert arr.dtype == np.uint16, "bf16 shapes take uint16 bit patterns"
                t = torch.from_numpy(arr.view(np.int16)).to(self.device).view(torch.bfloat16)
            else:
                t = torch.from_numpy(np.ascontiguousarray(arr, np.float32)).to(self.device)
            self._dev[name] = t.contiguous()
        L = shape.n_layers
        self._ptr_arrays = {}

        def arr_of(prefix):
            a = (C.c_void_p * L)(*[self._dev[f"{prefix}.{l}"].data_ptr() for l in range(L)])
            self._ptr_arrays[prefix] = a
            return C.cast(a, C.POINTER(C.c_void_p))

        w = LlmaWeights(self._dev["tok_emb"].data_ptr(), self._dev["lm_head"].data_ptr(),
                        self._dev["final_norm"].data_ptr(), arr_of("attn_norm"), arr_of("wq"), arr_of("wk"),
                        arr_of("wv"), arr_of("wo"), arr_of("ffn_norm"), arr_of("w_gate"), arr_of("w_up"),
                        arr_of("w_down"))
        self.cfg = LlmaConfig(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn, shape.vocab,
                              LLMA_DTYPE_BF16 if bf16 else LLMA_DTYPE_F32, max_batch, max_seq, max_ref, max_k,
                              shape.rms_eps, shape.rope_theta, eos_id, gemm_impl, int(keep_logits))
        self._stream = stream if stream is not None else torch.cuda.Stream(self.device)
        h = C.c_void_p()
        torch.cuda.synchronize(self.device)
        rc = lib().llma_create(C.byref(self.cfg), C.byref(w), C.c_void_p(self._stream.cuda_stream), C.byref(h))
        if rc != 0:
            raise LlmaError(rc, "llma_create")
        self._h = h

    @property
    def stream(self):
        return self._stream

    def _check(self, rc: int, where: str) -> int:
        if rc < 0:
            raise LlmaError(rc, where)
        return rc

    def llma_prefill(self, seq: int, prompt: Sequence[int]) -> None:
        p = _i32(prompt)
        self._check(lib().llma_prefill(self._h, seq, _pi32(p), len(p)), "llma_prefill")

    def llma_set_reference(self, seq: int, tokens: Sequence[int], doc_offsets: Optional[Sequence[int]] = None) -> None:
        t = _i32(tokens)
        if doc_offsets is None:
            rc = lib().llma_set_reference(self._h, seq, _pi32(t), len(t), None, 1)
        else:
            o = _i32(doc_offsets)
            rc = lib().llma_set_reference(self._h, seq, _pi32(t), len(t), _pi32(o), len(o) - 1)
        self._check(rc, "llma_set_reference")

    def llma_step(self, n: int, k: int) -> List[List[int]]:
        out = np.zeros((self.max_batch, self.max_k + 1), np.int32)
        cnt = np.zeros(self.max_batch, np.int32)
        self._check(lib().llma_step(self._h, n, k, _pi32(out), _pi32(cnt)), "llma_step")
        return [out[s, :cnt[s]].tolist() for s in range(self.max_batch)]

    def llma_generate(self, max_new: int, n: int, k: int) -> Tuple[List[List[int]], LlmaStats]:
        out = np.zeros((self.max_batch, max(max_new, 1)), np.int32)
        cnt = np.zeros(self.max_batch, np.int32)
        st = LlmaStats()
        self._check(lib().llma_generate(self._h, max_new, n, k, _pi32(out), _pi32(cnt), C.byref(st)), "llma_generate")
        return [out[s, :cnt[s]].tolist() for s in range(self.max_batch)], st

    def llma_debug_attention_tiles(self) -> int:
        return int(lib().llma_debug_attention_tiles(self._h))

    def llma_rewind(self, seq: int) -> None:
        self._check(lib().llma_rewind(self._h, seq), "llma_rewind")

    def llma_set_adaptive_k(self, seq: int, k_min: int, k_start: int) -> None:
        self._check(lib().llma_set_adaptive_k(self._h, seq, k_min, k_start), "llma_set_adaptive_k")

    def llma_reset(self, seq: int) -> None:
        self._check(lib().llma_reset(self._h, seq), "llma_reset")

    def llma_last_step_info(self) -> List[LlmaStepInfo]:
        arr = (LlmaStepInfo * self.max_batch)()
        self._check(lib().llma_last_step_info(self._h, arr), "llma_last_step_info")
        return list(arr)

    def llma_debug_logits(self) -> np.ndarray:
        rows = self.max_batch * (self.max_k + 1)
        out = np.empty((rows, self.shape.vocab), np.float32)
        self._check(lib().llma_debug_logits(self._h, out.ctypes.data_as(C.POINTER(C.c_float))), "llma_debug_logits")
        return out

    def llma_debug_kv_row(self, layer: int, seq: int, pos: int, which: int) -> np.ndarray:
        out = np.empty(self.shape.n_heads * self.shape.head_dim, np.float32)
        self._check(lib().llma_debug_kv_row(self._h, layer, seq, pos, which,
                                            out.ctypes.data_as(C.POINTER(C.c_float))), "llma_debug_kv_row")
        return out

    def llma_debug_buffer(self, which: int) -> np.ndarray:
        sh = self.shape
        cols = (sh.d_model, 3 * sh.n_heads * sh.head_dim, sh.n_heads * sh.head_dim, sh.d_ffn)[which]
        out = np.empty((self.llma_row_capacity(), cols), np.float32)
        self._check(lib().llma_debug_buffer(self._h, which, out.ctypes.data_as(C.POINTER(C.c_float)), out.size),
                    "llma_debug_buffer")
        return out

    def llma_kv_len(self, seq: int) -> int:
        return self._check(lib().llma_kv_len(self._h, seq), "llma_kv_len")

    def llma_profile_steps(self, n: int, k: int, steps: int) -> Dict[str, Dict[str, float]]:
        pr = LlmaProfile()
        self._check(lib().llma_profile_steps(self._h, n, k, steps, C.byref(pr)), "llma_profile_steps")
        out = {name: {"ms_per_step": pr.ms[i] / pr.steps, "launches_per_step": pr.launches[i] / pr.steps}
               for i, name in enumerate(K_NAMES) if pr.launches[i]}
        out["_total"] = {"ms_per_step": pr.total_ms / pr.steps, "launches_per_step": float(sum(pr.launches)) / pr.steps}
        return out

    def llma_row_capacity(self) -> int:
        return self._check(lib().llma_row_capacity(self._h), "llma_row_capacity")

    def llma_debug_timeline(self, clear: bool = True) -> np.ndarray:
        """Timestamps of the last step's kernels, uint64 [512, 160, 8] (a library built with LLMA_STAMPS only)."""
        out = np.zeros((512, 160, 8), np.uint64)
        self._check(lib().llma_debug_timeline(self._h, int(clear), out.ctypes.data), "llma_debug_timeline")
        return out

    def llma_debug_set_device_error(self, code: int) -> None:
        self._check(lib().llma_debug_set_device_error(self._h, code), "llma_debug_set_device_error")

    def llma_generate_forced(self, seq: int, trace: Sequence[Tuple[int, int]], target: Sequence[int]) -> LlmaStats:
        """trace: (input rows, emitted tokens) per step, as Algorithm 2 produces them; target: the text."""
        t = _i32(np.asarray(trace, np.int32).reshape(-1, 2))
        g = _i32(target)
        st = LlmaStats()
        self._check(lib().llma_generate_forced(self._h, seq, _pi32(t), len(t), _pi32(g), len(g), C.byref(st)),
                    "llma_generate_forced")
        return st

    def llma_gemm_impl(self) -> int:
        return self._check(lib().llma_gemm_impl(self._h), "llma_gemm_impl")

    def llma_destroy(self) -> None:
        if getattr(self, "_h", None):
            lib().llma_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.llma_destroy()
        except Exception:
            pass

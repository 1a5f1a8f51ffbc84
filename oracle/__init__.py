"""ctypes loader for the CPU oracle (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this package; the
product path never does.  `build()` compiles `fastcot_oracle.c` with gcc into this folder.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fastcot_oracle.c")
_LIB = os.path.join(_HERE, "libfastcot_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", _LIB, "-lm"])
    return _LIB


class _Shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim",
                                         "d_ffn", "vocab", "wdtype")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("bias_beta", C.c_float),
                ("max_seq", C.c_int32), ("kv_bf16", C.c_int32)]


_PP = C.POINTER(C.c_void_p)


class _Weights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p)] + \
               [(n, _PP) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "g_attn", "g_ffn")] + \
               [("g_final", C.c_void_p), ("lm_head", C.c_void_p), ("bias_perm", C.c_void_p)]


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.orc_new.restype = C.c_void_p
        lib.orc_new.argtypes = [C.POINTER(_Shape), C.POINTER(_Weights)]
        lib.orc_free.argtypes = [C.c_void_p]
        lib.orc_set_trace.argtypes = [C.c_void_p] + [C.c_void_p] * 3
        lib.orc_kv_len.argtypes = [C.c_void_p]
        lib.orc_n_gen.argtypes = [C.c_void_p]
        lib.orc_set_kv.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int]
        lib.orc_get_kv.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int]
        lib.orc_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        lib.orc_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int]
        lib.orc_jacobi_step.argtypes = [C.c_void_p] + [C.c_void_p] * 5
        lib.orc_generate.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.orc_set_window.argtypes = [C.c_void_p, C.c_int]
        lib.orc_finish_with_trigger.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]
        lib.orc_ar_generate.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                        C.c_void_p, C.c_void_p]
        lib.orc_round_bf16.restype = C.c_float
        lib.orc_round_bf16.argtypes = [C.c_float]
        lib.orc_accept.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int,
                                   C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.orc_linear_add.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p]
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().orc_threads())


def _host(t: torch.Tensor) -> torch.Tensor:
    return t.detach().to("cpu").contiguous()


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def round_bf16(x: float) -> float:
    return float(_load().orc_round_bf16(C.c_float(x)))


def accept(window, argmax, n_gen: int, prompt, refill: int = 0, pad_id: int = 0):
    """Verification + buffer update on plain arrays.  Returns (k, accepted[k], new_window[c])."""
    w, a, p = _i32(window), _i32(argmax), _i32(prompt)
    c = w.shape[0]
    k = C.c_int32(0)
    acc, w2 = np.empty(c, np.int32), np.empty(c, np.int32)
    _load().orc_accept(w.ctypes.data, a.ctypes.data, c, n_gen, p.ctypes.data, p.shape[0], refill, pad_id,
                       C.addressof(k), acc.ctypes.data, w2.ctypes.data)
    return int(k.value), acc[:k.value].copy(), w2


def linear_add(w: torch.Tensor, x: np.ndarray, y: np.ndarray) -> np.ndarray:
    """y + x . w^T with the oracle's fp32 dot product; w fp32 or bf16 [N, K], x [R, K], y [R, N]."""
    wh = _host(w)
    x = np.ascontiguousarray(x, np.float32)
    out = np.ascontiguousarray(y, np.float32).copy()
    _load().orc_linear_add(wh.data_ptr(), 0 if wh.dtype == torch.float32 else 1, wh.shape[0], wh.shape[1],
                           x.ctypes.data, x.shape[0], out.ctypes.data)
    return out


class Oracle:
    """One sequence's decoder + Jacobi state on the CPU.

    `weights` is the dict produced by the workload generator (torch tensors, fp32 or bf16);
    bf16 tensors are handed to C as raw bit patterns and up-converted exactly there.  For a bf16 model
    the K and V rows are rounded to bf16 where they are stored (kv_bf16, default = the weights' dtype):
    the cache holds the model dtype; the arithmetic stays fp32.
    """

    def __init__(self, cfg, weights: Dict[str, object], max_seq: int, kv_bf16: Optional[bool] = None):
        lib = _load()
        self.cfg, self.max_seq = cfg, max_seq
        self._keep: List[object] = []
        wd = 0 if cfg.dtype == "f32" else 1

        def ptr(t: torch.Tensor) -> int:
            h = _host(t)
            assert h.dtype == (torch.float32 if wd == 0 else torch.bfloat16)
            self._keep.append(h)
            return h.data_ptr()

        def ptrs(ts: Sequence[torch.Tensor]):
            arr = (C.c_void_p * len(ts))(*[ptr(t) for t in ts])
            self._keep.append(arr)
            return C.cast(arr, _PP)

        self._shape = _Shape(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim,
                             cfg.d_ffn, cfg.vocab, wd, cfg.rms_eps, cfg.rope_theta, cfg.bias_beta, max_seq,
                             int((wd == 1) if kv_bf16 is None else kv_bf16))
        perm = weights.get("bias_perm")
        perm_ptr = None
        if perm is not None:
            p = _host(perm).to(torch.int32)
            self._keep.append(p)
            perm_ptr = p.data_ptr()
        self._w = _Weights(ptr(weights["tok_emb"]),
                           *[ptrs(weights[n]) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up",
                                                        "w_down", "g_attn", "g_ffn")],
                           ptr(weights["g_final"]), ptr(weights["lm_head"]), perm_ptr)
        self._h = lib.orc_new(C.byref(self._shape), C.byref(self._w))
        if not self._h:
            raise ValueError("orc_new rejected the shape")
        self._lib = lib
        self.c = 0

    def close(self):
        if getattr(self, "_h", None):
            self._lib.orc_free(self._h)
            self._h = None

    __del__ = close

    @property
    def kv_len(self) -> int:
        return self._lib.orc_kv_len(self._h)

    @property
    def n_gen(self) -> int:
        return self._lib.orc_n_gen(self._h)

    def set_kv(self, layer: int, k: np.ndarray, v: np.ndarray):
        k = np.ascontiguousarray(k, dtype=np.float32)
        v = np.ascontiguousarray(v, dtype=np.float32)
        rc = self._lib.orc_set_kv(self._h, layer, k.ctypes.data, v.ctypes.data, k.shape[0])
        assert rc == 0, rc

    def get_kv(self, layer: int, length: int):
        kvd = self.cfg.n_kv_heads * self.cfg.head_dim
        k, v = np.empty((length, kvd), np.float32), np.empty((length, kvd), np.float32)
        rc = self._lib.orc_get_kv(self._h, layer, k.ctypes.data, v.ctypes.data, length)
        assert rc == 0, rc
        return k, v

    def forward(self, tokens, want_logits: bool = True, trace: bool = False):
        """Forward rows at positions kv_len.. without committing.  Returns (argmax, logits[, trace])."""
        tok = _i32(tokens)
        n = tok.shape[0]
        logits = np.empty((n, self.cfg.vocab), dtype=np.float32) if want_logits else None
        am = np.empty(n, dtype=np.int32)
        tr = None
        if trace:
            qd = self.cfg.n_heads * self.cfg.head_dim
            tr = {"q": np.empty((n, qd), np.float32), "attn": np.empty((n, qd), np.float32),
                  "x_out": np.empty((n, self.cfg.d_model), np.float32)}
            self._lib.orc_set_trace(self._h, tr["q"].ctypes.data, tr["attn"].ctypes.data,
                                    tr["x_out"].ctypes.data)
        rc = self._lib.orc_forward(self._h, tok.ctypes.data, n,
                                   logits.ctypes.data if want_logits else None, am.ctypes.data)
        if trace:
            self._lib.orc_set_trace(self._h, None, None, None)
        if rc:
            raise RuntimeError(f"orc_forward rc={rc}")
        return (am, logits, tr) if trace else (am, logits)

    def prefill(self, prompt, c: int, refill: int = 0, pad_id: int = 0):
        p = _i32(prompt)
        rc = self._lib.orc_prefill(self._h, p.ctypes.data, p.shape[0], c, refill, pad_id)
        if rc:
            raise RuntimeError(f"orc_prefill rc={rc}")
        self.c = c

    def jacobi_step(self, window_in=None, want_logits: bool = False):
        """Returns (k, accepted_tokens[k], new_window[c][, logits[c, vocab]])."""
        c = self.c
        k = C.c_int32(0)
        acc = np.empty(c, np.int32)
        wout = np.empty(c, np.int32)
        win = _i32(window_in) if window_in is not None else None
        logits = np.empty((c, self.cfg.vocab), np.float32) if want_logits else None
        rc = self._lib.orc_jacobi_step(self._h, win.ctypes.data if win is not None else None,
                                       C.addressof(k), acc.ctypes.data, wout.ctypes.data,
                                       logits.ctypes.data if want_logits else None)
        if rc:
            raise RuntimeError(f"orc_jacobi_step rc={rc}")
        res = (int(k.value), acc[:k.value].copy(), wout)
        return res + (logits,) if want_logits else res

    def generate(self, max_tokens: int, eos_id: int = -1, max_iters: int = 0):
        """Returns (tokens, accept_counts per step)."""
        out = np.empty(max_tokens, np.int32)
        counts = np.zeros(max(max_tokens, 1), np.int32)
        steps = C.c_int32(0)
        n = self._lib.orc_generate(self._h, max_tokens, eos_id, max_iters, out.ctypes.data, counts.ctypes.data,
                                   C.addressof(steps))
        if n < 0:
            raise RuntimeError(f"orc_generate rc={n}")
        return out[:n].copy(), counts[:steps.value].copy()

    def set_window(self, c: int):
        """Change the rows per forward between iterations; returns the resized window."""
        rc = self._lib.orc_set_window(self._h, c)
        if rc:
            raise RuntimeError(f"orc_set_window rc={rc}")
        self.c = c

    def finish_with_trigger(self, trigger, max_answer: int, eos_id: int = -1):
        """Exact + approximate tokens + answer trigger, then greedy answer tokens.  Ends the Jacobi state."""
        t = _i32(trigger)
        out = np.empty(max(max_answer, 1), np.int32)
        n = self._lib.orc_finish_with_trigger(self._h, t.ctypes.data if t.shape[0] else None, t.shape[0],
                                              max_answer, eos_id, out.ctypes.data)
        if n < 0:
            raise RuntimeError(f"orc_finish_with_trigger rc={n}")
        self.c = 0
        return out[:n].copy()

    def ar_generate(self, prompt, max_tokens: int, eos_id: int = -1):
        """Plain greedy decoding.  Returns (tokens, top1-top2 logit margins)."""
        p = _i32(prompt)
        out = np.empty(max_tokens, np.int32)
        mar = np.empty(max_tokens, np.float32)
        n = self._lib.orc_ar_generate(self._h, p.ctypes.data, p.shape[0], max_tokens, eos_id,
                                      out.ctypes.data, mar.ctypes.data)
        if n < 0:
            raise RuntimeError(f"orc_ar_generate rc={n}")
        return out[:n].copy(), mar[:n].copy()

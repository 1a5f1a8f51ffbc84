"""`Decoder`: owns the device buffers (through torch) and forwards every call to the C ABI.

PyTorch is used for device memory and the stream only; every step of the decode path runs in the
CUDA library.  Method names match the C entry points they call.
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, Optional

import numpy as np
import torch

from . import lib as _l


class FcError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        msg = _l.load().fc_strerror(code).decode()
        super().__init__(f"{where}: {msg} ({code}) {detail}".strip())


_GUARD, _GUARD_BYTE = 4096, 0xA5      # canary band on either side of the K/V slab and of the workspace


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


class Decoder:
    def __init__(self, cfg, weights: Dict[str, object], max_batch: int, max_c: int, max_seq: int,
                 flags: int = 0, device: str = "cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU fallback)")
        self.lib = _l.load()
        self.cfg, self.device = cfg, torch.device(device)
        torch.cuda.set_device(self.device)
        dt = _l.FC_F32 if cfg.dtype == "f32" else _l.FC_BF16
        self.shape = _l.fc_model_shape(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim,
                                       cfg.d_ffn, cfg.vocab, dt, cfg.rms_eps, cfg.rope_theta,
                                       max_batch, max_c, max_seq, cfg.bias_beta, flags)
        kvb = self.lib.fc_kv_bytes(C.byref(self.shape))
        wsb = self.lib.fc_workspace_bytes(C.byref(self.shape))
        if kvb == 0 or wsb == 0:
            raise FcError(_l.FC_ERR_SHAPE, "fc_kv_bytes")
        # each buffer sits between two canary bands (checked by fc_debug_check_guards)
        self._kv_bytes, self._ws_bytes = kvb, wsb
        self._kv_alloc = torch.full((kvb + 2 * _GUARD,), _GUARD_BYTE, dtype=torch.uint8, device=self.device)
        self._ws_alloc = torch.full((wsb + 2 * _GUARD,), _GUARD_BYTE, dtype=torch.uint8, device=self.device)
        self.kv = self._kv_alloc[_GUARD:_GUARD + kvb]
        self.ws = self._ws_alloc[_GUARD:_GUARD + wsb]
        self.kv.zero_()
        self.ws.zero_()
        self._keep = []

        def dev(t: torch.Tensor) -> int:
            t = t.to(self.device).contiguous()
            assert t.dtype == cfg.torch_dtype, (t.dtype, cfg.torch_dtype)
            self._keep.append(t)
            return t.data_ptr()

        def table(ts):
            arr = (C.c_void_p * len(ts))(*[dev(t) for t in ts])
            self._keep.append(arr)
            return C.cast(arr, _l._PP)

        perm = weights.get("bias_perm")
        perm_ptr = None
        if perm is not None:
            p = perm.to(self.device, torch.int32).contiguous()
            self._keep.append(p)
            perm_ptr = p.data_ptr()
        self.weights = _l.fc_weights(dev(weights["tok_emb"]),
                                     *[table(weights[n]) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up",
                                                                   "w_down", "g_attn", "g_ffn")],
                                     dev(weights["g_final"]), dev(weights["lm_head"]), perm_ptr)
        self.stream = torch.cuda.current_stream(self.device)
        h = C.c_void_p()
        rc = self.lib.fc_init(C.byref(h), C.byref(self.shape), C.byref(self.weights),
                              self.kv.data_ptr(), kvb, self.ws.data_ptr(), wsb, self.stream.cuda_stream)
        if rc != _l.FC_OK:
            raise FcError(rc, "fc_init")
        self.h = h
        self.batch = self.c = 0
        self._logits: Optional[torch.Tensor] = None

    def close(self):
        if getattr(self, "h", None):
            self.lib.fc_destroy(self.h)
            self.h = None

    __del__ = close

    def _check(self, rc: int, where: str):
        if rc != _l.FC_OK:
            raise FcError(rc, where, self.lib.fc_last_cuda_error(self.h).decode())

    # ---- C ABI calls -------------------------------------------------------------------------
    def fc_prefill(self, prompt_ids, prompt_lens, c: int, refill: int = 0, pad_id: int = 0):
        ids, lens = _i32(prompt_ids), _i32(prompt_lens)
        if ids.ndim == 1:
            ids = ids[None]
        self._check(self.lib.fc_prefill(self.h, ids.shape[0], ids.ctypes.data, ids.shape[1],
                                        lens.ctypes.data, c, refill, pad_id), "fc_prefill")
        self.batch, self.c = ids.shape[0], c

    def fc_jacobi_step(self, window_in=None):
        """Returns (accepted_count [B], accepted_tokens [B, c], window_out [B, c])."""
        B, c = self.batch, self.c
        cnt, tok, win = np.zeros(B, np.int32), np.zeros((B, c), np.int32), np.zeros((B, c), np.int32)
        wi = _i32(window_in).reshape(B, c) if window_in is not None else None
        self._check(self.lib.fc_jacobi_step(self.h, wi.ctypes.data if wi is not None else None,
                                            cnt.ctypes.data, tok.ctypes.data, win.ctypes.data), "fc_jacobi_step")
        return cnt, tok, win

    def fc_generate(self, max_tokens: int, eos_id: int = -1, c: int = 0, max_iters: int = 0):
        """Returns (tokens [B, max_tokens], lens [B], stats).  c = 0 keeps the current window size."""
        B = self.batch
        out, lens = np.zeros((B, max_tokens), np.int32), np.zeros(B, np.int32)
        st = _l.fc_stats()
        self._check(self.lib.fc_generate(self.h, max_tokens, c, eos_id, max_iters, out.ctypes.data, lens.ctypes.data,
                                         C.byref(st)), "fc_generate")
        if c > 0:
            self.c = c
        return out, lens, st

    def fc_set_window(self, c: int):
        self._check(self.lib.fc_set_window(self.h, c), "fc_set_window")
        self.c = c

    def fc_finish_with_trigger(self, trigger_ids, max_answer_tokens: int, eos_id: int = -1):
        """Returns (answer tokens [B, max_answer_tokens], lens [B]).  The sequences need fc_prefill afterwards."""
        B = self.batch
        t = _i32(trigger_ids)
        out, lens = np.zeros((B, max(max_answer_tokens, 1)), np.int32), np.zeros(B, np.int32)
        self._check(self.lib.fc_finish_with_trigger(self.h, t.ctypes.data if t.shape[0] else None, t.shape[0],
                                                    max_answer_tokens, eos_id, out.ctypes.data, lens.ctypes.data),
                    "fc_finish_with_trigger")
        return out[:, :max_answer_tokens], lens

    def fc_debug_inject_timeout(self):
        self._check(self.lib.fc_debug_inject_timeout(self.h), "fc_debug_inject_timeout")

    def fc_debug_check_guards(self) -> int:
        """Number of damaged canary bands: those between the workspace slices (kept by the library) plus the ones
        this binding keeps around the K/V slab and the workspace."""
        n = C.c_int32(0)
        self._check(self.lib.fc_debug_check_guards(self.h, C.byref(n)), "fc_debug_check_guards")
        bad = int(n.value)
        for buf, nbytes in ((self._kv_alloc, self._kv_bytes), (self._ws_alloc, self._ws_bytes)):
            lo, hi = buf[:_GUARD], buf[_GUARD + nbytes:]
            bad += int((lo != _GUARD_BYTE).any().item()) + int((hi != _GUARD_BYTE).any().item())
        return bad

    def fc_debug_set_state(self, kv_lens, pending, c: int, pad_id: int = 0):
        kl, pe = _i32(kv_lens), _i32(pending)
        self._check(self.lib.fc_debug_set_state(self.h, kl.shape[0], kl.ctypes.data, pe.ctypes.data, c, pad_id),
                    "fc_debug_set_state")
        self.batch, self.c = kl.shape[0], c

    def fc_debug_logits(self, enable: bool = True) -> Optional[torch.Tensor]:
        """Device tensor [max_batch*max_c, vocab] that receives the logits of every later step."""
        if enable:
            rows = self.shape.max_batch * self.shape.max_c
            self._logits = torch.zeros(rows, self.cfg.vocab, dtype=torch.float32, device=self.device)
            self._check(self.lib.fc_debug_logits(self.h, self._logits.data_ptr()), "fc_debug_logits")
        else:
            self._check(self.lib.fc_debug_logits(self.h, None), "fc_debug_logits")
            self._logits = None
        return self._logits

    def fc_get_state(self):
        kl, ng = np.zeros(self.batch, np.int32), np.zeros(self.batch, np.int32)
        self._check(self.lib.fc_get_state(self.h, kl.ctypes.data, ng.ctypes.data), "fc_get_state")
        return kl, ng

    def fc_bench_steps(self, n_steps: int, commit: bool = False):
        """Returns (device milliseconds for n_steps back-to-back steps, tokens committed)."""
        ms, tok = C.c_float(0), C.c_int64(0)
        self._check(self.lib.fc_bench_steps(self.h, n_steps, int(commit), C.byref(ms), C.byref(tok)),
                    "fc_bench_steps")
        return float(ms.value), int(tok.value)

    def fc_profile_step(self):
        """Returns {class name: (milliseconds, launches)} for one non-committing step."""
        n = len(_l.FC_CLASSES)
        ms, cnt = (C.c_float * n)(), (C.c_int32 * n)()
        self._check(self.lib.fc_profile_step(self.h, ms, cnt), "fc_profile_step")
        return {name: (float(ms[i]), int(cnt[i])) for i, name in enumerate(_l.FC_CLASSES)}

    def fc_last_launch_count(self) -> int:
        return int(self.lib.fc_last_launch_count(self.h))

    # ---- K/V slab view for the window-step sweep (the caller writes random K/V into it) --------
    def kv_view(self) -> torch.Tensor:
        s = self.shape
        return self.kv.view(self.cfg.torch_dtype).view(s.n_layers, 2, s.max_batch, s.n_kv_heads,
                                                       s.max_seq, s.head_dim)


def fc_op_linear(x: torch.Tensor, w: torch.Tensor, y: torch.Tensor, use_tensor_cores: bool) -> int:
    """y[R, N] += x[R, K] . w[N, K]^T on the device (x, y fp32; w fp32 or bf16)."""
    lib = _l.load()
    R, K = x.shape
    N = w.shape[0]
    assert x.is_cuda and w.is_cuda and y.is_cuda and x.dtype == torch.float32 and y.dtype == torch.float32
    assert x.is_contiguous() and w.is_contiguous() and y.is_contiguous()
    dt = _l.FC_F32 if w.dtype == torch.float32 else _l.FC_BF16
    return lib.fc_op_linear(x.data_ptr(), w.data_ptr(), y.data_ptr(), R, N, K, dt, int(use_tensor_cores),
                            torch.cuda.current_stream().cuda_stream)


def fc_op_accept(window, argmax, kv_len, n_gen, prompt, prompt_lens, refill: int, pad_id: int):
    """Runs the accept kernel on device int32 tensors; returns (accepted_count, accepted_tokens)."""
    lib = _l.load()
    B, c = window.shape
    cnt = torch.zeros(B, dtype=torch.int32, device=window.device)
    tok = torch.zeros(B, c, dtype=torch.int32, device=window.device)
    rc = lib.fc_op_accept(window.data_ptr(), argmax.data_ptr(), kv_len.data_ptr(), n_gen.data_ptr(),
                          cnt.data_ptr(), tok.data_ptr(),
                          prompt.data_ptr() if prompt is not None else None,
                          prompt_lens.data_ptr() if prompt_lens is not None else None,
                          B, c, prompt.shape[1] if prompt is not None else 1, refill, pad_id,
                          torch.cuda.current_stream().cuda_stream)
    if rc != _l.FC_OK:
        raise FcError(rc, "fc_op_accept")
    return cnt, tok


def fc_op_window_attention(q: torch.Tensor, kcache: torch.Tensor, vcache: torch.Tensor, kv_len: torch.Tensor,
                           c: int, n_heads: int, max_len: int) -> torch.Tensor:
    """Window attention of one layer.  q [B*c, n_heads*hd]; kcache/vcache [B, n_kv_heads, max_seq, hd];
    kv_len int32 [B] on the device.  Returns fp32 [B*c, n_heads*hd]."""
    lib = _l.load()
    B, hkv, max_seq, hd = kcache.shape
    dt = _l.FC_F32 if q.dtype == torch.float32 else _l.FC_BF16
    nbytes = lib.fc_op_window_attention_scratch_bytes(B, c, n_heads, hkv, hd, max_len, dt)
    scratch = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=q.device)
    out = torch.empty(B * c, n_heads * hd, dtype=torch.float32, device=q.device)
    rc = lib.fc_op_window_attention(q.data_ptr(), kcache.data_ptr(), vcache.data_ptr(), kv_len.data_ptr(),
                                    out.data_ptr(), B, c, n_heads, hkv, hd, max_seq, max_len, dt,
                                    scratch.data_ptr(), nbytes, torch.cuda.current_stream().cuda_stream)
    if rc != _l.FC_OK:
        raise FcError(rc, "fc_op_window_attention")
    return out


def fc_op_fused_window_attention(qkv_acc: torch.Tensor, sumsq: torch.Tensor, rms_eps: float, d_norm: int,
                                 rope_theta: float, kcache: torch.Tensor, vcache: torch.Tensor, kv_len: torch.Tensor,
                                 c: int, n_heads: int, max_len: int, n_splits: int = 0, q_tiles: int = 0) -> torch.Tensor:
    """The fused attention kernel of the bf16 step as one operation.  qkv_acc fp32 [B*c, (hq + 2 hkv) * hd] and sumsq
    fp32 [B*c] are consumed (cleared); kcache/vcache bf16 [B, hkv, max_seq, hd] receive the window's rows.
    Returns fp32 [B*c, hq*hd]."""
    lib = _l.load()
    B, hkv, max_seq, hd = kcache.shape
    nbytes = lib.fc_op_fused_window_attention_scratch_bytes(B, c, n_heads, hkv, hd, max_seq, max_len)
    if nbytes == 0:
        raise FcError(_l.FC_ERR_ARG, "fc_op_fused_window_attention_scratch_bytes")
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=qkv_acc.device)
    out = torch.empty(B * c, n_heads * hd, dtype=torch.float32, device=qkv_acc.device)
    rc = lib.fc_op_fused_window_attention(qkv_acc.data_ptr(), sumsq.data_ptr(), rms_eps, d_norm, rope_theta,
                                          kcache.data_ptr(), vcache.data_ptr(), kv_len.data_ptr(), out.data_ptr(),
                                          B, c, n_heads, hkv, hd, max_seq, max_len, n_splits, q_tiles,
                                          scratch.data_ptr(), nbytes, torch.cuda.current_stream().cuda_stream)
    if rc != _l.FC_OK:
        raise FcError(rc, "fc_op_fused_window_attention")
    return out

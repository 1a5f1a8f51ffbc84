"""Seeded synthetic inputs for the Jacobi-window decode step.

This module only *generates inputs* (weights, permutation table, prompts, random
K/V).  It holds none of the method's arithmetic, so both the CUDA path and the
CPU oracle may consume its output.  Every value is a pure function of
(seed, tensor id, element index): a counter-based integer hash followed by an
Irwin-Hall sum (12 uniform 16-bit integers), which is exact in integer
arithmetic and therefore bit-identical whether it runs on the CPU or on a GPU.

The synthetic models stand in for the Llama / Llama-2 7B and 13B checkpoints the
paper evaluates (Section 5.1); random prompts of the stated lengths stand in for
its few-shot chain-of-thought prompts.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import torch

_MASK64 = (1 << 64) - 1


@dataclasses.dataclass(frozen=True)
class ModelConfig:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    dtype: str            # "f32" | "bf16"
    bias_beta: float      # logit bonus on token f(prev)
    prompt_len: int
    c: int                # rows per forward (pending exact token + c-1 guesses)
    gen_tokens: int
    batch: int
    seed: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def weight_params(self) -> int:
        """Parameters streamed once per step (all layer matrices + LM head)."""
        d, hq, hkv, hd, f = self.d_model, self.n_heads, self.n_kv_heads, self.head_dim, self.d_ffn
        per_layer = d * hq * hd * 2 + 2 * d * hkv * hd + 3 * d * f
        return self.n_layers * per_layer + self.vocab * d

    def kv_bytes_per_token(self) -> int:
        return 2 * self.n_layers * self.n_kv_heads * self.head_dim * self.elem_bytes


CONFIGS: Dict[str, ModelConfig] = {
    "tiny": ModelConfig("tiny", 2, 128, 4, 4, 32, 512, 512, "f32", 4.0, 32, 8, 64, 1, 1001),
    "1b": ModelConfig("1b", 22, 2048, 32, 4, 64, 5632, 32000, "bf16", 6.0, 512, 16, 256, 1, 1002),
    "7b": ModelConfig("7b", 32, 4096, 32, 32, 128, 11008, 32000, "bf16", 6.0, 800, 16, 256, 1, 1003),
    "13b": ModelConfig("13b", 40, 5120, 40, 40, 128, 13824, 32000, "bf16", 6.0, 1024, 32, 256, 8, 1004),
}


def small_config(name: str = "small", **kw) -> ModelConfig:
    """A few-layer shape for tests; any field can be overridden."""
    base = dict(name=name, n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, head_dim=64,
                d_ffn=512, vocab=1024, dtype="bf16", bias_beta=6.0, prompt_len=40, c=8,
                gen_tokens=32, batch=1, seed=77)
    base.update(kw)
    return ModelConfig(**base)


# ----------------------------------------------------------------------------
# counter-based generator
# ----------------------------------------------------------------------------

def _wrap(v: int) -> int:
    """Python int -> the int64 two's-complement value with the same low 64 bits."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _mix64(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on int64 tensors (wrapping multiply, logical shifts)."""
    def lsr(x, s):
        return (x >> s) & ((1 << (64 - s)) - 1)
    z = (z ^ lsr(z, 30)) * _wrap(0xBF58476D1CE4E5B9)
    z = (z ^ lsr(z, 27)) * _wrap(0x94D049BB133111EB)
    return z ^ lsr(z, 31)


def _key(seed: int, tensor_id: int) -> int:
    k = (seed * 0x9E3779B97F4A7C15 + tensor_id * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & _MASK64
    k ^= k >> 29
    k = (k * 0xBF58476D1CE4E5B9) & _MASK64
    return k


def hash_normal(seed: int, tensor_id: int, numel: int, device="cpu",
                chunk: int = 1 << 24) -> torch.Tensor:
    """`numel` fp32 samples, approximately N(0,1): (sum of 12 uniform u16 - mean) / std.

    All arithmetic before the final scaling is exact integer work; the scaling is
    one fp32 multiply of an exactly representable integer, so the result does not
    depend on the device.
    """
    out = torch.empty(numel, dtype=torch.float32, device=device)
    key = _key(seed, tensor_id)
    inv_std = 1.0 / 65536.0  # std of the sum is sqrt(12 * (2^32 - 1)/12) ~= 65536
    for start in range(0, numel, chunk):
        n = min(chunk, numel - start)
        idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
        acc = torch.zeros(n, dtype=torch.int64, device=device)
        for j in range(3):
            h = _mix64(idx * 3 + j + _wrap(key))
            for s in (0, 16, 32, 48):
                acc += (h >> s) & 0xFFFF
        acc -= 12 * 65535 // 2
        out[start:start + n] = acc.to(torch.float32) * inv_std
    return out


def hash_uniform_int(seed: int, tensor_id: int, numel: int, high: int, device="cpu") -> torch.Tensor:
    """int32 ids uniform in [0, high) (modulo of a 31-bit hash; bias < high / 2^31)."""
    idx = torch.arange(numel, dtype=torch.int64, device=device)
    h = _mix64(idx + _wrap(_key(seed, tensor_id)))
    return (((h >> 17) & 0x7FFFFFFF) % high).to(torch.int32)


# tensor ids: 1 embedding, 2 final gain, 3 lm head, 4 permutation, 5 prompts, 6 random kv,
# 7 random window, 100 + 16*layer + slot for per-layer tensors
_SLOTS = {"wq": 0, "wk": 1, "wv": 2, "wo": 3, "w_gate": 4, "w_up": 5, "w_down": 6,
          "g_attn": 7, "g_ffn": 8}


def make_permutation(vocab: int, seed: int) -> torch.Tensor:
    """The table f: a seeded permutation of 0..vocab-1 (int32, CPU).

    Sorting distinct 64-bit hash keys yields a uniformly random permutation that
    does not depend on any library's random stream.
    """
    idx = torch.arange(vocab, dtype=torch.int64)
    h = _mix64(idx + _wrap(_key(seed, 4)))
    # ties are broken by index through a stable sort, so the table is well defined
    return torch.sort(h, stable=True).indices.to(torch.int32)


def make_weights(cfg: ModelConfig, device="cpu", zero_matrices: bool = False) -> Dict[str, object]:
    """Random-init weights in the model dtype.

    Matrices and the embedding are N(0, 0.02) rounded once to the model dtype and stored
    row-major as [out_features, in_features]; RMSNorm gains are 1 + N(0, 0.1) so that a
    missing gain shows up in the results.  `zero_matrices=True` zeroes every matrix
    (used by a closed-form test where the logits reduce to the permutation bias).
    """
    dt = cfg.torch_dtype
    d, hq, hkv, hd, f, v = cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn, cfg.vocab

    def mat(tid: int, rows: int, cols: int) -> torch.Tensor:
        if zero_matrices:
            return torch.zeros(rows, cols, dtype=dt, device=device)
        return (hash_normal(cfg.seed, tid, rows * cols, device) * 0.02).to(dt).view(rows, cols)

    def gain(tid: int) -> torch.Tensor:
        return (1.0 + 0.1 * hash_normal(cfg.seed, tid, d, device)).to(dt)

    w: Dict[str, object] = {"tok_emb": mat(1, v, d), "g_final": gain(2), "lm_head": mat(3, v, d)}
    shapes = {"wq": (hq * hd, d), "wk": (hkv * hd, d), "wv": (hkv * hd, d), "wo": (d, hq * hd),
              "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f)}
    for name in _SLOTS:
        w[name] = []
    for layer in range(cfg.n_layers):
        base = 100 + 16 * layer
        for name, (r, c) in shapes.items():
            w[name].append(mat(base + _SLOTS[name], r, c))
        w["g_attn"].append(gain(base + _SLOTS["g_attn"]))
        w["g_ffn"].append(gain(base + _SLOTS["g_ffn"]))
    w["bias_perm"] = make_permutation(v, cfg.seed).to(device)
    return w


def make_prompts(cfg: ModelConfig, batch: Optional[int] = None, lens: Optional[List[int]] = None):
    """Uniform-random prompt ids.  Returns (ids int32 [batch, P_max] on CPU, lens int32 [batch])."""
    b = batch if batch is not None else cfg.batch
    lens = lens if lens is not None else [cfg.prompt_len] * b
    pmax = max(lens)
    ids = hash_uniform_int(cfg.seed, 5, b * pmax, cfg.vocab).view(b, pmax).clone()
    for i, n in enumerate(lens):
        ids[i, n:] = 0
    return ids, torch.tensor(lens, dtype=torch.int32)


def make_random_kv(cfg: ModelConfig, numel: int, device="cpu", tensor_id: int = 6) -> torch.Tensor:
    """Cached K/V ~ N(0,1) in the model dtype, flat, for the window-step sweep."""
    return hash_normal(cfg.seed, tensor_id, numel, device).to(cfg.torch_dtype)


def make_random_window(cfg: ModelConfig, batch: int, c: int, salt: int = 0) -> torch.Tensor:
    return hash_uniform_int(cfg.seed + salt, 7, batch * c, cfg.vocab).view(batch, c).clone()

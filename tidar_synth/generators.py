"""Counter-based seeded generators and workload shape tables.

Nothing here belongs to the method (no mask, no attention, no acceptance rule):
only random numbers and shapes.  The generator is splitmix64 used as a counter
hash, so element ``i`` of tensor ``t`` under seed ``s`` is a pure function of
``(s, t, i)``.  All integer work is done on ``torch.int64`` tensors (two's
complement wrap-around), which behaves identically on the host and on a CUDA
device; the normal transform is Box-Muller in float64 followed by one
round-to-nearest-even conversion to bf16.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional

import torch

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB


def _s64(x: int) -> int:
    """Python int -> the signed 64-bit integer with the same low 64 bits."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_int(z: int) -> int:
    z &= _MASK64
    z = ((z ^ (z >> 30)) * _M1) & _MASK64
    z = ((z ^ (z >> 27)) * _M2) & _MASK64
    return z ^ (z >> 31)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right on int64 (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def stream_base(seed: int, tid: int) -> int:
    """Per-(seed, tensor) stream key, a python int in [0, 2^64)."""
    return _mix_int(_mix_int(seed + _GOLDEN) ^ (tid * _M2 + 1))


def splitmix64(seed: int, tid: int, index: torch.Tensor) -> torch.Tensor:
    """64 hash bits (as int64) for each element index of tensor ``tid``."""
    base = stream_base(seed, tid)
    return _mix(index * _s64(_GOLDEN) + _s64(base + _GOLDEN))


def uniform01(seed: int, tid: int, index: torch.Tensor) -> torch.Tensor:
    """float64 uniform in the open interval (0, 1)."""
    bits = _lsr(splitmix64(seed, tid, index), 11)
    return (bits.to(torch.float64) + 0.5) * (1.0 / 9007199254740992.0)


def gen_normal_bf16(seed: int, tid: int, numel: int, std: float, device="cpu",
                    out: Optional[torch.Tensor] = None, chunk: int = 1 << 24) -> torch.Tensor:
    """``numel`` draws of N(0, std^2), rounded once to bf16 (flat tensor)."""
    if out is None:
        out = torch.empty(numel, dtype=torch.bfloat16, device=device)
    assert out.numel() == numel and out.dtype == torch.bfloat16
    flat = out.view(-1)
    for lo in range(0, numel, chunk):
        hi = min(numel, lo + chunk)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=flat.device)
        u1 = uniform01(seed, tid, 2 * idx)
        u2 = uniform01(seed, tid, 2 * idx + 1)
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        flat[lo:hi] = (z * std).to(torch.bfloat16)
    return out


def gen_token_ids(seed: int, tid: int, n: int, vocab_exclusive: int) -> torch.Tensor:
    """``n`` uniform token ids in [0, vocab_exclusive), int32, on the host."""
    idx = torch.arange(n, dtype=torch.int64)
    bits = _lsr(splitmix64(seed, tid, idx), 1)
    return (bits % vocab_exclusive).to(torch.int32)


def acceptance_schedule(seed: int, n_steps: int, k: int, p_accept: float = 0.8969) -> torch.Tensor:
    """Seeded truncated-geometric acceptance lengths in [1, k] (int32, host).

    Each of the k-1 drafts after the always-certain first slot is kept
    independently with probability ``p_accept`` until the first failure.
    With p = 0.8969 and k = 16 the mean is 8.0.
    """
    idx = torch.arange(n_steps * k, dtype=torch.int64)
    u = uniform01(seed, TID_SCHEDULE, idx).view(n_steps, k)
    keep = (u[:, 1:] < p_accept).to(torch.int32)
    run = torch.cumprod(keep, dim=1).sum(dim=1)
    return (1 + run).to(torch.int32)


# ----------------------------------------------------------------------------
# tensor ids
# ----------------------------------------------------------------------------
_KINDS = {
    "embed": 1, "lm_head": 2, "final_norm": 3,
    "attn_norm": 10, "wq": 11, "wk": 12, "wv": 13, "wo": 14,
    "ffn_norm": 15, "w_gate": 16, "w_up": 17, "w_down": 18,
    "bq": 19, "bk": 20, "bv": 21, "q_norm": 22, "k_norm": 23,
    "prompt": 30, "drafts": 31, "q": 40, "k": 41, "v": 42, "perm": 43,
}
TID_SCHEDULE = 50 << 12


def tensor_id(kind: str, layer: int = 0) -> int:
    return (_KINDS[kind] << 12) + layer


# ----------------------------------------------------------------------------
# shapes
# ----------------------------------------------------------------------------
@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    tie_lm_head: bool
    rope_theta: float
    rms_eps: float = 1e-6
    seed: int = 0
    init_std: float = 0.02
    qkv_bias: bool = False       # biases on the Q/K/V projections
    qk_norm: bool = False        # RMSNorm over each head's dimensions of Q and K before RoPE
    # workload
    prompt_len: int = 64
    k: int = 4
    max_new_tokens: int = 32

    @property
    def mask_token_id(self) -> int:
        return self.vocab - 1

    def reduced(self, n_layers: int, vocab: Optional[int] = None) -> "ModelShape":
        """Same widths, fewer layers (and optionally a smaller vocabulary)."""
        return replace(self, name=f"{self.name}-L{n_layers}" + (f"-V{vocab}" if vocab else ""),
                       n_layers=n_layers, vocab=vocab or self.vocab)

    def n_params(self) -> int:
        per_layer = (self.d_model * (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim
                     + self.n_q_heads * self.head_dim * self.d_model
                     + 3 * self.d_model * self.d_ffn)
        head = self.vocab * self.d_model
        return self.n_layers * per_layer + head * (1 if self.tie_lm_head else 2)


CONFIGS: Dict[str, ModelShape] = {
    "tiny": ModelShape("tiny", 2, 256, 4, 2, 64, 704, 1024, True, 10000.0,
                       seed=0, prompt_len=64, k=4, max_new_tokens=32),
    "1.5b": ModelShape("1.5b", 28, 1536, 12, 2, 128, 8960, 151936, False, 1.0e6,
                       seed=1, prompt_len=512, k=16, max_new_tokens=1024),
    "8b": ModelShape("8b", 36, 4096, 32, 8, 128, 12288, 151936, False, 1.0e6,
                     seed=2, prompt_len=1024, k=16, max_new_tokens=1024),
}


def gen_model_weights(shape: ModelShape, device="cpu", layers=None, with_head: bool = True) -> dict:
    """bf16 weights for ``shape``; matrices are [out_features, in_features].

    Norm gains are 1 + N(0, 0.1^2), rounded to bf16, so that a kernel that
    drops or misplaces a gain cannot pass.
    ``layers`` restricts generation to a subset of layer indices (the rest are
    left out of the returned list), for bounded CPU samples of a big model;
    ``with_head=False`` leaves out the embedding, the LM head and the final norm
    (for callers that fetch a big model one layer at a time).
    """
    s, d, hd = shape.seed, shape.d_model, shape.head_dim
    std = shape.init_std

    def mat(kind, layer, rows, cols):
        return gen_normal_bf16(s, tensor_id(kind, layer), rows * cols, std, device).view(rows, cols)

    def gain(kind, layer):
        g = gen_normal_bf16(s, tensor_id(kind, layer), d, 0.1, device).to(torch.float32)
        return (1.0 + g).to(torch.bfloat16)

    w = {}
    if with_head:
        w = {"embed": mat("embed", 0, shape.vocab, d),
             "final_norm": gain("final_norm", 0)}
        w["lm_head"] = w["embed"] if shape.tie_lm_head else mat("lm_head", 0, shape.vocab, d)
    w["layers"] = []
    def vec(kind, layer, n, scale, offset):
        g = gen_normal_bf16(s, tensor_id(kind, layer), n, scale, device).to(torch.float32)
        return (offset + g).to(torch.bfloat16)

    for l in (range(shape.n_layers) if layers is None else layers):
        extra = {}
        if shape.qkv_bias:
            extra.update(bq=vec("bq", l, shape.n_q_heads * hd, 0.1, 0.0), bk=vec("bk", l, shape.n_kv_heads * hd, 0.1, 0.0),
                         bv=vec("bv", l, shape.n_kv_heads * hd, 0.1, 0.0))
        if shape.qk_norm:
            extra.update(q_norm=vec("q_norm", l, hd, 0.1, 1.0), k_norm=vec("k_norm", l, hd, 0.1, 1.0))
        w["layers"].append({
            **extra,
            "index": l,
            "attn_norm": gain("attn_norm", l),
            "wq": mat("wq", l, shape.n_q_heads * hd, d),
            "wk": mat("wk", l, shape.n_kv_heads * hd, d),
            "wv": mat("wv", l, shape.n_kv_heads * hd, d),
            "wo": mat("wo", l, d, shape.n_q_heads * hd),
            "ffn_norm": gain("ffn_norm", l),
            "w_gate": mat("w_gate", l, shape.d_ffn, d),
            "w_up": mat("w_up", l, shape.d_ffn, d),
            "w_down": mat("w_down", l, d, shape.d_ffn),
        })
    return w

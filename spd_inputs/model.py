"""Shapes and random-init bf16 weights of a Llama-style decoder.

The paper runs Llama-2-7B unchanged (Section 4); trained weights are not
available here, so the tensors are N(0, 0.02) draws rounded to bf16 and the
RMSNorm gains are 1 + N(0, 0.1) (so that a dropped gain is visible).
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, List

import torch

from .rng import hash_u64, uniform01


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    d_ffn: int
    vocab: int

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_heads

    @property
    def n_params(self) -> int:
        d, f = self.d_model, self.d_ffn
        return self.n_layers * (4 * d * d + 3 * d * f) + self.vocab * d

    @property
    def step_weight_bytes(self) -> int:
        """bf16 bytes of every matrix one decode step multiplies by (embedding table excluded)."""
        return 2 * self.n_params


SHAPES: Dict[str, ModelShape] = {
    "tiny": ModelShape("tiny", 2, 256, 4, 688, 4096),
    "7b": ModelShape("7b", 32, 4096, 32, 11008, 32000),
    "13b": ModelShape("13b", 40, 5120, 40, 13824, 32000),
}

_CHUNK = 1 << 22


def normal_bf16(seed: int, tensor_id: int, numel: int, std: float, mean: float = 0.0,
                device: str | torch.device = "cpu") -> torch.Tensor:
    """bf16 (round-to-nearest-even) of mean + std * N(0,1) by Box-Muller in float64."""
    out = torch.empty(numel, dtype=torch.bfloat16, device=device)
    for lo in range(0, numel, _CHUNK):
        hi = min(numel, lo + _CHUNK)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        u1 = uniform01(hash_u64(seed, tensor_id, 2 * idx))
        u2 = uniform01(hash_u64(seed, tensor_id, 2 * idx + 1))
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        out[lo:hi] = (mean + std * z).to(torch.float32).to(torch.bfloat16)
    return out


def make_weights(shape: ModelShape, seed: int = 0, device: str | torch.device = "cpu",
                 std: float = 0.02) -> Dict[str, object]:
    """All tensors of the decoder, bf16, row-major [out][in].

    Keys: tok_emb [V,d], lm_head [V,d], final_norm [d]; per-layer lists attn_norm [d],
    wq/wk/wv/wo [d,d], ffn_norm [d], wgate/wup [f,d], wdown [d,f].
    """
    d, f, v = shape.d_model, shape.d_ffn, shape.vocab
    tid = [0]

    def mat(r: int, c: int) -> torch.Tensor:
        tid[0] += 1
        return normal_bf16(seed, tid[0], r * c, std, 0.0, device).view(r, c)

    def gain() -> torch.Tensor:
        tid[0] += 1
        return normal_bf16(seed, tid[0], d, 0.1, 1.0, device)

    w: Dict[str, object] = {"tok_emb": mat(v, d), "lm_head": mat(v, d), "final_norm": gain()}
    names: List[str] = ["attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "wgate", "wup", "wdown"]
    for n in names:
        w[n] = []
    for _ in range(shape.n_layers):
        w["attn_norm"].append(gain())
        w["wq"].append(mat(d, d))
        w["wk"].append(mat(d, d))
        w["wv"].append(mat(d, d))
        w["wo"].append(mat(d, d))
        w["ffn_norm"].append(gain())
        w["wgate"].append(mat(f, d))
        w["wup"].append(mat(f, d))
        w["wdown"].append(mat(d, f))
    return w

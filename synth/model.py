"""Model shapes of the measured workloads and their seeded random-init weights.

Tensor layouts are the ones the CUDA library's ``bita_weights`` documents
(every matrix is ``[out_features, in_features]`` with the input dimension
contiguous, as in a Linear layer).  Values are N(0, 0.02)-like pseudo-normals
(the init the paper states for its learnable embeddings, Sec. 4.1
"Implementation Details"), norm gains are 1 + 0.02 z so a missing gain shows up,
and the per-layer prompt prefix keys/values are drawn at the scale projected
keys/values have (0.02 * sqrt(d)) so that an indexing mistake in the prefix path
moves the outputs by more than the parity tolerance.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch

from .rng import pseudo_normal


@dataclass(frozen=True)
class ModelShape:
    name: str
    L: int
    d: int
    H: int
    H_kv: int
    D: int
    F: int
    V: int
    P: int = 16          # prompt (prefix) tokens per layer
    n_mask: int = 4      # mask tokens per group
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    prompt_len: int = 512
    steps: int = 256
    tree_K: tuple = (10, 6, 4, 2)
    tree_B: tuple = (10, 6, 6, 4)

    def with_layers(self, L: int) -> "ModelShape":
        return replace(self, L=L, name=f"{self.name}-L{L}")

    @property
    def layer_params(self) -> int:
        return (self.H + 2 * self.H_kv) * self.D * self.d + self.d * self.H * self.D + 3 * self.d * self.F

    @property
    def streamed_params(self) -> int:
        """Parameters every step must read once: all layer matrices + LM head."""
        return self.L * self.layer_params + self.V * self.d

    def kv_bytes_per_token(self) -> int:
        return self.L * 2 * self.H_kv * self.D * 2


CONFIGS = {
    "tiny": ModelShape("tiny", L=2, d=256, H=4, H_kv=4, D=64, F=688, V=1024, P=16, n_mask=3,
                       prompt_len=64, steps=32, tree_K=(3, 3, 3), tree_B=(3, 3, 3)),
    "7b": ModelShape("7b", L=32, d=4096, H=32, H_kv=32, D=128, F=11008, V=32000, prompt_len=512, steps=256),
    "13b": ModelShape("13b", L=40, d=5120, H=40, H_kv=40, D=128, F=13824, V=32000, prompt_len=1024, steps=256),
    "70b": ModelShape("70b", L=80, d=8192, H=64, H_kv=8, D=128, F=28672, V=32000, prompt_len=1024, steps=128),
}

_GLOBAL = {"tok_emb": 1, "mask_emb": 2, "g_final": 3, "lm_head": 4}
_LAYER = {"wqkv": 0, "wo": 1, "wg": 2, "wu": 3, "wd": 4, "g_attn": 5, "g_ffn": 6, "prompt_k": 7, "prompt_v": 8}


def global_weight_specs(s: ModelShape):
    return {
        "tok_emb": (s.V, s.d),
        "mask_emb": (s.n_mask, s.d),
        "g_final": (s.d,),
        "lm_head": (s.V, s.d),
    }


def layer_weight_specs(s: ModelShape):
    return {
        "wqkv": ((s.H + 2 * s.H_kv) * s.D, s.d),
        "wo": (s.d, s.H * s.D),
        "wg": (s.F, s.d),
        "wu": (s.F, s.d),
        "wd": (s.d, s.F),
        "g_attn": (s.d,),
        "g_ffn": (s.d,),
        "prompt_k": (s.H_kv, s.P, s.D),
        "prompt_v": (s.H_kv, s.P, s.D),
    }


def _gen(seed, stream, name, shape, s: ModelShape, dtype, device):
    if name.startswith("g_"):
        # gains are tiny: always drawn on the CPU (mean added in fp32 there) then moved
        return pseudo_normal(seed, stream, shape, 0.02, mean=1.0, dtype=dtype, device="cpu").to(device)
    if name.startswith("prompt_"):
        return pseudo_normal(seed, stream, shape, 0.02 * math.sqrt(s.d), dtype=dtype, device=device)
    return pseudo_normal(seed, stream, shape, 0.02, dtype=dtype, device=device)


def make_global_weights(s: ModelShape, seed: int, *, dtype=torch.bfloat16, device="cpu"):
    return {k: _gen(seed, _GLOBAL[k], k, shp, s, dtype, device) for k, shp in global_weight_specs(s).items()}


def make_layer_weights(s: ModelShape, seed: int, layer: int, *, dtype=torch.bfloat16, device="cpu"):
    return {k: _gen(seed, 100 + 16 * layer + _LAYER[k], k, shp, s, dtype, device)
            for k, shp in layer_weight_specs(s).items()}


def make_weights(s: ModelShape, seed: int, *, dtype=torch.bfloat16, device="cpu"):
    """All weights: ``{"tok_emb":…, "layers": [ {...}, … ], …}``."""
    w = make_global_weights(s, seed, dtype=dtype, device=device)
    w["layers"] = [make_layer_weights(s, seed, l, dtype=dtype, device=device) for l in range(s.L)]
    return w

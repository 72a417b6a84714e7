"""Glue used by the tests: turns seeded synthetic tensors into oracle inputs."""
from __future__ import annotations

import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402
from oracle import bita_oracle as orc  # noqa: E402


def _np(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy()


def to_numpy_weights(w):
    out = {k: _np(v) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: _np(v) for k, v in lw.items()} for lw in w["layers"]]
    return out


class LazyLayers:
    """Regenerates a layer's weights on access, so that a 13 GB model never sits in host memory at once."""

    def __init__(self, shape, seed, dtype=torch.bfloat16):
        self.shape, self.seed, self.dtype = shape, seed, dtype
        self._cache = (None, None)

    def __getitem__(self, l):
        if self._cache[0] != l:
            lw = synth.model.make_layer_weights(self.shape, self.seed, l, dtype=self.dtype)
            self._cache = (l, {k: _np(v) for k, v in lw.items()})
        return self._cache[1]


def oracle_model(shape: synth.ModelShape, seed: int, *, dtype=torch.bfloat16, lazy=False, weights=None):
    """Oracle model whose weights are the given torch weights (or seeded ones) converted value-for-value."""
    if weights is not None:
        w = to_numpy_weights(weights)
    elif lazy:
        g = synth.model.make_global_weights(shape, seed, dtype=dtype)
        w = {k: _np(v) for k, v in g.items()}
        w["layers"] = LazyLayers(shape, seed, dtype)
    else:
        w = to_numpy_weights(synth.make_weights(shape, seed, dtype=dtype))
    return orc.Model(L=shape.L, d=shape.d, H=shape.H, H_kv=shape.H_kv, D=shape.D, F=shape.F, V=shape.V,
                     P=shape.P, n_mask=shape.n_mask, rms_eps=shape.rms_eps, rope_theta=shape.rope_theta,
                     weights=w)


def block_for(tmpl: synth.Template, n_mask: int) -> orc.Block:
    return orc.Block(tmpl.parent, tmpl.rank, tmpl.attach, n_mask)


def prompt_tokens(seed: int, length: int, vocab: int):
    return synth.uniform_ints(seed, 5001, length, vocab).tolist()


MICRO = synth.ModelShape("micro", L=2, d=32, H=4, H_kv=2, D=8, F=48, V=40, P=3, n_mask=3,
                         prompt_len=6, steps=8, tree_K=(3, 3, 3), tree_B=(3, 3, 3))

"""Glue between the seeded input generators (``synth``) and the CPU oracle.

TEST INFRASTRUCTURE ONLY, like the rest of this directory: turns synthetic weight tensors into the
oracle's model container and tree templates into its block layout.  Holds no arithmetic of the
method and is never imported by the CUDA package.
"""
from __future__ import annotations

import numpy as np
import torch

import synth

from . import bita_oracle as orc


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


class LayersFromDevice:
    """Per-layer fp64 host copies of device-resident weights, converted on access (one layer held at
    a time), so that the oracle of a full-depth model sees the very tensors the library was given
    without tens of gigabytes of fp64 sitting in host memory."""

    def __init__(self, layers):
        self._layers = layers
        self._cache = (None, None)
        self.observer = None       # callable(l, layer_weights), told about every layer as it is converted

    def __len__(self):
        return len(self._layers)

    def __getitem__(self, l):
        if self._cache[0] != l:
            self._cache = (l, {k: v.detach().cpu().to(torch.float64).numpy() for k, v in self._layers[l].items()})
            if self.observer is not None:
                self.observer(l, self._cache[1])
        return self._cache[1]


def _model(shape: synth.ModelShape, w) -> orc.Model:
    return orc.Model(L=shape.L, d=shape.d, H=shape.H, H_kv=shape.H_kv, D=shape.D, F=shape.F, V=shape.V,
                     P=shape.P, n_mask=shape.n_mask, rms_eps=shape.rms_eps, rope_theta=shape.rope_theta,
                     weights=w)


def oracle_model(shape: synth.ModelShape, seed: int, *, dtype=torch.bfloat16, lazy=False, weights=None) -> orc.Model:
    """Oracle model whose weights are the given torch weights (or seeded ones) converted value-for-value."""
    if weights is not None:
        w = to_numpy_weights(weights)
    elif lazy:
        g = synth.model.make_global_weights(shape, seed, dtype=dtype)
        w = {k: _np(v) for k, v in g.items()}
        w["layers"] = LazyLayers(shape, seed, dtype)
    else:
        w = to_numpy_weights(synth.make_weights(shape, seed, dtype=dtype))
    return _model(shape, w)


def oracle_model_from_device(shape: synth.ModelShape, weights) -> orc.Model:
    """Oracle model over the given (device) weights, value for value; layers converted lazily."""
    w = {k: _np(v) for k, v in weights.items() if k != "layers"}
    w["layers"] = LayersFromDevice(weights["layers"])
    return _model(shape, w)


def block_for(tmpl: synth.Template, n_mask: int) -> orc.Block:
    return orc.Block(tmpl.parent, tmpl.rank, tmpl.attach, n_mask)

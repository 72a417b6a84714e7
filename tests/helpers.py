"""Names the tests share: the seeded generators, the oracle and the glue between them."""
from __future__ import annotations

import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402
from oracle import bita_oracle as orc  # noqa: E402
from oracle.inputs import (  # noqa: E402,F401
    LayersFromDevice, LazyLayers, block_for, oracle_model, oracle_model_from_device, to_numpy_weights)


def prompt_tokens(seed: int, length: int, vocab: int):
    return synth.uniform_ints(seed, 5001, length, vocab).tolist()


MICRO = synth.ModelShape("micro", L=2, d=32, H=4, H_kv=2, D=8, F=48, V=40, P=3, n_mask=3,
                         prompt_len=6, steps=8, tree_K=(3, 3, 3), tree_B=(3, 3, 3))

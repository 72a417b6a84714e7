"""Seeded synthetic inputs (weights, prompts, tree templates, planted drafts).

This package only *produces inputs*. It holds none of the decoding method's
arithmetic: no attention rule, no verification walk, no model forward.  Both the
CUDA library's callers and the CPU oracle's callers draw their inputs from here,
so that the two sides see bit-identical tensors without sharing any code of the
method itself.
"""
from .rng import pseudo_normal, uniform_ints, uniform_unit  # noqa: F401
from .model import CONFIGS, ModelShape, make_weights, layer_weight_specs  # noqa: F401
from .trees import (  # noqa: F401
    product_rule_template,
    comb_template,
    full_tree_template,
    chain_template,
    random_recursive_template,
    empty_template,
    Template,
)
from .planting import plant_tree  # noqa: F401
from .acceptance import AcceptanceModel, tokens_per_pass  # noqa: F401

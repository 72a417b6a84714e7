"""B200-native BiTA tree-decoding step (arXiv 2401.12522): Python binding of the C-ABI library.

The package only marshals arguments: every step of a decoding pass runs in the CUDA kernels of
``libbita.so``.  PyTorch supplies device memory and the stream.  There is no CPU fallback: without
the built library the import fails.
"""
from .binding import (  # noqa: F401
    Bita,
    BitaError,
    StepOut,
    lib,
    bita_gemm_bf16,
    bita_tree_attention,
    bita_tree_attention_static,
    MAX_ROWS,
    MAX_NODES,
    MAX_TOPK,
    MAX_DEPTH,
)

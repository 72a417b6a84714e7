"""B200-native BiTA tree-decoding step (arXiv 2401.12522): Python binding of the C-ABI library.

The package only marshals arguments: every step of a decoding pass runs in the CUDA kernels of
``libbita.so``.  PyTorch supplies device memory and the stream.  There is no CPU fallback: the first
use of any name below loads the library and raises ImportError if it has not been built
(``python -m paper_2401_12522_b200.build``).  The ``build`` submodule itself imports without it.
"""
_NAMES = ("Bita", "BitaError", "StepOut", "lib", "bita_gemm_bf16", "bita_tree_attention",
          "bita_tree_attention_static", "set_attention_route", "MAX_ROWS", "MAX_NODES", "MAX_TOPK", "MAX_DEPTH")
__all__ = list(_NAMES)


def __getattr__(name):
    if name in _NAMES:
        from . import binding          # loads libbita.so; ImportError when it is missing
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")

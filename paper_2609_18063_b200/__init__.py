"""B200-native streaming-MoE per-layer decode step: thin ctypes binding over the CUDA library.

The C-ABI functions live in ``binding`` and are re-exported here on first use, which loads
``libedgmoe.so`` (built in-tree by ``python -m paper_2609_18063_b200.build``).  There is no CPU
or PyTorch fallback: a missing or stale library raises on that first use.  ``build`` itself can
be imported without the library.
"""
import importlib

_LAZY = ("binding", "layer_io")


def __getattr__(name):
    if name in ("build",) + _LAZY:
        return importlib.import_module(f"{__name__}.{name}")
    binding = importlib.import_module(f"{__name__}.binding")
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None


def __dir__():
    binding = importlib.import_module(f"{__name__}.binding")
    return sorted(set(globals()) | set(binding.__all__))

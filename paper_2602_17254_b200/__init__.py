"""B200-native engine for the Trivance AllReduce hot path (n simulated ranks in one GPU's HBM).

The CUDA library is loaded on first use of anything in :mod:`.binding`; importing
the package (for example for :mod:`.synth`) needs no GPU and no built library.
"""

__all__ = ["binding", "synth"]


def __getattr__(name):
    if name in ("binding", "synth"):
        import importlib
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)

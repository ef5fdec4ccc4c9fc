"""B200-native CIAR hot path: per-token interval quantification and speculative verification
over visual-vocabulary logits, as hand-written sm_100a CUDA behind a C ABI.

``ciar`` (the ctypes binding of ``libciar.so``) is imported on first attribute access so that
the input generators in ``synth`` stay importable on a machine without the built library.
"""
__all__ = ["synth", "ciar"]


def __getattr__(name):
    if name in ("ciar", "synth"):
        import importlib
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)

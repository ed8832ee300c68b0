"""B200-native budgeted MoE verify layer (MoE-Spec, Algorithm 1) behind a C ABI.

`synth` makes seeded inputs and is importable anywhere.  `moespec` is the thin
ctypes binding over the CUDA library; it is imported lazily so that tools that
only need shapes or inputs work on a machine without the built library, while
any attempt to run the layer without it raises.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "moespec"]


def __getattr__(name):
    if name == "moespec":
        import importlib
        return importlib.import_module(__name__ + ".moespec")
    raise AttributeError(name)

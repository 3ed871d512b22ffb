"""B200-native CUDA implementation of MixDQ's quantized linear / conv inference path.

The package is a thin ctypes binding (``mixdq``) over the C-ABI library built from
``csrc/``, plus seeded synthetic input generators (``synth``).  The CUDA library is
loaded on first use; there is no CPU fallback.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "mixdq"]


def __getattr__(name):
    if name == "mixdq":
        import importlib
        return importlib.import_module(".mixdq", __name__)
    raise AttributeError(name)

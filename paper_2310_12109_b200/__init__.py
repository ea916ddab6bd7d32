"""B200-native Monarch Mixer hot path: Monarch matmul and Monarch (FFT) convolution.

The compute lives in ``csrc/`` behind a C ABI (``include/m2.h``); ``binding`` is the
thin ctypes layer over it and ``synth`` the seeded input generator.  Importing the
package does not load the shared library; the first call into ``binding`` does and
raises if it has not been built.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(__name__ + ".binding")
    raise AttributeError(name)

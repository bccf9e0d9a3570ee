"""B200-native gated N-D long convolution (the FFT hot path of HyenaND).

``hyenand`` is the thin binding over the C-ABI CUDA library; ``workloads``
holds the seeded synthetic input generators.  Importing the package does not
load the CUDA library; the first call that needs it does, and fails loudly if
it has not been built.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "hyenand"]


def __getattr__(name):
    if name == "hyenand":
        import importlib
        return importlib.import_module(".hyenand", __name__)
    raise AttributeError(name)

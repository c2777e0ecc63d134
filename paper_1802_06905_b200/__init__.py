"""Communication-optimal direct convolution (seven-nested-loop CNN, Eq. 1) for B200 / sm_100a.

The package is a thin binding over the C-ABI library ``libcconv.so`` built from ``csrc/``.
Importing the package does not load the library; the first call does, and fails loudly when the
library or a CUDA device is missing.  There is no CPU fallback.
"""
from .synth import CONFIGS, ConvShape, make_inputs  # noqa: F401


def __getattr__(name):
    # Lazy so that the seeded input generators can be imported without the native library.
    if name in ("conv_forward", "lower_bound", "tiling_lp", "Plan", "library_path",
                "load_library", "CconvError"):
        import importlib
        return getattr(importlib.import_module(__name__ + ".binding"), name)
    raise AttributeError(name)

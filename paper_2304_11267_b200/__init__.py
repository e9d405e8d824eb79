"""B200-native scaled-dot-product attention for the Stable Diffusion 1.4 UNet.

The product is the C-ABI library built from ``csrc/`` (hand-written sm_100a CUDA kernels);
``binding`` marshals arguments into it and ``workloads`` draws seeded synthetic inputs.
There is no CPU fallback: every call fails loudly when the CUDA library is missing.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(__name__ + ".binding")
    raise AttributeError(name)

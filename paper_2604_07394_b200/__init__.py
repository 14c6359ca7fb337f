"""B200-native routed hybrid attention (Flux Attention hot path).

``flux`` is the Python binding of the C-ABI library ``libflux_attn.so``
(hand-written sm_100a kernels); ``synth`` draws the seeded synthetic workloads.
Importing the package does not load the CUDA library; ``flux.load()`` does, and
fails loudly when the library has not been built.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "flux"]


def __getattr__(name):
    if name == "flux":
        import importlib

        return importlib.import_module(".flux", __name__)
    raise AttributeError(name)

"""LoSA per-denoising-step attention hot path for block-wise diffusion LMs, B200-native (sm_100a).

`binding` exposes the C-ABI library (`include/losa.h`) one-to-one; `workloads` holds the seeded
synthetic input generators.  The CUDA library is loaded on first use and its absence is an error:
there is no CPU fallback.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(__name__ + ".binding")
    raise AttributeError(name)

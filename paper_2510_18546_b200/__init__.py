"""Selective-KV attention over per-group cached K/V with fused per-group attention mass
(B200 / sm_100a).  ``enl`` is the thin binding over the C-ABI library; ``synth`` holds the
seeded synthetic workloads.  Submodules are imported on first use so that importing the
workload generator alone does not load the CUDA library."""
import importlib

__all__ = ["enl", "synth", "dist"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)

"""B200 (sm_100a) operator kernels of a transformer encoder layer behind a C ABI.

``paper_2511_03586_b200.inputs`` holds the seeded synthetic input generators and
imports without the CUDA library; everything else lives in
``paper_2511_03586_b200.api`` (loaded on first attribute access), which needs
``libpd.so`` built by ``paper_2511_03586_b200.build``.
"""
import importlib

__all__ = ["api", "inputs", "build", "replicas"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)

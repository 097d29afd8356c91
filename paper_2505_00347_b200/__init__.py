"""B200-native fused low-bit (SOLO) optimizer step: C-ABI CUDA library + thin binding.

``binding`` wraps the C ABI of ``include/solo.h`` (the CUDA library must have been built:
``python -m paper_2505_00347_b200._build``); ``synth`` generates the seeded synthetic
workloads.  Nothing here computes any part of the optimizer step in Python.
"""
from . import synth  # noqa: F401


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)

"""B200-native A2SF hot path: causal prefill scoring + fused decode step.

The work is done by hand-written sm_100a CUDA kernels behind the C-ABI library
``liba2sf.so`` (``include/a2sf.h``).  ``paper_2407_20485_b200.binding`` is the thin
ctypes layer over it; ``paper_2407_20485_b200.workloads`` holds the synthetic
workloads.  There is no CPU fallback: importing the binding without the built
library raises.
"""

__all__ = ["binding", "workloads", "build"]


def __getattr__(name):
    if name in __all__:
        import importlib

        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)

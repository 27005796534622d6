"""B200-native hot path of DPPO's pruned GRPO training step.

The work is done by hand-written sm_100a CUDA kernels behind a C ABI
(``include/dppo.h``, built into ``libdppo.so``); :mod:`.binding` marshals
arguments to it and nothing else.  There is no CPU fallback: using the binding
without the built library raises.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)

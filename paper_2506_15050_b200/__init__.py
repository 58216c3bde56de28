"""B200-native T-PPO token-selective update path (EGAE scan, token compaction, fused
log-softmax + clipped-surrogate loss with gradient, value loss).

The arithmetic runs in hand-written sm_100a CUDA kernels behind a C ABI (include/tppo.h);
``binding`` marshals torch device tensors into that ABI and ``synth`` draws the synthetic
workloads.  There is no CPU fallback: every call raises if the CUDA library is missing.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)

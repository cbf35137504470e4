"""tik: bitwise-consistent causal GQA attention and token log-probability kernels for B200.

The compute path is the C-ABI library built from ``csrc/`` (hand-written
sm_100a CUDA); ``binding`` marshals torch tensors into it and ``synth`` draws
the seeded benchmark inputs.  There is no CPU or library fallback: calling an
operator without the built library raises.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)

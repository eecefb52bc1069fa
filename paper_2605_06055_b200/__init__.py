"""libmoecomm: relay-buffer-free MoE dispatch / combine for NVIDIA B200 (sm_100a).

The compute path lives in ``csrc/`` (CUDA, C ABI declared in ``include/moecomm.h``).
``binding`` marshals arguments to it and nothing else; ``synth`` draws seeded
synthetic inputs.  There is no CPU fallback: using the binding without the
built CUDA library raises.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]

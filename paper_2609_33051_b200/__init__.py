"""SketchSSM decode hot path for NVIDIA B200: CUDA library behind a C ABI plus a thin binding.

`synth` holds the seeded synthetic workloads; `binding` loads libsketchssm.so (built by `build`).
Nothing here computes on the CPU: without the CUDA library the calls fail.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build", "calibrate"]

"""B200 (sm_100a) speech augmentation and feature extraction.

`binding` wraps the C-ABI library (built by `build`), `synth` draws seeded
synthetic workloads.  Nothing here computes on the CPU: without the CUDA
library the compute calls raise."""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]

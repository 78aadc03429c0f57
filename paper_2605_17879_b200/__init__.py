"""B200-native robust straggler scoring (Guard, Sections 4.2 and 5.2-5.4 of the paper).

`guard` is the ctypes binding of the CUDA library, `synth` the seeded synthetic
telemetry generators, `build` compiles the library in-tree with nvcc.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "guard", "build"]

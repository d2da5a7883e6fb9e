"""B200-native 3D Deformable Slide Attention (forward and backward) as a C-ABI CUDA library.

``binding`` wraps the shared library's entry points (same names as the C header);
``inputs`` holds the seeded synthetic workloads; ``build`` compiles the library for
sm_100a.  Nothing is loaded at import time: the first call into ``binding`` loads the
library and raises if it has not been built.
"""
__all__ = ["binding", "inputs", "build"]

"""B200-native Draft-Then-Verify decoding loop of LASER (arXiv 2408.05676).

The package holds the CUDA kernels plus their C-ABI library (``csrc/``), a thin
ctypes binding with the same entry-point names (``binding``), the build step
(``build``) and the seeded synthetic input generators (``synth``).  Nothing is
imported eagerly: ``synth`` carries none of the method's arithmetic and must be
usable without the CUDA library, while ``binding`` raises as soon as the
library is missing.
"""

__all__ = ["binding", "build", "synth"]
__version__ = "0.1.0"

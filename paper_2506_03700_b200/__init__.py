"""B200-native layer-parallel decode step of AdaDecode (Algorithm 1).

Importing the package loads nothing heavy.  `binding` holds the ctypes view of
the C-ABI library (it fails loudly when the CUDA library is missing); `synth`
holds the seeded input generators, which contain none of the method's
arithmetic and are the only module shared with the test oracle's harness.
"""

__all__ = ["binding", "synth"]

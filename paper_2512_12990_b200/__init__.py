"""B200-native SliceMoE hot path: the MoE expert FFN computed from bit-sliced AMAT weights.

`paper_2512_12990_b200.binding` is the thin ctypes binding over the C-ABI shared library
(`libslicemoe.so`, built from `csrc/`); `paper_2512_12990_b200.synth` draws the seeded
synthetic inputs.  Importing the package does not load the library; the first call into
`binding` does, and raises if the library has not been built.
"""
__all__ = ["binding", "synth", "build"]

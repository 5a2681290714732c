"""FF-INT8 per-layer Forward-Forward INT8 train step for NVIDIA B200 (sm_100a).

`paper_2506_22771_b200.binding` is the thin ctypes layer over the C-ABI library
(`libffint8.so`, built from `csrc/` by `paper_2506_22771_b200.build`); `synth` draws the
seeded synthetic inputs.  Importing this package loads nothing heavy.
"""
__all__ = ["binding", "build", "synth"]

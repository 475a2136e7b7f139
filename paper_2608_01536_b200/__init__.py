"""B200-native batch-1 dual-sparse decode product y = W.x on RLC-CSC weights (Celty).

`paper_2608_01536_b200.celty` is the thin binding over the C-ABI CUDA library
(`csrc/`, built in-tree by `paper_2608_01536_b200.build`); `synth` makes seeded synthetic
inputs.  Importing this package loads no native code; the binding loads the library on
first use and raises if it is missing.
"""
__all__ = ["celty", "synth", "build"]

"""B200-native complete-expert sparse-MoE layer forward (ExactMoE hot path).

`paper_2608_15383_b200.binding` is the thin ctypes layer over the C-ABI library
built from `csrc/` (declared in `include/exmoe.h`); `synth` draws the seeded
synthetic inputs.  Importing the package loads nothing: the library is opened on
first use and its absence is an error, there is no CPU fallback.
"""
__all__ = ["binding", "synth", "build"]

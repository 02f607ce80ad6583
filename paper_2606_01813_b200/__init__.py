"""B200-native CaDDTree hot path: batched cost-aware draft-tree construction and tree verification.

`binding` wraps the C-ABI library (libcadd.so, built from csrc/); `synth` draws seeded inputs.
Nothing is imported eagerly so that the input generators can be used without the CUDA library.
"""
__all__ = ["binding", "synth", "build"]

"""B200-native DDG (decoupled parallel backpropagation with delayed gradients) training step.

`nets` and `synth` are plain-Python helpers (network specifications and seeded synthetic inputs) that hold
none of the method's arithmetic.  `binding` is the thin ctypes layer over the C-ABI CUDA library; importing it
loads the library and fails loudly when the library has not been built.
"""
__all__ = ["nets", "synth", "binding"]

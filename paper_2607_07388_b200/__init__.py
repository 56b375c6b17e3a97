"""B200-native Engram lookup-and-inject (TF-Engram inference hot path).

``binding`` wraps the C-ABI CUDA library (``csrc/``); ``synth`` makes the
seeded synthetic inputs.  Importing the package loads neither: the binding
loads the shared library on first use and raises if it is missing.
"""
__all__ = ["binding", "synth", "build"]

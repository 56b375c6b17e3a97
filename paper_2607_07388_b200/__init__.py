"""B200-native Engram lookup-and-inject (TF-Engram inference hot path).

``binding`` wraps the C-ABI CUDA library (``csrc/``) one to one; ``engine`` holds
the convenience classes ``Engram`` (phrase index + GPU tier: lookup-and-inject,
miss list, prefetch candidates, retention ranking, install) and
``EarlyExitHead`` (softmax(W_pref h) + top-K on the tensor cores); ``synth``
makes the seeded synthetic inputs; ``build`` compiles the library in-tree.
Importing the package loads none of them: the binding loads the shared
library on first use and raises if it is missing.
"""
__all__ = ["binding", "engine", "synth", "build"]

"""B200-native sink+window attention over a rolling per-layer KV cache.

``binding`` exposes the C ABI of ``libllattn.so`` (hand-written sm_100a CUDA);
``synth`` holds the seeded synthetic inputs; ``build`` compiles the library.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]

"""B200-native FastMMoE MoE-layer hot path: Python binding over the C-ABI library.

`inputs` (seeded synthetic workloads) imports nothing from the binding, so it can
be used without the compiled library; `binding` loads the library lazily and
raises if it is missing (there is no CPU fallback).
"""
__all__ = ["inputs", "binding"]

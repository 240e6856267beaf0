"""B200-native bounded-state restoration: probe -> bounded window -> install -> commit.

`synth` (seeded inputs) imports without a GPU.  Everything else goes through `binding`, which
loads the CUDA library and raises if it is missing: there is no CPU fallback.
"""
__all__ = ["synth", "binding", "build"]

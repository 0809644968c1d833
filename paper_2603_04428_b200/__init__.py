"""B200-native batched attention over 4-bit group-quantized KV caches (C-ABI library + thin binding).

`synth` (seeded input generators) imports without the CUDA library; everything
else lives in `binding`, which loads libq4kv.so and raises if it is missing.
"""
__all__ = ["synth", "binding"]

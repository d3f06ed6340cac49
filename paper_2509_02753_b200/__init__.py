"""B200-native per-layer top-k Mixture-of-Experts forward pass (LExI's hot path).

``synth`` draws the seeded synthetic workloads; ``binding`` is the thin ctypes
layer over the C-ABI CUDA library (loaded on first use, never at import).
"""
__all__ = ["synth", "binding"]

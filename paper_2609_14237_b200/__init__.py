"""B200-native decode attention stage for operator-disaggregated serving.

``synth`` holds the seeded input generators; ``binding`` is the ctypes layer over the
C-ABI library built from ``csrc/`` (argument marshalling only -- every step of the hot
path runs in the CUDA kernels).
"""
__all__ = ["synth", "binding"]

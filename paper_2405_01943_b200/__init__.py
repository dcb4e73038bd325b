"""B200-native (sm_100a) hot path of DaSS: fused GLU calibration norms, N:M scoring and compression.

The compute lives in ``csrc/`` behind a C-ABI shared library (``include/dass.h``);
``binding`` is the thin ctypes layer over it, ``layer`` chains its calls for one MLP layer and ``synth`` holds
the seeded input generators.
"""
__all__ = ["binding", "layer", "synth"]

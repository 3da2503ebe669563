"""B200-native PRQuant hot path: the compensated W4A4 MXFP4 linear layer.

``synth`` draws the seeded inputs; ``binding`` is the thin ctypes layer over the
C-ABI CUDA library (``libprq.so``, built in-tree by ``build``).
"""

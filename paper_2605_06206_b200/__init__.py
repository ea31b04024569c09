"""B200-native forward pass of a Federation-of-Experts transformer block.

`synth` holds the seeded synthetic inputs; `binding` is the thin ctypes layer over the
C-ABI library (include/foe.h) built from csrc/ by `build`.
"""
__all__ = ["synth"]

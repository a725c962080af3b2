"""B200-native hot path of Pacer (blockwise pre-verification for speculative
decoding with adaptive draft length).

Sub-modules:
  synth    seeded synthetic inputs (weights, successor tables, prompts, shapes).
           Holds no arithmetic of the method; importing it loads no native code.
  binding  thin ctypes binding of the C-ABI library ``libpacer.so``; importing
           it fails loudly when the CUDA library has not been built.

Nothing is imported eagerly, so the input generators can be used on a machine
that has no GPU and no built library.
"""

__all__ = ["synth", "binding"]

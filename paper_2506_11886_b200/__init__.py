"""B200-native hybrid-KV (FourierAttention) decode path.

``paper_2506_11886_b200.fa`` is the thin ctypes binding of the C-ABI library
(``include/fa.h``); ``paper_2506_11886_b200.synth`` draws the seeded synthetic
inputs.  Importing the package does not load the CUDA library; the first call
into ``fa`` does, and fails loudly if it has not been built.
"""
__all__ = ["synth"]

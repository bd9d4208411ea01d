"""Block Selective Reprogramming (BSR) fine-tuning step for Vision Transformers on B200.

The package holds the CUDA kernels and their C-ABI library (``csrc/``), a thin
ctypes binding with the same entry-point names (``binding``), and the seeded
synthetic input generators (``synth``).  Importing the package does not load the
native library; the first call into ``binding`` does, and raises if it is missing.
"""

__all__ = ["binding", "synth"]

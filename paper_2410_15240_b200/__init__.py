"""B200-native GPU side of Fastrack's CPU<->GPU secure channel (arXiv 2410.15240).

``paper_2410_15240_b200.fastrack`` is the ctypes binding of the C-ABI CUDA library (it raises at
import time if the library has not been built); ``paper_2410_15240_b200.synth`` holds the seeded
synthetic input generators.  Nothing here falls back to a CPU implementation.
"""
__all__ = ["fastrack", "synth"]

"""B200-native residual-expanded quantized layer (PIPE, arXiv 2311.15806).

The product is the CUDA library ``libpipe.so`` (C ABI declared in ``include/pipe.h``) and the
thin ctypes binding in :mod:`paper_2311_15806_b200.binding`.  Nothing here computes on the CPU.
"""
__all__ = ["binding", "synth", "build"]

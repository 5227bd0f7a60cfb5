"""B200 (sm_100a) hot path of multi-LoRA / multi-stream / DS2D decoding behind a C ABI.

The Python layer only marshals arguments into ``libmlora.so``; every step of the path runs in the
CUDA kernels of that library.  Importing this package never builds or loads anything; the first use of
``binding`` loads the library and raises if it is missing.
"""
__all__ = ["binding", "build"]

"""LayerPipe training hot path for NVIDIA B200 (sm_100a).

``inputs`` holds the workload shapes and seeded generators; ``binding`` is the
thin ctypes layer over the C-ABI library ``liblayerpipe.so`` (see
``include/layerpipe.h``).  Importing this package does not load the library;
``binding`` does, and fails loudly when it is missing.
"""
__all__ = ["inputs", "binding", "build"]

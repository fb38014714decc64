"""LayerPipe training hot path for NVIDIA B200 (sm_100a).

``inputs`` holds the workload shapes and seeded generators; ``binding`` is the
thin ctypes layer over the C-ABI library ``liblayerpipe.so`` (see
``include/layerpipe.h``).  Importing this package does not load the library;
``binding`` does, and fails loudly when it is missing.
"""
import os as _os

# The stage scheduler runs three streams per pipeline stage.  Streams only overlap while each has
# a hardware work queue of its own, and a process gets 8 of them unless this variable says
# otherwise when its CUDA context is created (maximum 32).  Importing the package before the
# first CUDA call is therefore enough; a value the caller has already chosen is kept.
_os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")

__all__ = ["inputs", "binding", "build"]

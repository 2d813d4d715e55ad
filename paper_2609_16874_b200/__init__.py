"""B200-native decoder of sinusoidal centroid positional encodings into instance masks.

``binding`` is the ctypes front end of the CUDA library (``libcpe.so``, C ABI in ``include/cpe.h``);
``workloads`` makes the seeded synthetic inputs; ``build`` compiles the library with nvcc for sm_100a.
"""
from . import binding, build, workloads  # noqa: F401
from .binding import Decoder, HostDecoder, CpeError  # noqa: F401

__all__ = ["binding", "build", "workloads", "Decoder", "HostDecoder", "CpeError"]

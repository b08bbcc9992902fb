"""B200-native CLADA sparse gated FFN decode path (hand-written CUDA behind a C ABI).

``workloads`` draws the seeded synthetic inputs; ``binding`` is the thin ctypes layer over
``libclada.so`` (built by ``build.build()`` from ``csrc/``).  The CUDA library is loaded on
first use and its absence is an error: there is no CPU fallback.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "build"]

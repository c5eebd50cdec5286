"""B200-native biased graph attention + SPD build (C-ABI library ``libgtattn.so`` and its
thin ctypes binding).  ``workloads`` holds the seeded synthetic inputs."""
from . import workloads  # noqa: F401  (pure numpy; the CUDA library loads lazily on first call)

__all__ = ["workloads", "binding", "build"]

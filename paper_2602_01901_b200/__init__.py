"""B200-native Lazy Attention / Q Cache decode path (arxiv 2602.01901).

The package holds the CUDA kernels and host runtime behind a C ABI (``csrc/``,
``include/qc.h`` at the repository root), a thin ctypes binding (``binding``), and the
seeded synthetic workload generators (``workloads``).  Importing the package does not
load the native library; ``binding.load()`` does, and raises if it is missing.
"""

__all__ = ["binding", "workloads"]

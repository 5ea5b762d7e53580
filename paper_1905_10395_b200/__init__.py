"""Leader SGD step for a worker population resident on one B200 (CUDA library + thin binding).

`inputs` holds the seeded synthetic workload generators; `api` is the ctypes binding of
include/lsgd.h; `build` compiles the library in-tree.  The library is loaded on first use."""
from . import inputs  # noqa: F401

__all__ = ["inputs", "api", "build"]

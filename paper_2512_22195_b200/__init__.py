"""B200 (sm_100a) attention over materialised KV chunks: Python binding of the C-ABI library.

The package is a thin layer over ``libmatkv.so`` (built in-tree from ``csrc/`` by
``paper_2512_22195_b200.build``).  Importing it loads the library and raises if the
library is missing: there is no CPU or PyTorch fallback for any step of the path.
"""
from . import binding
from .binding import *  # noqa: F401,F403  (the matkv_* entry points, error codes, MatkvError)
from .binding import MatkvError, lib

lib()  # fail loudly at import time when the CUDA library has not been built

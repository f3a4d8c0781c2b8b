"""CFGzip decode-step path for NVIDIA B200: C-ABI CUDA library + a thin ctypes binding.

``from paper_2605_29986_b200 import binding`` gives the calls of ``include/cfgzip.h`` under the
same names. The CUDA library is built in-tree with nvcc (sm_100a) on first use.
"""
from . import binding  # noqa: F401
from .binding import *  # noqa: F401,F403

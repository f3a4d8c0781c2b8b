"""CFGzip decode-step path for NVIDIA B200: C-ABI CUDA library + a thin ctypes binding.

``from paper_2605_29986_b200 import binding`` gives the calls of ``include/cfgzip.h`` under the
same names. The CUDA library is built in-tree with nvcc (sm_100a) on first use.
"""
from . import rows  # noqa: F401


def __getattr__(name):
    # the CUDA binding is imported on first use, so that host-only helpers work without nvcc or a GPU
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)

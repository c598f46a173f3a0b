"""B200-native low-bit tensor-parallel synchronisation codec (arXiv 2411.07942).

The product is the C-ABI library ``libtpq.so`` (hand-written CUDA for sm_100a,
sources under ``csrc/``, declarations in ``include/tpq.h``); ``binding`` is the
thin ctypes front end with the same names.  Nothing here falls back to a CPU
path: loading fails loudly when the library is missing.
"""

__all__ = ["binding", "synth", "build"]

"""HBM-resident parameter store with dynamic parameter allocation for one NVIDIA B200.

The product is the CUDA library `libps_b200.so` (C interface: include/ps.h);
this package holds its sources (`csrc/`), the build step (`build.py`) and a
thin ctypes binding (`binding.py`).
"""
from . import binding  # noqa: F401
from .binding import *  # noqa: F401,F403

"""CPU oracle of the parameter-server hot path.  Test infrastructure only.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do.
"""
from .ps_oracle import OracleStore, build_oracle  # noqa: F401
from .keymap import OracleKeyMap, KeyMapFull, ABSENT  # noqa: F401
from . import dsgd  # noqa: F401

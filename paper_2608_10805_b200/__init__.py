"""B200 (sm_100a) WTConv forward/backward: CUDA library + thin ctypes binding."""
from . import inputs, io_model  # noqa: F401  (pure host helpers; the CUDA binding loads lazily in .wtconv)

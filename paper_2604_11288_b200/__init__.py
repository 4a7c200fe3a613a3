"""B200-native Transactional Attention KV-cache compaction: hand-written sm_100a kernels behind a C ABI
(include/ta.h) with a thin ctypes binding of the same names (paper_2604_11288_b200.binding)."""
from . import binding  # noqa: F401
from .binding import *  # noqa: F401,F403

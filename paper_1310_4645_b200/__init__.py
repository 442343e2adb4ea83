"""Schedule-exact pipelined reduction on one B200 (uni-greedy / bi-greedy and the classic trees).

The package is a thin binding over librd.so (CUDA kernels + C ABI, built in-tree by
`paper_1310_4645_b200.build`).  Importing it never compiles anything and never falls back to a
CPU path: calls raise when the library is missing.
"""
from .binding import *  # noqa: F401,F403
from .binding import lib, LIB_PATH, EXPORTS, ALGOS, RdError, LibraryMissing, rd_model_t, rd_stats_t, PointerTable  # noqa: F401

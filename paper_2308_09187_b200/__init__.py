"""qgx: the data-parallel hot path of Q-GenX (arXiv 2308.09187) as hand-written CUDA for sm_100a.

The package is a thin binding over the C-ABI library libqgx.so (declared in include/qgx.h,
kernels in csrc/).  There is no CPU or PyTorch fallback: if the library cannot be built or
loaded, using the package raises.
"""
from .binding import *  # noqa: F401,F403
from .binding import lib, library_path, Context, EgState, QgxError, make_quant_cfg, make_operator, EXPORTS  # noqa: F401

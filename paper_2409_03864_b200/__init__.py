"""tdx: B200 (sm_100a) dense contractions -- matmul with folded transposes / negate and
zero-padded conv2d + bias + ReLU -- behind a C ABI (include/tdx.h, libtdx.so).

This package is the thin Python binding; every step of the computation runs in the CUDA
library.  There is no CPU or PyTorch fallback: importing a function works anywhere, calling
it needs libtdx.so (built in-tree with `python -m paper_2409_03864_b200.build`) and a B200.
"""
from .binding import *  # noqa: F401,F403
from .binding import TdxError, check, lib, tdx_config  # noqa: F401

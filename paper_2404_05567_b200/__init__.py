"""B200-native DS-MoE feed-forward layer (inference hot path): a ctypes binding over the C-ABI CUDA
library ``libdsmoe.so`` built from ``csrc/``.  See ``include/dsmoe.h`` for the contract."""
from .binding import *  # noqa: F401,F403
from .binding import (LayerDesc, DsmoeError, lib, make_desc, width, amax, status_string, EXPORTS,
                      F32, BF16, SELECT_THRESHOLD, SELECT_TOPK, SELECT_ALL)

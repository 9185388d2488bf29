"""PosS speculative-round library for B200 (sm_100a): C-ABI CUDA kernels plus a thin ctypes binding."""
from .binding import (POSS_BF16, POSS_FP32, POSS_MAX_DEPTH, POSS_MAX_ROWS, POSS_MAX_TOPK, Poss, PossError,  # noqa: F401
                      load_library, make_config, poss_config, to_device)
from .loop import plain_generate, speculative_generate  # noqa: F401

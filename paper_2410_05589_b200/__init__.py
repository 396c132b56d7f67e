"""B200-native ParallelSpec hot path: single-pass parallel draft step + lossless verify.

The work is done by hand-written sm_100a kernels behind the C ABI in ``include/ps.h``;
this package is the ctypes binding.  There is no CPU path.
"""
from .binding import (  # noqa: F401
    PS_DTYPE_BF16,
    PS_DTYPE_F32,
    PS_FLAG_FC_BIAS,
    PS_FLAG_UNFUSED_KERNELS,
    Drafter,
    PsError,
    load_library,
    philox_fill,
    verify_static,
)
from .build import build  # noqa: F401
from .synth_bridge import drafter_from_shape, to_device  # noqa: F401

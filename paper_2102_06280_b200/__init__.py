"""cb-DyBW round on one B200: thin Python binding over the C-ABI CUDA library (libdbw.so)."""
from .binding import (  # noqa: F401
    DbwError,
    Dbw,
    ModelLayout,
    lib,
    model_layout,
    WEIGHT_METROPOLIS,
    WEIGHT_UNIFORM,
    ORDER_LOCAL_THEN_MIX,
    ORDER_MIX_THEN_CORRECT,
    GEMM_FP32,
    GEMM_BF16,
    STATUS_BAD_B,
    STATUS_NAN_TIME,
    STATUS_WAIT_TIMEOUT,
    STATUS_BAD_INDEX,
)

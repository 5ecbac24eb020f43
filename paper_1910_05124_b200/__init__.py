"""B200 (sm_100a) PipeMare hot path: Python binding of the C-ABI library.

Importing the package does not load the CUDA library; the first use of
`binding.lib()` does, and fails loudly if it is missing.  There is no CPU
fallback.
"""
from . import binding  # noqa: F401
from .binding import (  # noqa: F401
    PM_F32, PM_BF16, PM_SGDM, PM_ADAM, PM_ACT_NONE, PM_ACT_RELU, PM_ACT_GELU, PM_OP_LINEAR, PM_LOSS_MSE,
    PipeMareError, Pipeline, FlatUpdate, lib,
)

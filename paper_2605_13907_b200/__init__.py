"""B200 (sm_100a) library for the LM-head step of an AIS-GRPO update.

Thin ctypes binding over ``libais_b200.so`` (C ABI in ``include/ais.h``).  The functions here only marshal
arguments: every step of the path runs in the library's CUDA kernels.  PyTorch supplies device memory and
the current stream.  There is no CPU fallback: without the built library, or without an sm_100 device, the
calls raise.
"""

from .binding import (  # noqa: F401
    AisError, Params, Diag, Shape, lib, lib_path, default_params, make_shape, workspace_bytes, workspace_min_bytes,
    quantize_fp8, quantize_fp8_cols, W_VD, W_DV, FP8_MX32, FP4_MX32, mx_scale_bytes, logprob_fwd, diagnostics, loss_bwd, AisStep, logprob_train_static, STATIC_MAX_ROWS, diag_moments, diag_finalize, NUM_MOMENTS, RowCompaction,
    FLAG_EMPTY, FLAG_TOKEN_RANGE, FLAG_NONFINITE, FLAG_TIMEOUT, set_wait_cycles,
)

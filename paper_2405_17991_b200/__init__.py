"""B200 (sm_100a) implementation of VeLoRA's rank-1 sub-token projection for linear layers.

The work is done by hand-written CUDA kernels in ``libvelora.so`` (sources in
``csrc/``, C-ABI in ``include/velora.h``); this package only marshals
arguments.  Build the library with ``python -m paper_2405_17991_b200.build``.
"""
from .binding import (  # noqa: F401
    BF16, F32, LIB_PATH, OP_INIT_V, OP_LINEAR_BACKWARD_EXPLICIT, OP_LINEAR_BACKWARD_FACTORED,
    OP_LINEAR_FORWARD, OP_WEIGHT_GRAD_EXPLICIT, OP_WEIGHT_GRAD_FACTORED, SIGNATURES, WG_EXPLICIT,
    WG_FACTORED, VeloraError, lib, num_subtokens, velora_compress, velora_init_v, velora_init_v_static,
    velora_linear_backward, velora_linear_forward, velora_reconstruct, velora_status_string,
    velora_version, velora_weight_grad, velora_workspace_alloc, velora_workspace_bytes,
    velora_workspace_init, velora_workspace_status, velora_launch_count, velora_device_error, velora_subtoken_sum, velora_normalize_v,
    velora_update_v, OP_UPDATE_V, ERR_DEGENERATE_V, ERR_TIMEOUT, velora_selftest_wait_timeout,
    velora_z8_calibrate, FP8_E4M3, OP_Z8_CALIBRATE, Z8_TORCH,
    velora_dense_product, PRODUCT_A_BT, PRODUCT_A_B, PRODUCT_AT_B,
    velora_weight_grad_p, velora_expand_p,
    velora_host_step_staging_bytes, velora_linear_step_host,
)
from .memory_model import saved_activation_bytes  # noqa: F401

"""MUXQ quantized linear layer for NVIDIA B200 (sm_100a): Python binding of the C-ABI library.

Every step of the method runs inside libmuxq.so's CUDA kernels; this package only marshals
torch tensors (device memory, streams) into the C calls.  There is no CPU or framework fallback:
if the library has not been built, importing a function from here raises.
"""
from .binding import (  # noqa: F401
    MuxqParams, Workspace, lib, library_path, muxq_aux_cols, muxq_build_aux, muxq_detect_outliers,
    muxq_gemm, muxq_linear, muxq_linear_events, muxq_linear_host, muxq_linear_decode_noalloc, muxq_quantize, muxq_read_status, muxq_status_string, muxq_int8_mma_peak, muxq_test_hooks, Chain, MUXQ_LAYER_WAIT_PREV,
    muxq_workspace_bytes, muxq_small_workspace_bytes, muxq_host_workspace_bytes, muxq_workspace_view,
    MUXQ_OK, MUXQ_ERR_INVALID_ARG, MUXQ_ERR_UNSUPPORTED, MUXQ_ERR_WORKSPACE, MUXQ_ERR_CUDA,
    MUXQ_ERR_CAPACITY, MUXQ_ERR_TIMEOUT, MUXQ_ERR_STATIC_LIMIT, MUXQ_PER_TENSOR, MUXQ_PER_VECTOR, MUXQ_OUT_F16,
    MUXQ_OUT_F32, MUXQ_OUT_ACC_I32, MUXQ_AUX_SHARED, MUXQ_AUX_OWN, MuxqError,
)

"""B200 (sm_100a) SBP library: boxing transforms between SBP signatures and the sharded
operators they feed, over k logical shards resident in one GPU's memory.

This package is a thin ctypes binding over the C ABI declared in include/sbp.h.  It
marshals arguments only -- every step runs in the library's CUDA kernels -- and it fails
loudly when the compiled library is missing: there is no CPU or PyTorch fallback.
"""
from .binding import (  # noqa: F401
    B, P_MAX, P_SUM, S, Sig, SbpError, SbpTensor,
    empty_global, lib_path, load_library,
    sbp_boxing, sbp_boxing_shard, sbp_boxing_host, sbp_boxing_host_workspace_bytes, sbp_boxing_host_copy_bytes, sbp_boxing_host_multi, sbp_boxing_host_multi_workspace_bytes, sbp_boxing_host_multi_copy_bytes, sbp_boxing_set_copy_engine,
    sbp_check_device_errors, sbp_debug_bounds_enabled, sbp_selftest_debug_bounds, sbp_tensor_map_stats, sbp_matmul_form_stats, sbp_matmul_route, sbp_matmul_set_form, SBP_TC_FORM_AUTO, SBP_TC_FORM_SQUARE, SBP_TC_FORM_TALL, SBP_TC_FORM_MIXED, sbp_view_b_to_s, sbp_embedding, sbp_embedding_backward, sbp_launch_count, sbp_local_shape, sbp_matmul,
    sbp_matmul_infer, sbp_matmul_softmax_xent, sbp_matmul_softmax_xent_backward, sbp_matmul_softmax_xent_workspace_bytes, sbp_matmul_workspace_bytes, sbp_selftest_wait_timeout, sbp_softmax_xent,
    sbp_softmax_xent_backward, sbp_transfer_cost, sbp_softmax_xent_static, sbp_softmax_xent_workspace_bytes, SBP_EPILOGUE_GELU, SBP_TRANS_X, SBP_TRANS_W,
)

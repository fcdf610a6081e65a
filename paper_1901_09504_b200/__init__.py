"""B200 (sm_100a) library for outlier channel splitting post-training quantization
(arXiv:1901.09504): Python binding of the C ABI declared in include/ocs.h."""
from .binding import (  # noqa: F401
    CLIP_ACIQ, CLIP_KL, CLIP_MSE, CLIP_MSE_EXACT, CLIP_NONE, DEV_BAD_INDEX, DEV_DEPTH, DEV_NONFINITE, DEV_OVERFLOW, DEV_TIMEOUT, EXPORTS, LIB_PATH, OcsError, lib,
    new_status, ocs_kernel_launches, ocs_num_splits, ocs_conv_packed_k, ocs_pack_conv_weights, ocs_pack_conv_weights_batch, ocs_poll_status, ocs_qconv, ocs_qlinear, ocs_quantize, ocs_quantize_noalloc,
    ocs_split, ocs_split_quantize, ocs_split_quantize_batch, ocs_dup_weight_columns, ocs_fold_duplicates, ocs_act_select_channels, ocs_act_split_quantize_static, ocs_add_relu, ocs_maxpool3x3s2, ocs_global_avgpool, ocs_nchw_to_nhwc, ocs_embedding,
    ocs_lstm_cell, ocs_transpose_codes, ocs_selftest_force_gemm_plan, ocs_selftest_wait_expiry, ocs_range_curve, ocs_knapsack_allocate, ocs_trace_start, ocs_trace_stop, round_up,
)

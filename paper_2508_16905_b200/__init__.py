"""Tri-Accel fused optimizer pass for NVIDIA B200 (sm_100a): Python binding of the C-ABI library.

The compute lives in libtriaccel.so (hand-written CUDA, built in-tree by build.py); this package
only marshals arguments.  Nothing here falls back to PyTorch or the CPU.
"""
from .binding import (dev_ptr, TA_FLAG_COOPERATIVE_LAUNCH, ta_path, TA_FLAG_GUARD_WORKSPACES, ta_test_check_guards, RECORD_BYTES, ta_create_shard, ta_shard_apply, ta_shard_sweep, TA_FLAG_INPUTS_FINITE, TA_FLAG_NO_ONE_LAUNCH, ta_plan_pipeline, ta_plan_items, ta_task, TA_CODE_BF16, TA_CODE_FP16, TA_CODE_FP32, TA_ERR_ALIGN, TA_ERR_ARG, TA_ERR_CUDA,  # noqa: F401
                      TA_ERR_NOMEM, TA_ERR_STATE, TA_OK, TriAccelError, make_hparams, ta_batch_ctrl, ta_batch_next,
                      ta_create, ta_destroy, ta_grad_moments_static, ta_hparams, ta_launch_count, ta_layer_stats, ta_masks,
                      ta_masks_to_host, ta_mem_reader, ta_plan_one_launch, ta_power_iterate, ta_set_curvature, ta_precision_codes, ta_probe, ta_set_lr, ta_state_load,
                      ta_state_save, ta_stats, ta_step, ta_step_host, ta_step_status, ta_test_expire_next_wait, ta_timing_begin,
                      ta_timing_end)

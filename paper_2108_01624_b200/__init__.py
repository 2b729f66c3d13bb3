"""B200-native DP-SGD privatised-gradient step (per-example clip, accumulate, noise, AdamW).

The compute lives in libdp_b200.so (hand-written sm_100a CUDA behind the C ABI of include/dp.h);
`binding` marshals torch tensors into it and `step` strings the calls into a macro-step.
Importing the package does not load the library; the first call does, and fails loudly if it is absent.
"""
from . import binding, synth  # noqa: F401
from .binding import (DP_PATH_AUTO, DP_PATH_GRAM, DP_PATH_MATERIALIZED, DpError, Layer, LayerList,  # noqa: F401
                      alloc_workspace, dp_adamw_step, dp_add_noise_and_scale, dp_clip_factors, dp_clip_stats, dp_noise_scale_adamw_step_snr,
                      dp_clipped_accumulate, dp_clipped_accumulate_after_sqnorms, dp_noise_scale_adamw_step, dp_reduce_noise_adamw_step, dp_per_example_sqnorms, dp_philox_u32,
                      dp_launch_count, dp_layernorm_sqnorms_static, dp_poll_status, dp_shared_table_cross_sqnorms, dp_token_equality_mask, dp_version, dp_workspace_bytes)
from .step import DeviceStatusError, DPStep  # noqa: F401

"""B200-native per-example gradient clipping (DP-SGD hot path).

The product is the C-ABI library `libdpclip.so` (hand-written sm_100a CUDA);
this package only marshals arguments to it.  Importing the package does not
load the library; the first call does, and fails loudly if it is missing.
"""
from .binding import (  # noqa: F401
    DPCLIP_AUTO, DPCLIP_BF16, DPCLIP_F32, DPCLIP_GRAM, DPCLIP_MATERIALIZE, DPCLIP_SIMT, DPCLIP_T1,
    DpclipError, HostStep, Layer, ModelLayer, ModelPlan, StepPlan,
    DPCLIP_KIND_CONV, DPCLIP_KIND_DENSE, DPCLIP_KIND_ELEMENTWISE, dpclip_model_step, dpclip_model_workspace_bytes, dpclip_add_noise, dpclip_clipped_grad, dpclip_clipped_grad_noalloc, dpclip_clipped_grad_noise, dpclip_conv_clipped_grad, dpclip_conv_sqnorms, dpclip_conv_workspace_bytes, dpclip_dp_adam_step, dpclip_dp_sgd_step, dpclip_noalloc_max_output_bytes, dpclip_elementwise_clipped_grad, dpclip_elementwise_sqnorms, dpclip_factors, dpclip_launch_count, dpclip_debug_build, dpclip_reload_path_switches, dpclip_null_launch,
    dpclip_layer_sqnorms, dpclip_pick_method, dpclip_read_status, dpclip_status_string,
    dpclip_gram_layers_sqnorms, dpclip_same_shape_layers_clipped_grad_noise, dpclip_step, dpclip_step_workspace_bytes, dpclip_step_streams, dpclip_model_step_streams, dpclip_step_host, dpclip_step_noise, dpclip_step_per_layer, dpclip_t1_layers_clipped_grad_noise, dpclip_t1_layers_sqnorms, dpclip_t1_layers_supported, dpclip_version, dpclip_workspace_bytes, dpclip_workspace_init,
    library_path, load_library,
)

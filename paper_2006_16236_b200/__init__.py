"""Linear attention ("Transformers are RNNs") for NVIDIA B200: Python face of the C ABI.

The names mirror ``include/la.h``.  Importing this package does not load the CUDA
library; the first call does, and raises if it has not been built.
"""
from .binding import (  # noqa: F401
    LaError, la_problem, make_problem, workspace, saved_buffer, linear_saved_buffer,
    la_feature_map, la_feature_map_poly2, la_feature_map_poly2_backward, poly2_columns, la_feature_map_rff, la_feature_map_rff_backward, prepare_recurrent_step, PreparedStep, la_linear_attention, la_linear_attention_noalloc, la_linear_attention_backward,
    la_linear_attention_varlen, la_linear_attention_varlen_backward,
    la_causal_forward, la_causal_backward, la_recurrent_step, la_recurrent_steps, la_decode_layer_step,
    la_workspace_bytes, la_last_device_status, la_kernel_launches, la_profile_enable, la_profile_read, la_version,
    la_causal_plan, la_plan_override,
    LA_F32, LA_BF16, LA_PHI_ELU1, LA_PHI_IDENTITY,
    LA_OP_LINEAR_FORWARD, LA_OP_LINEAR_BACKWARD, LA_OP_CAUSAL_FORWARD, LA_OP_CAUSAL_BACKWARD, LA_OP_CAUSAL_SAVED, LA_OP_DECODE_LAYER,
)

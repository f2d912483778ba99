"""xrl: the per-step forward pass of the X-RLflow agent on one B200 (hand-written CUDA, sm_100a).

The compute lives in libxrl.so (C ABI, declared in include/xrl.h); this package only marshals
arguments.  There is no CPU fallback: importing works without a GPU, creating a context does not.
"""
from .binding import (  # noqa: F401
    XrlError, Agent, load_library, library_path, model_config,
    xrl_create, xrl_destroy, xrl_weights_size, xrl_set_weights, xrl_get_weights, xrl_init_weights, xrl_pack, xrl_pack_flat,
    xrl_batch_free, xrl_batch_info, xrl_batch_export, xrl_encode, xrl_debug_node_features,
    xrl_policy_value, xrl_sample, xrl_last_device_status, xrl_launch_counts, xrl_version,
    xrl_profile, xrl_profile_read, xrl_pack_csr_static, xrl_encode_delta, xrl_delta_rows, xrl_graph_begin,
    xrl_graph_launch, xrl_batch_set_edge_attr, xrl_ppo_grad, xrl_gae, xrl_grad_weigh, xrl_grad_unweigh, allreduce_ppo_grad, STATUS_NAMES, EXPORTED_SYMBOLS, PROFILE_FAMILIES,
)

"""B200 (sm_100a) FIRP draft+verify decoder step: Python binding of the C ABI in include/firp.h.

The binding only marshals arguments (ctypes); every step of the path runs in the CUDA
kernels of libfirp_b200.so.  There is no CPU fallback: importing `binding` fails loudly
when the library has not been built.
"""
from .binding import (FirpError, FirpEngine, StepOut, firp_create, firp_destroy, firp_last_error,  # noqa: F401
                      firp_workspace_bytes, firp_kv_bytes, firp_bind_buffers, firp_init_weights, firp_prefill,
                      firp_step, firp_kv_commit, firp_context_len, firp_set_context_len,
                      firp_last_launch_count, firp_profile_enable, firp_profile_read,
                      firp_kernel_class_name, firp_topb_static, firp_prefill_layers, firp_step_layers, firp_step_chains, firp_step_trees, firp_set_pseudo_masked,
                      firp_set_fused, firp_set_pred_prenorm, firp_set_kv_pages, firp_set_activation_planes, firp_set_attention_planes, firp_set_attention_kernel, firp_set_wait_limit_us, firp_selftest_wait, lib_path, load_library, ModelCfg, Weights, StepOutC)

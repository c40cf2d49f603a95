"""B200-native fused attention (forward + backward) behind a C ABI.

``libvtattn.so`` (hand-written sm_100a kernels, built in-tree by
``paper_2601_16238_b200.build``) does all the work; this package only marshals
arguments.  Importing the package does not need a GPU; calling any ``vt_attn_*``
function does, and raises if the library has not been built.
"""
from .binding import (ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_INVALID_ARGUMENT, ERR_STATIC_SCRATCH_TOO_SMALL, ERR_UNSUPPORTED,  # noqa: F401
                      ERR_WORKSPACE_TOO_SMALL, EXPORTS, LIB_PATH, OK, VtAttnError, load_library,
                      STATIC_SCRATCH_ROWS, vt_attn_accumulate_partial, vt_attn_bwd, vt_attn_bwd_static_scratch, vt_attn_bwd_static_scratch_f16, vt_attn_bwd_varlen, vt_attn_bwd_varlen_workspace_bytes,
                      vt_attn_bwd_workspace_bytes, vt_attn_bwd_kernel_kind, vt_attn_bwd_dv, vt_attn_bwd_dv_f16, vt_attn_bwd_f16, vt_attn_fwd_f16, vt_attn_fwd_dv, vt_attn_fwd_rope, vt_attn_fwd_dv_f16, vt_attn_fwd_kernel_kind, vt_attn_fwd_varlen, vt_attn_device_status, vt_attn_device_status_async, vt_attn_device_status_clear, vt_attn_fwd,
                      vt_attn_fwd_bwd_host, vt_attn_fwd_bwd_host_f16, vt_attn_fwd_host, vt_attn_fwd_host_f16, vt_attn_fwd_splitkv, vt_attn_fwd_splitkv_f16, vt_attn_fwd_splitkv_varlen, vt_attn_fwd_splitkv_varlen_f16, vt_attn_fwd_splitkv_varlen_plan, vt_attn_fwd_splitkv_plan, vt_attn_fwd_varlen_f16, vt_attn_bwd_varlen_f16, vt_attn_get_info, vt_attn_host_staging_bytes, vt_attn_merge_finish, vt_attn_merge_partial,
                      vt_attn_selftest_tile, vt_attn_selftest_timeout)

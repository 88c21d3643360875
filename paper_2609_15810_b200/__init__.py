"""VC-Attention hot path for NVIDIA B200 (sm_100a): thin Python binding over libvc.so.

Every step of the path runs in the library's CUDA kernels; this package only marshals
arguments (PyTorch supplies device memory and streams).  Importing the binding raises if
the library has not been built (``python -m paper_2609_15810_b200.build``): there is no
CPU fallback.
"""
from .binding import (VcError, Params, QuantView, load_library, vc_attn, vc_attn_fwd,  # noqa: F401
                      vc_attn_host, vc_group, vc_group_schedule, vc_group_workspace_bytes,
                      VC_GROUP_FROZEN, VC_GROUP_RECOMPUTE, VC_GROUP_REUSE, vc_launch_count, vc_poll_status, vc_prep, vc_prep_noalloc, vc_quant_bytes,
                      vc_quant_view, vc_status_string, vc_workspace_bytes,
                      vc_test_set_wait_limit, vc_test_expcast_codes, vc_mma_peak, vc_prep_with_stats, vc_prep_stats_view, VC_FLAG_CHECK_PERM, VC_GROUP_LABELS_OFFSET,
                      VC_OK, VC_ERR_INVALID_ARG, VC_ERR_UNSUPPORTED, VC_ERR_TIMEOUT,
                      VC_FLAG_ALL, VC_FLAG_HADAMARD, VC_FLAG_INT8_QK, VC_FLAG_K_SMOOTH, VC_FLAG_ROPE, VC_FLAG_V_SMOOTH,
                      VC_P_DEFAULT, VC_P_EXPCAST_E4M3, VC_P_EXP_E4M3, VC_P_NVFP4,
                      VC_P_EXP_POLY_E4M3, VC_P_EXP_MIX_E4M3)

"""B200 (sm_100a) verification step of speculative decoding for VLMs.

The product is ``libmassv.so`` (C ABI declared in ``include/massv.h``); this
package is its thin Python binding plus a convenience wrapper that runs one
whole verify step on a workload.
"""
from .binding import (AcceptDesc, AttnDesc, MassvError, accept_desc, alloc_workspace, attn_desc, massv_accept, massv_accept_static,
                      massv_accept_workspace_size, massv_kv_commit, massv_launch_count, massv_tvd, massv_tvd_after_accept, massv_tvd_workspace_size, massv_strerror, massv_verify_attn,
                      massv_verify_attn_workspace_size, massv_version, massv_set_timing_events, massv_set_kernel_timing, massv_sample_top_p, massv_tvd_histogram, LIB_PATH)
from .step import VerifyStep

__all__ = ["AcceptDesc", "AttnDesc", "MassvError", "accept_desc", "alloc_workspace", "attn_desc", "massv_accept", "massv_accept_static",
           "massv_accept_workspace_size", "massv_kv_commit", "massv_launch_count", "massv_tvd", "massv_tvd_after_accept", "massv_tvd_workspace_size", "massv_strerror", "massv_verify_attn",
           "massv_verify_attn_workspace_size", "massv_version", "massv_set_timing_events", "massv_set_kernel_timing", "massv_sample_top_p", "massv_tvd_histogram", "VerifyStep", "LIB_PATH"]

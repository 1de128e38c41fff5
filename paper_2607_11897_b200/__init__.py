"""Python binding of the SFDA C-ABI library (``libsfda.so``, hand-written CUDA for sm_100a).

Argument marshalling only: every step of the path runs in the library's kernels.
PyTorch is used for device memory and streams.  There is no CPU or PyTorch
fallback: a missing library raises.
"""
from .binding import (SFDA_BF16, SFDA_F32, SfdaError, last_launch_count, lib_path, load, sfda_chunk_factors,
                      sfda_backward, sfda_backward_workspace_bytes, sfda_forward, sfda_forward_decoupled, sfda_forward_blocks, sfda_step_blocks, ERASE_COMPLEX, ERASE_REAL, sfda_forward_two_level, sfda_forward_two_level_workspace_bytes, sfda_forward_fused, sfda_forward_fused_workspace_bytes, sfda_frontend, sfda_frontend_backward, sfda_forward_host, sfda_forward_noalloc, sfda_forward_phase, sfda_forward_withheld_handoff, sfda_noalloc_status, sfda_forward_host_arena_bytes, sfda_forward_simt, sfda_forward_partition, sfda_plan, sfda_status_string, sfda_step, sfda_step_decoupled, sfda_step_fused,
                      sfda_workspace_bytes, sfda_workspace_status)

__all__ = ["SFDA_BF16", "SFDA_F32", "SfdaError", "last_launch_count", "lib_path", "load", "sfda_chunk_factors",
           "sfda_backward", "sfda_backward_workspace_bytes", "sfda_forward", "sfda_forward_decoupled", "sfda_forward_blocks", "sfda_step_blocks", "ERASE_COMPLEX", "ERASE_REAL", "sfda_forward_two_level", "sfda_forward_two_level_workspace_bytes", "sfda_forward_fused", "sfda_forward_fused_workspace_bytes", "sfda_frontend", "sfda_frontend_backward", "sfda_forward_host", "sfda_forward_noalloc", "sfda_forward_phase", "sfda_forward_withheld_handoff", "sfda_noalloc_status", "sfda_forward_host_arena_bytes", "sfda_forward_simt", "sfda_forward_partition", "sfda_plan", "sfda_status_string", "sfda_step", "sfda_step_decoupled", "sfda_step_fused",
           "sfda_workspace_bytes", "sfda_workspace_status"]

"""B200-native speculative rejection-sampling verify step (C-ABI library + thin binding).

The arithmetic lives entirely in the CUDA library ``libbebop.so`` (built in-tree
from ``csrc/`` for sm_100a).  This package only marshals arguments; there is no
CPU or PyTorch fallback: importing the binding without the built library, or
calling it without a CUDA device, raises.
"""
from .binding import (BEBOP_BF16, BEBOP_F32, BebopError, bebop_debug_expire_wait, bebop_debug_fallback_offset, bebop_debug_last_kernel, bebop_debug_set_draw_kappa,
                      bebop_debug_force_general_path, bebop_debug_set_timing_events, bebop_greedy_verify, bebop_status_string,
                      bebop_tv, bebop_tv_static, bebop_verify, bebop_workspace_bytes, library_path, load_library)

__all__ = ["bebop_verify", "bebop_tv", "bebop_tv_static", "bebop_greedy_verify", "bebop_workspace_bytes",
           "bebop_status_string", "bebop_debug_force_general_path", "bebop_debug_expire_wait", "bebop_debug_set_draw_kappa", "bebop_debug_last_kernel", "bebop_debug_fallback_offset", "bebop_debug_set_timing_events", "BebopError", "BEBOP_F32", "BEBOP_BF16", "library_path",
           "load_library"]

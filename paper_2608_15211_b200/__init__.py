"""B200 (sm_100a) shifted-window attention block of the TERRA forecaster.

The product is the C-ABI CUDA library (include/terra.h, csrc/); this package builds it
in-tree and exposes a thin ctypes binding with the same names.  Importing the package
does not load the library; the first call does, and raises if it is missing.
"""
from .binding import (TerraError, launch_count, profile_enable, profile_read, selftest_bounded_wait, load_library, make_desc, terra_route_sizes,  # noqa: F401
                      terra_fixed_assignment_padding, terra_ragged_window_range, terra_swin_attn_bwd_packed, terra_swin_attn_fwd_packed,
                      terra_swin_attn_bwd, terra_swin_attn_fwd, terra_swin_attn_fwd_noalloc, terra_swin_check, terra_swin_desc, terra_swin_workspace_bytes,
                      terra_window_route, terra_pad_grid, terra_crop_grid, padded_extent)
from .workloads import CONFIGS, SwinConfig, make_inputs  # noqa: F401

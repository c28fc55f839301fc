"""B200-native multi-coil SENSE data-consistency step (GLEAM, arXiv 2207.08393, Eq. 3) and its
vector-Jacobian product, plus the MoDL model inversion (Eq. 7) by conjugate gradients.  The arithmetic lives in the CUDA library ``libgleam_dc.so`` (C ABI in
``include/gleam.h``); this package is the argument-marshalling binding plus the seeded synthetic
workload generators."""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    DataConsistency, GleamError, GLEAM_MASK_FULL, GLEAM_MASK_READOUT_INVARIANT, gleam_dc_forward,
    gleam_dc_length_supported, gleam_dc_vjp, gleam_dc_workspace_size, gleam_dims, gleam_status_string,
    gleam_version, load_library, make_dims, gleam_dc_forward_host, gleam_dc_vjp_host, gleam_dc_host_arena_size,
    gleam_dc_forward_static, gleam_dc_static_scratch_bytes, gleam_dc_launch_count, gleam_dc_profile_begin, gleam_dc_profile_end, KERNEL_CLASSES,
    gleam_dc_prepare, gleam_dc_forward_prepared, gleam_dc_forward_aty, gleam_dc_adjoint, gleam_dc_check_status, gleam_dc_debug_fused, gleam_dc_fused_wait_stats, gleam_dc_set_fused, gleam_dc_grad_eta, gleam_dc_grad_y, gleam_dc_grad_workspace_size, gleam_dc_forward_layout, gleam_dc_vjp_layout,
    gleam_l1_loss, gleam_l1_loss_workspace_size, gleam_measure_fp32_peak, gleam_dc_rowtile_split, GLEAM_X_CHANNELS, GLEAM_OUT_CHANNELS, ModlCG, gleam_modl_cg_forward, gleam_modl_cg_vjp, gleam_modl_cg_workspace_size,
)

"""B200-native fused vocabulary projection + cross-entropy (single-device Ring-DTP, paper §3.2 / App. C).

The package is a thin binding over the C-ABI library ``libvpce.so`` (hand-written sm_100a
kernels).  There is no CPU or PyTorch fallback: every call raises if the library is missing.
"""
from .binding import (  # noqa: F401
    VpceError,
    library_path,
    load_library,
    vp_ce_backward,
    vp_ce_device_status,
    vp_ce_forward,
    vp_ce_backward_f32,
    vp_ce_forward_f32,
    vp_ce_forward_static,
    vp_ce_workspace_bytes_f32,
    vp_ce_fwd_bwd_host,
    vp_ce_profile_collect,
    vp_ce_profile_enable,
    vp_ce_set_tail_parts,
    vp_ce_tail_choice,
    vp_ce_set_wait_limit_ns,
    vp_ce_debug_drop_copy,
    KERNEL_KINDS,
    vp_ce_launch_count,
    vp_ce_mean_loss,
    vp_ce_meeting_backward,
    vp_ce_meeting_forward,
    vp_ce_meeting_workspace_bytes,
    PHASE_RESIDUAL,
    PHASE_INPUT_GRAD,
    PHASE_WEIGHT_GRAD,
    vp_ce_mean_loss_grad,
    vp_ce_status_string,
    vp_ce_workspace_bytes,
    osadamw_create,
    osadamw_destroy,
    osadamw_staging_bytes,
    osadamw_step,
    osadamw_update_device,
    osadamw_wait,
)


def __getattr__(name):
    # the autograd front end needs torch; import it lazily so the C-ABI binding works without it
    if name in ("vocab_proj_cross_entropy", "vocab_proj_cross_entropy_mean"):
        from . import autograd as _ag
        return getattr(_ag, name)
    if name == "HostStepPipeline":
        from . import host_pipeline as _hp
        return _hp.HostStepPipeline
    if name in ("RingDTP", "DistTransport", "CudaMeetings", "choose_schedule", "shard_interval"):
        from . import ring as _ring
        return getattr(_ring, name)
    raise AttributeError(name)

"""IMPACT learner hot path for B200: fused loss + gradient kernels and the circular buffer.

The package is a thin binding over `libimpact.so` (built from `csrc/` for sm_100a); the
library is loaded on first use and its absence is an error.
"""
from .binding import (  # noqa: F401
    Coefficients, ImpactBuffer, ImpactError, PreparedCall, TERM_NAMES,
    impact_gather_rows, impact_loss_fwd_bwd, impact_loss_fwd_bwd_gaussian,
    impact_get_option, impact_loss_fwd_bwd_static_scratch, impact_loss_static_scratch_status, impact_set_option,
    impact_loss_workspace_bytes, impact_loss_workspace_init, impact_loss_workspace_status, impact_status_string,
    impact_version, load_library, new_workspace, prepare_loss_fwd_bwd,
    new_loss_inputs_record, prepare_loss_fwd_bwd_from_record, prepare_loss_fwd_bwd_gaussian, prepare_stream_copy,
)
from . import binding  # noqa: F401
from .kl_controller import AdaptiveKL  # noqa: F401
from .sharded import impact_loss_fwd_bwd_sharded, reduce_loss_terms, shard_bounds  # noqa: F401

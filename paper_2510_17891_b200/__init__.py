"""B200-native HRD policy-gradient scoring path (TritonRL, Section 2.3).

The work is done by libtrl.so (hand-written CUDA for sm_100a, C ABI declared in
include/trl.h).  This package is a thin ctypes binding with the same entry-point names;
torch is used only for device buffers and streams.  There is no CPU or PyTorch fallback:
every call raises if the library is missing or reports an error.
"""
from .binding import (  # noqa: F401
    TRL_F32, TRL_BF16, TRL_CALL_TOKEN_LOGPROBS, TRL_CALL_PG_LOSS_FWD, TRL_CALL_PG_LOSS_BWD, TRL_CALL_PG_STEP_FUSED,
    TrlError, PgConfig, lib_path, load_library, exported_symbols,
    trl_workspace_bytes, trl_workspace_bytes_min, trl_status_string, trl_kernel_launches, trl_config_string,
    trl_token_logprobs, trl_hrd_advantages, trl_pg_loss_fwd, trl_pg_loss_fwd_static, trl_pg_loss_bwd, trl_pg_step_fused,
    trl_pg_step_fused_banded, trl_pg_step_fused_banded_workspace_bytes, trl_dw_band_plan,
    check_status, hrd_pg_step,
)

"""B200-native A-3PO log-prob + loss hot path: thin binding over the C-ABI library liba3po.so.

Importing the package does not load the compiled library; the first call does, and raises if
it is missing (build it with `python -m paper_2512_06547_b200.build`).
"""
from .binding import (  # noqa: F401
    A3PO_BF16,
    A3PO_F32,
    STATUS_TARGET_OUT_OF_RANGE,
    STATUS_WAIT_TIMEOUT,
    A3poError,
    a3po_decoupled_loss_fwd_bwd,
    a3po_grpo_advantages,
    a3po_grpo_workspace_bytes,
    a3po_kernel_launch_count,
    a3po_selftest_wait_timeout,
    a3po_loss_bwd,
    a3po_loss_fwd,
    a3po_loss_fwd_bwd,
    a3po_loss_fwd_static,
    a3po_loss_workspace_bytes,
    a3po_profile_enable,
    a3po_profile_read,
    a3po_token_logprobs_bwd,
    a3po_token_logprobs_fwd,
    a3po_token_logprobs_min_workspace_bytes,
    a3po_token_logprobs_workspace_bytes,
    a3po_train_step,
    a3po_train_step_host,
    a3po_train_step_min_workspace_bytes,
    a3po_train_step_stage_bytes,
    a3po_train_step_workspace_bytes,
    a3po_version,
    exported_symbols,
    load_library,
    new_stats,
    new_workspace,
    read_stats,
)

"""mdraft: conv1d + selective-SSM (S6) + gate for a Mamba drafter on NVIDIA B200 (sm_100a).

The product is the CUDA library ``libmdraft.so`` (C ABI in ``include/mdraft.h``);
``binding`` marshals torch tensors into it.  Nothing here computes on the CPU and
nothing falls back: without the built library every call raises.
"""

from .binding import (  # noqa: F401
    MDRAFT_A_POWERS, MDRAFT_BF16, MDRAFT_CONV_ONLY, MDRAFT_DEV_BAD_SEQLENS, MDRAFT_DEV_BAD_SLOT,
    MDRAFT_DEV_WAIT_EXPIRED, MDRAFT_DT_SOFTPLUS, MDRAFT_F32, MDRAFT_PRECONV,
    Layer, MdraftError, StateCache, UcbBandit, load_library, mdraft_ucb_reward,
    mdraft_classify_A, mdraft_conv_scan_prefill, mdraft_conv_scan_prefill_noalloc, mdraft_prefill_workspace_bytes,
    NOALLOC_SCRATCH_BYTES,
    SsdLayer, mdraft_ssd_prefill, mdraft_ssd_prefill_workspace_bytes, mdraft_ssd_tree_step,
    mdraft_state_commit, mdraft_tree_step, mdraft_tree_step_proj, mdraft_version, status_string,
)

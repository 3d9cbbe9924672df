"""B200-native fused LM-head log-probability + GRPO policy-loss path.

The compute lives in librlhead.so (hand-written sm_100a kernels, C ABI in
include/rlhead.h); `binding` marshals torch tensors into it; `workloads` holds
the seeded synthetic input generators.  Importing this package loads nothing;
the shared library is opened on first use and its absence is an error.
"""
from .binding import (Context, RLHeadError, default_context, load_library, rl_grpo_advantages,  # noqa: F401
                      rl_policy_loss_fwd_bwd, rl_token_logprobs)

"""B200-native fused UloRL token-loss path (LM head + log-softmax + entropy + SAIS/POIS ratio +
MPT mask + clipped token-normalised loss, forward and backward) behind a C ABI.

`binding` wraps libulorl.so (hand-written CUDA for sm_100a); `dp` is the host logic of the data-parallel
step (rank launch, sharding, the collectives); `segments` the bookkeeping of the segment rollout.
Importing the package does not load the library; the first call does and raises if it is missing.
"""
from . import binding, dp  # noqa: F401
from .binding import (Params, UlorlError, alloc_fwd_outputs, alloc_workspace, check_status, launch_count,  # noqa: F401
                      token_loss_bwd, token_loss_decide, token_loss_fwd, workspace_bytes)

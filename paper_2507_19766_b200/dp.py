"""Data-parallel host logic of the token-loss path: one process per GPU, whole sequences per rank.

Per-token quantities (log-prob, entropy, the mean entropy of a sequence, the mask and clip decisions,
dHidden) never cross ranks when sequences are not split.  What does: the normaliser N of Eq. 10 (the
global count of response tokens, known before the step), the head gradient d_W (summed), and the
scalar loss and counters (summed).  The collective is whatever backend torch.distributed was
initialised with (NCCL over NVLink on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def shard_sequences(lengths: Sequence[int], world_size: int) -> List[List[int]]:
    """Assign whole sequences to ranks, longest first to the least loaded rank, so that token
    counts are as even as the long tail allows.  Returns, per rank, the sequence indices in
    ascending order.  Every rank gets at least one sequence when there are enough of them."""
    order = sorted(range(len(lengths)), key=lambda i: (-int(lengths[i]), i))
    loads = [0] * world_size
    shards: List[List[int]] = [[] for _ in range(world_size)]
    for i in order:
        r = min(range(world_size), key=lambda k: (loads[k], k))
        shards[r].append(i)
        loads[r] += int(lengths[i])
    return [sorted(s) for s in shards]


def global_token_count(local_tokens: int, device=None) -> int:
    """N of Eq. 10 over all ranks (each rank passes it as norm_tokens)."""
    if not (dist.is_available() and dist.is_initialized()):
        return int(local_tokens)
    t = torch.tensor([int(local_tokens)], dtype=torch.int64, device=device)
    dist.all_reduce(t)
    return int(t.item())


def reduce_step_outputs(d_W: torch.Tensor, loss: torch.Tensor, counters: torch.Tensor = None):
    """Sum d_W, the loss and (optionally) an int64 counter vector over ranks, in place.  With
    norm_tokens = global N on every rank the summed loss is the loss of the global batch."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return
    dist.all_reduce(d_W)
    dist.all_reduce(loss)
    if counters is not None:
        dist.all_reduce(counters)

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


# ---------------------------------------------------------------------------------------------
# Token-range sharding: when one ultra-long response dominates the batch, whole sequences no longer
# balance and a rank takes a contiguous range of tokens instead.  A sequence can then straddle ranks,
# and the mean entropy of Eq. 10 that gates its mask is the one quantity of the decision stage that
# needs every piece: each rank sums the entropies of its pieces, one small all-reduce of
# (sum, count) per sequence follows, and the decision stage runs with the means supplied.
# ---------------------------------------------------------------------------------------------

def shard_token_ranges(total_tokens: int, world_size: int, align: int = 1) -> List[tuple]:
    """Contiguous [lo, hi) token ranges, one per rank, equal up to `align` (the row-tile height, so that
    only the last rank has a ragged tile)."""
    per = -(-total_tokens // world_size)
    per = -(-per // align) * align
    return [(min(total_tokens, r * per), min(total_tokens, (r + 1) * per)) for r in range(world_size)]


def local_sequence_pieces(seq_offsets: Sequence[int], lo: int, hi: int):
    """The pieces of sequences inside the token range [lo, hi): (ids, local_offsets) with ids the global
    sequence indices that have at least one token in the range and local_offsets [len(ids) + 1] their
    boundaries relative to lo."""
    ids, offs = [], [0]
    for i in range(len(seq_offsets) - 1):
        a, b = max(int(seq_offsets[i]), lo), min(int(seq_offsets[i + 1]), hi)
        if b > a:
            ids.append(i)
            offs.append(b - lo)
    return ids, offs


def sequence_entropy_partials(piece_mean: torch.Tensor, piece_tokens: torch.Tensor, ids: Sequence[int],
                              num_seqs: int) -> torch.Tensor:
    """[num_seqs, 2] float64 (entropy sum, token count) of this rank's pieces, zero elsewhere.  piece_mean is
    what the forward call reports per local sequence (its seq_entropy output), piece_tokens their lengths."""
    acc = torch.zeros(num_seqs, 2, dtype=torch.float64, device=piece_mean.device)
    idx = torch.as_tensor(list(ids), dtype=torch.int64, device=acc.device)
    n = piece_tokens.to(torch.float64).to(acc.device)
    acc[idx, 0] = piece_mean.to(torch.float64) * n
    acc[idx, 1] = n
    return acc


def sequence_entropy_from_partials(acc: torch.Tensor, ids: Sequence[int]) -> torch.Tensor:
    """Mean entropy (float32, the type the decision stage compares with sigma) of the sequences `ids` from
    the summed partials."""
    idx = torch.as_tensor(list(ids), dtype=torch.int64, device=acc.device)
    return (acc[idx, 0] / acc[idx, 1]).to(torch.float32)


def exchange_sequence_entropy(piece_mean: torch.Tensor, piece_tokens: torch.Tensor, ids: Sequence[int],
                              num_seqs: int) -> torch.Tensor:
    """Mean entropy per sequence over all ranks' pieces, returned for this rank's pieces: one all-reduce of
    [num_seqs, 2] float64 between the forward call and the decision stage (ent_scope = supplied)."""
    acc = sequence_entropy_partials(piece_mean, piece_tokens, ids, num_seqs)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(acc)
    return sequence_entropy_from_partials(acc, ids)


def step_entropy_gate(call_mean_entropy: Sequence[float], call_tokens: Sequence[int], device=None) -> float:
    """The gate entropy of Eq. 10 read as the entropy of the model over one optimiser step: the
    token-weighted mean of the per-call mean entropies (the forward call's mean_entropy statistic) of all
    micro-batches of this rank and, when a process group is up, of all ranks.  Every call of the step then
    takes it for each of its sequences (ent_scope = supplied), so that micro-batching and sharding do not
    change which tokens are masked."""
    acc = torch.zeros(2, dtype=torch.float64, device=device)
    for m, n in zip(call_mean_entropy, call_tokens):
        acc[0] += float(m) * int(n)
        acc[1] += int(n)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(acc)
    return float(acc[0] / acc[1]) if float(acc[1]) > 0 else 0.0

"""Data-parallel host logic of the token-loss path: one process per GPU, whole sequences per rank.

Per-token quantities (log-prob, entropy, the mean entropy of a sequence, the mask and clip decisions,
dHidden) never cross ranks when sequences are not split.  What does: the normaliser N of Eq. 10 (the
global count of response tokens, known before the step), the head gradient d_W (summed), and the
scalar loss and counters (summed).  The collective is whatever backend torch.distributed was
initialised with (NCCL over NVLink on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import List, Optional, Sequence

import torch
import torch.distributed as dist


# ---------------------------------------------------------------------------------------------
# Launch: one process per GPU on this node.
# ---------------------------------------------------------------------------------------------

def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def launch_ranks(script: str, argv: Sequence[str], world_size: int, port: Optional[int] = None,
                 env: Optional[dict] = None) -> int:
    """Run `script argv...` as `world_size` ranks on this node (torch.distributed.run, rendezvous on
    127.0.0.1) and return the launcher's exit code.  The ranks read RANK / LOCAL_RANK / WORLD_SIZE /
    MASTER_* from their environment."""
    if world_size < 1:
        raise ValueError("world_size must be at least 1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world_size}",
           "--master-addr", "127.0.0.1", "--master-port", str(port or free_port()), script, *argv]
    return subprocess.run(cmd, env=dict(os.environ, **(env or {}))).returncode


def world_from_env(expected: int) -> tuple:
    """(world size, rank, local rank) from the launcher's environment, or None when this process was not
    started by a launcher; raises if the launcher's world size is not the one asked for."""
    if "WORLD_SIZE" not in os.environ:
        return None
    world = int(os.environ["WORLD_SIZE"])
    if world != expected:
        raise RuntimeError(f"launched with WORLD_SIZE={world} but {expected} ranks were asked for")
    return world, int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0"))


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


class SlabAllReduce:
    """Sum of d_W over ranks, slab by slab, under the tail of the backward.  An instance is passed as the
    slab callback of the backward call (ulorl_token_loss_bwd_slabs): each time the launches that make rows
    [first_row, first_row + rows) of d_W final have been queued it starts an asynchronous all-reduce of
    those rows.  The collective orders itself behind the work queued so far on the current stream and runs
    on the backend's own stream, so the kernels queued afterwards (the next slab, d_hidden) overlap with
    it; finish() makes the current stream wait for every slab.  The result equals one all-reduce of the
    whole array: every element is summed over the same ranks either way."""

    def __init__(self, d_W: torch.Tensor, group=None):
        self.d_W = d_W
        self.group = group
        self.works = []
        self.slabs = []
        self.active = dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1

    def __call__(self, first_row: int, rows: int):
        self.slabs.append((first_row, rows))
        if self.active and rows > 0:
            self.works.append(dist.all_reduce(self.d_W[first_row:first_row + rows], group=self.group, async_op=True))

    def finish(self):
        for w in self.works:
            w.wait()
        self.works = []
        covered = sorted(self.slabs)
        self.slabs = []
        return covered


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


def all_reduce_sequence_entropy(table: torch.Tensor) -> torch.Tensor:
    """Sum, in place and over all ranks, the int64 [num_seqs, 2] tables (entropy sum in units of 2^-34 nats,
    token count) that ulorl_sequence_entropy_partials fills from each rank's pieces.  Integer addition is
    exact, so every rank ends with the sums of the unsplit batch bit for bit; the means are then taken on the
    device by ulorl_sequence_entropy_combine and go to the decision stage as ent_scope = supplied.  This is
    the one exchange between the forward call and the decision stage that token-range sharding adds.

    The same tables serve the gate of Eq. 10 read as the entropy of the model over one optimiser step: add the
    tables of the step's micro-batches (integer addition, any order), all-reduce them here, and the batch mean
    that ulorl_sequence_entropy_combine returns is the token mean entropy of the whole step on every rank; each
    call of the step then takes it for all of its sequences (ent_scope = supplied), so that micro-batching and
    sharding do not change which tokens are masked."""
    if table.dtype != torch.int64:
        raise TypeError("the table of per-sequence entropy sums is int64")
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(table)
    return table

"""Host-side bookkeeping of RL training with segment rollouts (Algorithm 1), the step just upstream of
the token-loss kernels.

A response of up to `global_max_seq_len` tokens is decoded in at most `max_segment_count` segments of
`each_segment_length` tokens, one segment per training step.  After each rollout a sample either
  * hit end-of-sequence: it is complete and goes to the experience pool;
  * filled its segment without reaching the global maximum: it waits in the unfinished pool and is
    continued in the next step, by the policy version of that step;
  * reached the global maximum: it is truncated and goes to the experience pool (Section 3.5 scores
    such samples as incorrect).
Every token remembers the policy version that generated its segment and the log-prob that version
gave it (the map f and the denominators of Eq. 8).  `pack_experience` lays finished samples out as
the packed arrays the kernels take.

The rollout engine itself is outside this library: `rollout_fn(samples, max_len, version)` is the
caller's; it returns, per sample, the new tokens, their log-probs and whether EOS was produced.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Sequence, Tuple

import numpy as np


@dataclass
class Sample:
    prompt_id: int
    response_id: int                      # index of the response inside its prompt's group
    tokens: List[int] = field(default_factory=list)
    old_logp: List[float] = field(default_factory=list)
    segment_version: List[int] = field(default_factory=list)
    n_segments: int = 0
    finished: bool = False                # EOS seen
    truncated: bool = False               # global maximum reached without EOS

    def __len__(self) -> int:
        return len(self.tokens)


RolloutFn = Callable[[Sequence[Sample], int, int], Sequence[Tuple[Sequence[int], Sequence[float], bool]]]


class SegmentRollout:
    """The pools and the per-step update of Algorithm 1."""

    def __init__(self, global_max_seq_len: int, max_segment_count: int):
        if global_max_seq_len <= 0 or max_segment_count <= 0 or global_max_seq_len % max_segment_count:
            raise ValueError("global_max_seq_len must be a positive multiple of max_segment_count")
        self.global_max_seq_len = global_max_seq_len
        self.max_segment_count = max_segment_count
        self.each_segment_length = global_max_seq_len // max_segment_count
        self.unfinished_pool: List[Sample] = []
        self.experience_pool: List[Sample] = []

    def step(self, rollout_fn: RolloutFn, new_prompts: Sequence[int], samples_per_prompt: int, version: int):
        """One iteration of the loop of Algorithm 1 up to (not including) update_model: roll out the
        unfinished samples and `samples_per_prompt` fresh samples per new prompt for one segment with
        the policy `version`, then update both pools.  Returns the samples that were rolled out."""
        batch: List[Sample] = list(self.unfinished_pool)
        for pid in new_prompts:
            batch.extend(Sample(prompt_id=pid, response_id=j) for j in range(samples_per_prompt))
        results = rollout_fn(batch, self.each_segment_length, version)
        if len(results) != len(batch):
            raise ValueError("rollout_fn must return one result per sample")
        self.unfinished_pool = []
        for s, (toks, logps, eos) in zip(batch, results):
            room = min(self.each_segment_length, self.global_max_seq_len - len(s))
            if len(toks) != len(logps) or len(toks) > room:
                raise ValueError("rollout_fn returned more tokens than the segment allows")
            s.tokens.extend(int(t) for t in toks)
            s.old_logp.extend(float(x) for x in logps)
            s.segment_version.extend([version] * len(toks))
            s.n_segments += 1
            if eos:                                           # condition 1: complete
                s.finished = True
                self.experience_pool.append(s)
            elif len(s) >= self.global_max_seq_len:           # condition 3: truncated at the global maximum
                s.truncated = True
                self.experience_pool.append(s)
            else:                                             # condition 2: continue next step
                self.unfinished_pool.append(s)
        return batch

    def take_experience(self) -> List[Sample]:
        """Hand the experience pool to the model update and empty it."""
        out, self.experience_pool = self.experience_pool, []
        return out


def pack_experience(samples: Sequence[Sample], advantages: Sequence[float]):
    """Packed arrays for ulorl_token_loss_fwd/bwd from finished samples: targets and old_logp [T],
    segment_version [T], seq_offsets [S + 1], advantages [S], and the id of the latest policy.
    Samples without tokens are skipped (they contribute no token)."""
    keep = [i for i, s in enumerate(samples) if len(s) > 0]
    lengths = np.array([len(samples[i]) for i in keep], dtype=np.int64)
    seq_offsets = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    cat = lambda name, dt: (np.concatenate([np.asarray(getattr(samples[i], name), dtype=dt) for i in keep])
                            if keep else np.zeros(0, dtype=dt))
    targets = cat("tokens", np.int32)
    old_logp = cat("old_logp", np.float32)
    version = cat("segment_version", np.int32)
    adv = np.asarray([advantages[i] for i in keep], dtype=np.float32)
    current_version = int(version.max()) if version.size else 0
    return dict(targets=targets, old_logp=old_logp, segment_version=version, seq_offsets=seq_offsets,
                advantages=adv, current_version=current_version)


def balance_into_calls(lengths: Sequence[int], max_tokens_per_call: int) -> List[List[int]]:
    """Split finished samples into calls of at most `max_tokens_per_call` tokens each, whole samples only,
    with near-equal token counts: the long-tailed length mix of ultra-long rollouts otherwise leaves one
    call (or one data-parallel rank) holding the few longest samples.  The number of calls is the least
    that the capacity allows for a first-fit-decreasing packing; samples are then dealt longest first to
    the lightest call that still has room.  Returns the sample indices of each call, each list ascending.
    A sample longer than the capacity is an error."""
    order = sorted(range(len(lengths)), key=lambda i: (-int(lengths[i]), i))
    if any(int(lengths[i]) > max_tokens_per_call for i in order):
        raise ValueError("a sample is longer than max_tokens_per_call")
    bins: List[int] = []                                   # first-fit decreasing fixes the number of calls
    for i in order:
        for b in range(len(bins)):
            if bins[b] + int(lengths[i]) <= max_tokens_per_call:
                bins[b] += int(lengths[i])
                break
        else:
            bins.append(int(lengths[i]))
    n_calls = len(bins)
    while True:
        load = [0] * n_calls
        calls: List[List[int]] = [[] for _ in range(n_calls)]
        ok = True
        for i in order:
            fits = [b for b in range(n_calls) if load[b] + int(lengths[i]) <= max_tokens_per_call]
            if not fits:
                ok = False
                break
            b = min(fits, key=lambda c: (load[c], c))
            load[b] += int(lengths[i])
            calls[b].append(i)
        if ok:
            return [sorted(c) for c in calls]
        n_calls += 1                                       # balancing can need one call more than first-fit

"""Shared helpers of the test-suite: build parameter objects for both sides from a workload,
run the oracle on a batch, and the comparison metrics."""
from __future__ import annotations

import numpy as np

from oracle import ulorl_oracle as O
from workloads import synth
from paper_2507_19766_b200.binding import Params

# tolerances of the parity contract
TOL_LOGP = 2e-3       # abs, per-token log-prob and entropy
TOL_LOSS = 1e-3       # rel
TOL_GRAD = 1e-2       # rel L2


def both_params(batch: synth.Batch, **over):
    wl = batch.workload
    kw = dict(is_mode=wl.is_mode, mpt_mode=wl.mpt_mode, ent_scope="per_seq", clip_eps_low=wl.clip_eps_low,
              clip_eps_high=wl.clip_eps_high, mpt_tau=wl.mpt_tau, entropy_target=wl.entropy_target,
              inv_temperature=1.0, norm_tokens=0, current_version=batch.current_version, loss_norm="tokens", norm_seqs=0,
              kl_beta=0.0)
    extra = {k: over.pop(k) for k in list(over) if k in ("kernel_path", "bwd_panel_tokens", "dw_accumulate",
                                                         "adv_per_token", "compact_rows")}
    kw.update(over)
    gp = Params(T=wl.T, H=wl.H, V=wl.V, num_seqs=wl.S, dtype=wl.dtype, **kw, **extra)
    op = O.OracleParams(**kw)
    return gp, op


def oracle_inputs(batch: synth.Batch):
    return dict(hidden=batch.host_f32("hidden"), W=batch.host_f32("W"), targets=batch.targets.numpy(),
                old_logp=batch.old_logp.numpy(), segment_version=batch.segment_version.numpy(),
                advantages=batch.advantages.numpy(), seq_offsets=batch.seq_offsets.numpy())


def rel_l2(a, b) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def near_threshold(logp64, old_logp, seq_entropy64, seq_offsets, op: O.OracleParams, margin=TOL_LOGP):
    """Tokens whose decision could flip under a log-prob / entropy error of `margin`."""
    ln_tau, ln_hi, ln_lo = O.decision_thresholds(op)
    d = logp64 - old_logp.astype(np.float64)
    near = np.abs(logp64 - float(ln_tau)) <= margin
    if op.is_mode == "sais":
        near |= np.abs(d - float(ln_hi)) <= margin
        near |= np.abs(d - float(ln_lo)) <= margin
    if op.mpt_mode == "dynamic":
        lens = np.diff(seq_offsets)
        seq_near = np.abs(np.asarray(seq_entropy64) - float(np.float32(op.entropy_target))) <= margin
        near |= np.repeat(seq_near, lens)
    return near

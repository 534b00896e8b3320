"""fp64 CPU oracle for the UloRL per-token policy-update path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain restatement of what the
fused GPU path must compute.  It shares no code with the CUDA library or its Python
binding and imports neither; nothing but the test-suite, the smoke check and the
CPU-baseline leg of the benchmark may import it.

Everything is NumPy in float64.  One chunk of token rows is handled at a time and its
full row of V logits is materialised, so every step can be checked against the paper
by eye:

  step 1  logits                z = kappa * hidden @ W^T              (policy of Eq. 6)
  step 2  log-softmax, entropy  logp = z_y - lse ; Hent = -sum p ln p (Eq. 6, Eq. 10 H-bar)
  (Eq. 4  group-normalised advantages and the dynamic-sampling filter of Eq. 7: group_advantages)
  step 3  mean entropy          H-bar_i = mean over the sequence       (Eq. 10)
  step 4  MPT mask              Eq. 9 and the indicator of Eq. 10
  step 5  importance ratio      SAIS (Eq. 8) or POIS (Section 3.1.2)
  step 6  clipped surrogate     token-normalised objective of Eq. 10 / Eq. 7
  step 7  d loss / d logp       derivative of step 6
  step 8  dHidden, dW           chain rule through steps 1-2

Readings taken where the paper is silent or garbled (each is also listed in the design
notes of the repository):
  * H-bar is printed as +sum p log p; entropy is taken as -sum p ln p >= 0 (nats).
  * "positive sample" (reward 1) is read as advantage > 0 (Section 3.3).
  * p(t) in Eq. 9 is the current policy's probability of the token.
  * the normaliser counts every response token, masked or not (Eq. 10).
  * clipping kills the gradient only on strict violation of the bound.
  * POIS: ratio == 1 in value with unit derivative w.r.t. logp; old log-probs unread.

Decision stage.  Mask and clip decisions are integers decided by floating point, so they
are taken in float32 on float32 inputs with no transcendental inside the comparison:
logp32 >= LN_TAU, d32 = logp32 - old_logp (one IEEE float32 subtraction), d32 > LN_HI,
d32 < LN_LO, Hbar32 < sigma, with LN_* = float32(log / log1p evaluated in float64).
Values (ratio, surrogate, loss, gradient coefficient) are then float64 functions of d32.

Pins (tests/test_oracle_*.py): softmax sums to one, zero hidden state gives logp = -ln V
and entropy = ln V, binary-entropy closed form, SciPy's log_softmax on small shapes,
a hand-expanded T=3,V=4,H=2 case in scalar Python, the four clip quadrants, mask
invariants, mean-NLL special case, column sums of dW, central finite differences.
The paper prints no numeric value for any quantity on this path, so no pin is a value
quoted from the paper.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np

# flag bits written per token by the decision stage
FLAG_MASKED = 1      # MPT and gate open: excluded from the objective (Eq. 10 indicator)
FLAG_CLIP_HIGH = 2   # A > 0 and ratio above 1 + eps_high
FLAG_CLIP_LOW = 4    # A < 0 and ratio below 1 - eps_low
FLAG_MPT = 8         # token is an MPT (Eq. 9), whatever the gate says

N_STALENESS = 16     # staleness buckets in the statistics


@dataclass
class OracleParams:
    is_mode: str = "sais"            # "sais" (Eq. 8) | "pois" (Section 3.1.2)
    mpt_mode: str = "dynamic"        # "off" | "always" | "dynamic" (Eq. 10)
    ent_scope: str = "per_seq"       # "per_seq" | "batch" | "supplied"
    clip_eps_low: float = 0.2
    clip_eps_high: float = 0.2
    mpt_tau: float = 0.99            # Section 4.1
    entropy_target: float = 0.2      # sigma, Section 4.1
    inv_temperature: float = 1.0     # kappa
    norm_tokens: int = 0             # N of Eq. 10; 0 means the T tokens of the call
    loss_norm: str = "tokens"        # "tokens": 1 / sum_i |o_i| (Eq. 7, Eq. 10) | "sequence": (1/G) sum_i 1/|o_i| (Eq. 5)
    norm_seqs: int = 0               # G of Eq. 5 in "sequence" mode; 0 means the sequences of the call
    current_version: int = 0
    kl_beta: float = 0.0             # beta of Eq. 5's KL-to-reference term; 0 = none (the paper's method, Section 2.3)


def _f64(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x), dtype=np.float64)


# --------------------------------------------------------------------------- steps 1-2
def logits_rows(hidden, W, rows, kappa: float = 1.0) -> np.ndarray:
    """Step 1: z[t, v] = kappa * sum_h hidden[t, h] * W[v, h] for the given rows (Eq. 6)."""
    hidden = np.asarray(hidden)
    h = _f64(hidden[rows])
    return float(kappa) * (h @ _f64(W).T)


def token_stats(hidden, W, targets, kappa: float = 1.0, rows=None, chunk: int = 256):
    """Steps 1-2 for every row (or the rows listed): log-prob of the target token,
    entropy of the row's softmax, and the row's log-sum-exp, all float64.

    p_v = exp(z_v - lse);  logp = z_y - lse  (Eq. 6);  Hent = -sum_v p_v ln p_v  (Eq. 10).
    """
    hidden = np.asarray(hidden)
    targets = np.asarray(targets)
    T = hidden.shape[0]
    rows = np.arange(T) if rows is None else np.asarray(rows, dtype=np.int64)
    W64 = _f64(W)
    n = rows.shape[0]
    logp = np.empty(n)
    ent = np.empty(n)
    lse = np.empty(n)
    for a in range(0, n, chunk):
        r = rows[a:a + chunk]
        z = float(kappa) * (_f64(hidden[r]) @ W64.T)
        m = z.max(axis=1)
        lse_c = m + np.log(np.exp(z - m[:, None]).sum(axis=1))
        lnp = z - lse_c[:, None]
        p = np.exp(lnp)
        logp[a:a + chunk] = lnp[np.arange(r.shape[0]), targets[r]]
        ent[a:a + chunk] = -(p * lnp).sum(axis=1)
        lse[a:a + chunk] = lse_c
    return logp, ent, lse


# --------------------------------------------------------------------------- upstream of step 4: Eq. 4
def group_advantages(rewards, group_size: int):
    """Eq. 4: A_i = (R_i - mean(group)) / std(group) over each group of `group_size` consecutive
    responses to one prompt, and the dynamic-sampling constraint of Eq. 7: a group is kept only if
    0 < #(reward == 1) < G.  Readings: std is the population standard deviation (the paper does not
    say which); a group with zero spread gets advantage 0 (it is dropped by the constraint anyway)."""
    r = _f64(rewards)
    S = r.shape[0]
    adv = np.zeros(S)
    keep = np.zeros(S, dtype=np.uint8)
    for a in range(0, S, group_size):
        grp = r[a:a + group_size]
        G = grp.shape[0]
        mean = 0.0
        for x in grp:
            mean += x
        mean /= G
        var = 0.0
        for x in grp:
            var += (x - mean) * (x - mean)
        std = (var / G) ** 0.5
        n_correct = int(np.count_nonzero(grp == 1.0))
        kept = 0 < n_correct < G
        for j in range(G):
            adv[a + j] = (grp[j] - mean) / std if std > 0 else 0.0
            keep[a + j] = 1 if kept else 0
    return adv, keep


# --------------------------------------------------------------------------- step 3
def sequence_mean_entropy(entropy32, seq_offsets):
    """Step 3: H-bar_i = (1/|o_i|) sum_t Hent_t over the tokens of sequence i, and the
    token-weighted batch mean (Eq. 10).  Input is the float32 per-token entropy; sums
    run in float64 in token order."""
    e = _f64(np.asarray(entropy32, dtype=np.float32))
    off = np.asarray(seq_offsets, dtype=np.int64)
    S = off.shape[0] - 1
    seq_mean = np.zeros(S)
    for i in range(S):
        a, b = int(off[i]), int(off[i + 1])
        if b > a:
            tot = 0.0
            for x in e[a:b]:
                tot += x
            seq_mean[i] = tot / (b - a)
    total = 0.0
    for x in e:
        total += x
    batch_mean = total / max(1, e.shape[0])
    return seq_mean, batch_mean


def gate_entropy(entropy32, seq_offsets, scope: str, supplied=None) -> np.ndarray:
    """The float32 entropy value that sequence i is gated on: its own mean, the batch
    mean, or a caller-supplied value (one per sequence)."""
    S = len(seq_offsets) - 1
    if scope == "supplied":
        return np.asarray(supplied, dtype=np.float32).reshape(S).copy()
    seq_mean, batch_mean = sequence_mean_entropy(entropy32, seq_offsets)
    if scope == "per_seq":
        return seq_mean.astype(np.float32)
    if scope == "batch":
        return np.full(S, np.float32(batch_mean), dtype=np.float32)
    raise ValueError(scope)


# --------------------------------------------------------------------------- steps 4-7
def decision_thresholds(p: OracleParams):
    """float32 thresholds of the decision stage, each from a float64 evaluation of the
    float32 parameter."""
    tau = np.float64(np.float32(p.mpt_tau))
    hi = np.float64(np.float32(p.clip_eps_high))
    lo = np.float64(np.float32(p.clip_eps_low))
    with np.errstate(divide="ignore", invalid="ignore"):
        ln_tau = np.float32(np.log(tau))
        ln_hi = np.float32(np.log1p(hi))
        ln_lo = np.float32(np.log1p(-lo)) if lo < 1.0 else np.float32(-np.inf)
    return ln_tau, ln_hi, ln_lo


def kl_estimate(ref_minus_logp):
    """Per-token estimate of D_KL[pi_theta || pi_ref] in Eq. 5 from the one generated token:
    with u = ln pi_ref(o_t) - ln pi_theta(o_t), k = e^u - u - 1.  It is non-negative, zero iff the two
    log-probs agree, and its mean under o_t ~ pi_theta is the KL divergence (E[e^u] = 1, E[-u] = KL).
    The paper prints the divergence without an estimator; this is the one of the work Eq. 5 is
    quoted from."""
    u = np.asarray(ref_minus_logp, dtype=np.float64)
    return np.exp(u) - u - 1.0


def decide(logp32, gate_ent32, old_logp, advantages, seq_offsets, segment_version,
           p: OracleParams, adv_per_token: bool = False, ref_logp=None):
    """Steps 4-7 on float32 log-probs: mask, ratio, clipped surrogate, loss, d loss/d logp.
    With p.kl_beta > 0 the token term of Eq. 5 is s_t - beta k_t (k_t = kl_estimate of the token,
    ref_logp the reference policy's recorded log-prob), inside the mask like the surrogate.

    Returns a dict with flags (uint8[T]), ratio, surrogate, grad_coef (float64[T]),
    loss (float64) and the statistics.
    """
    logp32 = np.asarray(logp32, dtype=np.float32)
    T = logp32.shape[0]
    off = np.asarray(seq_offsets, dtype=np.int64)
    S = off.shape[0] - 1
    gate_ent32 = np.asarray(gate_ent32, dtype=np.float32)
    adv_in = np.asarray(advantages, dtype=np.float32)
    ln_tau, ln_hi, ln_lo = decision_thresholds(p)
    sigma32 = np.float32(p.entropy_target)
    if p.loss_norm == "tokens":      # one weight 1/N for every token (Eq. 10)
        N = float(p.norm_tokens) if p.norm_tokens > 0 else float(T)
    else:                            # GRPO's per-sample mean (Eq. 5): token of sequence i weighs 1 / (G |o_i|)
        N = float(p.norm_seqs) if p.norm_seqs > 0 else float(S)
    eps_hi = float(np.float32(p.clip_eps_high))
    eps_lo = float(np.float32(p.clip_eps_low))

    beta = float(np.float32(p.kl_beta))
    if beta > 0.0 and ref_logp is None:
        raise ValueError("kl_beta > 0 needs ref_logp")
    flags = np.zeros(T, dtype=np.uint8)
    ratio = np.ones(T)
    surrogate = np.zeros(T)
    grad_coef = np.zeros(T)
    d_abs = np.zeros(T)
    kl = np.zeros(T)
    loss_sum = 0.0
    for i in range(S):
        if p.mpt_mode == "always":
            gate = True
        elif p.mpt_mode == "dynamic":
            gate = bool(gate_ent32[i] < sigma32)          # strict, as printed in Eq. 10
        else:
            gate = False
        wlen = 1.0 if p.loss_norm == "tokens" else 1.0 / max(1.0, float(off[i + 1] - off[i]))
        for t in range(int(off[i]), int(off[i + 1])):
            A32 = adv_in[t] if adv_per_token else adv_in[i]
            A = float(A32)
            # step 4 (Eq. 9): positive sample and probability at least tau
            mpt = bool(A32 > 0) and bool(logp32[t] >= ln_tau)
            msk = mpt and gate
            # step 5: ratio
            if p.is_mode == "sais":                      # Eq. 8
                d32 = np.float32(logp32[t] - np.float32(old_logp[t]))
                r = float(np.exp(np.float64(d32)))
                hi = bool(A32 > 0) and bool(d32 > ln_hi)
                lo = bool(A32 < 0) and bool(d32 < ln_lo)
                d_abs[t] = abs(float(d32))
            else:                                        # POIS: ratio identically one
                r, hi, lo = 1.0, False, False
            # step 6 (Eq. 10): min(r A, clip(r, 1-eps, 1+eps) A)
            c = min(max(r, 1.0 - eps_lo), 1.0 + eps_hi)
            s = min(r * A, c * A)
            keep = 0.0 if msk else 1.0
            # Eq. 5's KL term, when asked for: objective s - beta k, d k / d logp = 1 - e^u
            dk = 0.0
            if beta > 0.0:
                u = float(np.float64(np.float32(ref_logp[t])) - np.float64(logp32[t]))
                kl[t] = float(kl_estimate(u))
                dk = 1.0 - float(np.exp(u))
            loss_sum += keep * (s - beta * kl[t]) * wlen
            # step 7
            g = -(1.0 / N) * keep * (A * r * (0.0 if (hi or lo) else 1.0) - beta * dk) * wlen + 0.0   # + 0.0: no -0
            f = 0
            if msk:
                f |= FLAG_MASKED
            if hi:
                f |= FLAG_CLIP_HIGH
            if lo:
                f |= FLAG_CLIP_LOW
            if mpt:
                f |= FLAG_MPT
            flags[t] = f
            ratio[t] = r
            surrogate[t] = s
            grad_coef[t] = g
    loss = -loss_sum / N

    sv = np.asarray(segment_version, dtype=np.int64) if segment_version is not None \
        else np.full(T, p.current_version, dtype=np.int64)
    stale = np.clip(p.current_version - sv, 0, N_STALENESS - 1)
    clipped = (flags & (FLAG_CLIP_HIGH | FLAG_CLIP_LOW)) != 0
    stale_tokens = np.bincount(stale, minlength=N_STALENESS)
    stale_clipped = np.bincount(stale, weights=clipped, minlength=N_STALENESS).astype(np.int64)
    stale_abs = np.bincount(stale, weights=d_abs, minlength=N_STALENESS)
    stats = dict(
        n_tokens=T,
        n_active=int(np.count_nonzero(grad_coef)),
        n_mpt=int(np.count_nonzero(flags & FLAG_MPT)),
        n_masked=int(np.count_nonzero(flags & FLAG_MASKED)),
        n_clip_high=int(np.count_nonzero(flags & FLAG_CLIP_HIGH)),
        n_clip_low=int(np.count_nonzero(flags & FLAG_CLIP_LOW)),
        stale_tokens=stale_tokens.astype(np.int64),
        stale_clipped=stale_clipped,
        stale_mean_abs_logratio=np.where(stale_tokens > 0, stale_abs / np.maximum(stale_tokens, 1), 0.0),
        mean_kl=float(kl.mean()) if T > 0 else 0.0,
    )
    return dict(flags=flags, ratio=ratio, surrogate=surrogate, grad_coef=grad_coef, kl=kl,
                loss=loss, stats=stats)


# --------------------------------------------------------------------------- step 8
def backward(hidden, W, targets, grad_coef, kappa: float = 1.0, rows=None,
             grad_loss: float = 1.0, chunk: int = 256, want_dW: bool = True):
    """Step 8: dz[t, v] = kappa * g_t * (1[v = y_t] - p[t, v]);
    dHidden[t, :] = sum_v dz[t, v] W[v, :];  dW[v, :] = sum_t dz[t, v] hidden[t, :].

    grad_coef is indexed by token (length T).  With rows given, only those rows are
    processed: dHidden has one line per listed row and dW sums over the listed rows.
    """
    hidden = np.asarray(hidden)
    targets = np.asarray(targets)
    T, H = hidden.shape
    rows = np.arange(T) if rows is None else np.asarray(rows, dtype=np.int64)
    W64 = _f64(W)
    V = W64.shape[0]
    g = _f64(grad_coef)
    dH = np.zeros((rows.shape[0], H))
    dW = np.zeros((V, H)) if want_dW else None
    for a in range(0, rows.shape[0], chunk):
        r = rows[a:a + chunk]
        h = _f64(hidden[r])
        z = float(kappa) * (h @ W64.T)
        m = z.max(axis=1)
        lse = m + np.log(np.exp(z - m[:, None]).sum(axis=1))
        dz = -np.exp(z - lse[:, None])
        dz[np.arange(r.shape[0]), targets[r]] += 1.0
        dz *= (float(kappa) * float(grad_loss) * g[r])[:, None]
        dH[a:a + chunk] = dz @ W64
        if want_dW:
            dW += dz.T @ h
    return dH, dW


# --------------------------------------------------------------------------- composition
def forward(hidden, W, targets, old_logp, segment_version, advantages, seq_offsets,
            p: OracleParams, adv_per_token: bool = False, entropy_supplied=None,
            rows=None, chunk: int = 256, ref_logp=None):
    """Steps 1-7.  With rows=None every token is processed.  The decision stage takes the
    float32 rounding of the float64 log-prob and entropy."""
    logp, ent, lse = token_stats(hidden, W, targets, p.inv_temperature, rows=rows, chunk=chunk)
    out = dict(logp=logp, entropy=ent, lse=lse)
    if rows is not None:
        return out
    logp32 = logp.astype(np.float32)
    ent32 = ent.astype(np.float32)
    seq_mean, batch_mean = sequence_mean_entropy(ent32, seq_offsets)
    gate32 = gate_entropy(ent32, seq_offsets, p.ent_scope, entropy_supplied)
    dec = decide(logp32, gate32, old_logp, advantages, seq_offsets, segment_version, p,
                 adv_per_token=adv_per_token, ref_logp=ref_logp)
    out.update(dec)
    out.update(seq_entropy=seq_mean, mean_entropy=batch_mean, gate_entropy=gate32)
    return out


def fwd_bwd(hidden, W, targets, old_logp, segment_version, advantages, seq_offsets,
            p: OracleParams, adv_per_token: bool = False, entropy_supplied=None,
            grad_loss: float = 1.0, chunk: int = 256, ref_logp=None):
    """Steps 1-8 on the whole batch."""
    out = forward(hidden, W, targets, old_logp, segment_version, advantages, seq_offsets, p,
                  adv_per_token=adv_per_token, entropy_supplied=entropy_supplied, chunk=chunk, ref_logp=ref_logp)
    dH, dW = backward(hidden, W, targets, out["grad_coef"], p.inv_temperature,
                      grad_loss=grad_loss, chunk=chunk)
    out.update(d_hidden=dH, d_W=dW)
    return out


def objective_value(hidden, W, targets, old_logp, advantages, seq_offsets, masked,
                    p: OracleParams, adv_per_token: bool = False, ref_logp=None) -> float:
    """The negated objective of Eq. 10 as a smooth function of (hidden, W) with the mask
    held fixed (the indicator is not differentiated) and everything in float64: used by
    the finite-difference pins.  POIS is evaluated through its defining expression
    r = exp(logp - stopgrad(logp)); since its value is identically one, the finite
    difference of this function is taken in SAIS form with old = the unperturbed logp
    by the caller."""
    logp, _, _ = token_stats(hidden, W, targets, p.inv_temperature)
    T = logp.shape[0]
    off = np.asarray(seq_offsets, dtype=np.int64)
    adv_in = np.asarray(advantages, dtype=np.float64)
    N = float(p.norm_tokens) if p.norm_tokens > 0 else float(T)
    G = float(p.norm_seqs) if p.norm_seqs > 0 else float(off.shape[0] - 1)
    eps_hi = float(np.float32(p.clip_eps_high))
    eps_lo = float(np.float32(p.clip_eps_low))
    tot = 0.0
    per_sample = 0.0
    for i in range(off.shape[0] - 1):
        seq = 0.0
        for t in range(int(off[i]), int(off[i + 1])):
            A = float(adv_in[t] if adv_per_token else adv_in[i])
            r = float(np.exp(logp[t] - float(old_logp[t])))
            c = min(max(r, 1.0 - eps_lo), 1.0 + eps_hi)
            if not masked[t]:
                seq += min(r * A, c * A)
                if p.kl_beta > 0.0:      # Eq. 5: the token term is s - beta k
                    seq -= float(np.float32(p.kl_beta)) * float(kl_estimate(float(ref_logp[t]) - logp[t]))
        tot += seq
        if off[i + 1] > off[i]:
            per_sample += seq / float(off[i + 1] - off[i])
    if p.loss_norm == "sequence":    # Eq. 5: mean over the group of each sample's token mean
        return -per_sample / G
    return -tot / N

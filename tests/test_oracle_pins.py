"""Pins for the fp64 oracle: closed forms, invariants, a library second opinion, a scalar
brute force and finite differences.  None of the expected values comes from the oracle
itself or from the CUDA path."""
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import ulorl_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")


def golden(kind):
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            if parts[0] == kind:
                rows.append([float(x) for x in parts[1:]])
    assert rows
    return rows


def rand_problem(T, H, V, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    hidden = rng.standard_normal((T, H)).astype(np.float32)
    W = (scale * rng.standard_normal((V, H))).astype(np.float32)
    targets = rng.integers(0, V, size=T).astype(np.int32)
    return hidden, W, targets


# ------------------------------------------------------------------ softmax / log-prob
def test_softmax_sums_to_one():
    hidden, W, targets = rand_problem(37, 16, 301, 0)
    _, _, lse = O.token_stats(hidden, W, targets, kappa=0.7)
    z = O.logits_rows(hidden, W, np.arange(37), kappa=0.7)
    p = np.exp(z - lse[:, None])
    assert np.abs(p.sum(axis=1) - 1.0).max() < 1e-12


@pytest.mark.parametrize("row", golden("uniform"))
def test_uniform_row_closed_form(row):
    V, ln_v = int(row[0]), row[1]
    H = 8
    hidden = np.zeros((3, H), dtype=np.float32)
    W = np.random.default_rng(1).standard_normal((V, H)).astype(np.float32)
    targets = np.array([0, V // 2, V - 1], dtype=np.int32)
    logp, ent, lse = O.token_stats(hidden, W, targets)
    assert np.allclose(logp, -ln_v, rtol=0, atol=1e-12)
    assert np.allclose(ent, ln_v, rtol=0, atol=1e-11)
    assert np.allclose(lse, ln_v, rtol=0, atol=1e-12)


def test_binary_entropy_closed_form():
    ln_odds, p_small, ent_expected = golden("binary")[0]
    # H = 1: hidden = 1, W = [[0], [ln 3]]  => logits (0, ln 3)
    hidden = np.ones((2, 1), dtype=np.float64)
    W = np.array([[0.0], [ln_odds]])
    logp, ent, _ = O.token_stats(hidden, W, np.array([0, 1], dtype=np.int32))
    assert abs(math.exp(logp[0]) - p_small) < 1e-15
    assert abs(math.exp(logp[1]) - (1 - p_small)) < 1e-15
    assert np.allclose(ent, ent_expected, atol=1e-15)


def test_dominating_logit_limits():
    H, V = 4, 50
    W = np.zeros((V, H), dtype=np.float32)
    W[7, 0] = 60.0
    hidden = np.zeros((1, H), dtype=np.float32)
    hidden[0, 0] = 1.0
    logp, ent, _ = O.token_stats(hidden, W, np.array([7], dtype=np.int32))
    assert -1e-20 > logp[0] > -1e-22 * 1e4 or abs(logp[0]) < 1e-20
    assert 0.0 <= ent[0] < 1e-20


def test_shift_invariance():
    hidden, W, targets = rand_problem(9, 6, 40, 2)
    # an extra hidden feature equal to one with a constant weight column adds c to every logit
    h2 = np.concatenate([hidden, np.ones((9, 1), np.float32)], axis=1)
    W2 = np.concatenate([W, np.full((40, 1), 3.25, np.float32)], axis=1)
    a = O.token_stats(hidden, W, targets)
    b = O.token_stats(h2, W2, targets)
    assert np.allclose(a[0], b[0], atol=1e-12)
    assert np.allclose(a[1], b[1], atol=1e-12)
    assert np.allclose(a[2] + 3.25, b[2], atol=1e-12)


@pytest.mark.parametrize("shape", [(5, 3, 7), (11, 8, 8), (4, 8, 4)])
def test_against_scipy_log_softmax(shape):
    """Library second opinion; V == H and V < H shapes would expose a transposed operand."""
    T, H, V = shape
    hidden, W, targets = rand_problem(T, H, V, 3)
    kappa = 1.0 / 0.85
    z = kappa * np.einsum("th,vh->tv", hidden.astype(np.float64), W.astype(np.float64))
    ref_lnp = scipy.special.log_softmax(z, axis=1)
    ref_ent = scipy.stats.entropy(scipy.special.softmax(z, axis=1), axis=1)
    logp, ent, lse = O.token_stats(hidden, W, targets, kappa=kappa)
    assert np.allclose(logp, ref_lnp[np.arange(T), targets], atol=1e-12)
    assert np.allclose(ent, ref_ent, atol=1e-12)
    assert np.allclose(lse, scipy.special.logsumexp(z, axis=1), atol=1e-12)


def test_entropy_bounds_and_two_forms():
    hidden, W, targets = rand_problem(64, 12, 500, 4, scale=0.8)
    logp, ent, lse = O.token_stats(hidden, W, targets)
    assert (ent >= 0).all() and (ent <= math.log(500) + 1e-12).all()
    z = O.logits_rows(hidden, W, np.arange(64))
    p = np.exp(z - lse[:, None])
    assert np.allclose(ent, lse - (p * z).sum(axis=1), atol=1e-11)
    assert (logp <= 0).all()


def test_chunking_and_row_subset_agree():
    hidden, W, targets = rand_problem(50, 8, 90, 5)
    full = O.token_stats(hidden, W, targets, chunk=256)
    small = O.token_stats(hidden, W, targets, chunk=7)
    rows = np.array([3, 49, 0, 17])
    sub = O.token_stats(hidden, W, targets, rows=rows)
    for a, b, c in zip(full, small, sub):
        assert np.array_equal(a, b) or np.allclose(a, b, atol=1e-13)
        assert np.allclose(a[rows], c, atol=1e-13)


# ------------------------------------------------------------------ scalar brute force
def brute_force(hidden, W, targets, old_logp, adv, offsets, eps_lo, eps_hi, tau, sigma, mode,
                mpt_mode, kappa, N):
    """Everything by scalar Python loops straight from the equations (float64)."""
    T, H = len(hidden), len(hidden[0])
    V = len(W)
    logp, ent, P = [], [], []
    for t in range(T):
        z = [kappa * sum(hidden[t][h] * W[v][h] for h in range(H)) for v in range(V)]
        m = max(z)
        den = sum(math.exp(x - m) for x in z)
        p = [math.exp(x - m) / den for x in z]
        P.append(p)
        logp.append(math.log(p[targets[t]]))
        ent.append(-sum(q * math.log(q) for q in p))
    seq_of = []
    hbar = []
    for i in range(len(offsets) - 1):
        toks = range(offsets[i], offsets[i + 1])
        hbar.append(sum(ent[t] for t in toks) / len(toks))
        seq_of += [i] * len(toks)
    loss, g, msk_all = 0.0, [], []
    for t in range(T):
        A = adv[seq_of[t]]
        mpt = A > 0 and math.exp(logp[t]) >= tau
        gate = mpt_mode == "always" or (mpt_mode == "dynamic" and hbar[seq_of[t]] < sigma)
        msk = mpt and gate
        r = math.exp(logp[t] - old_logp[t]) if mode == "sais" else 1.0
        c = min(max(r, 1 - eps_lo), 1 + eps_hi)
        s = min(r * A, c * A)
        if not msk:
            loss -= s / N
        clipped = (A > 0 and r > 1 + eps_hi) or (A < 0 and r < 1 - eps_lo)
        if mode != "sais":
            clipped = False
        g.append(0.0 if (msk or clipped) else -A * r / N)
        msk_all.append(msk)
    dH = [[0.0] * H for _ in range(T)]
    dW = [[0.0] * H for _ in range(V)]
    for t in range(T):
        for v in range(V):
            dz = kappa * g[t] * ((1.0 if v == targets[t] else 0.0) - P[t][v])
            for h in range(H):
                dH[t][h] += dz * W[v][h]
                dW[v][h] += dz * hidden[t][h]
    return logp, ent, hbar, loss, g, msk_all, dH, dW


@pytest.mark.parametrize("mode,mpt_mode", [("sais", "always"), ("sais", "dynamic"),
                                            ("pois", "always"), ("sais", "off")])
def test_brute_force_T3_V4_H2(mode, mpt_mode):
    # values exactly representable in float32 so that storage rounding plays no part
    hidden = [[1.0, -0.5], [4.0, 4.0], [0.25, 2.0]]
    W = [[0.5, -1.0], [2.0, 2.0], [-1.5, 0.75], [0.0, 1.0]]
    targets = [2, 1, 3]
    old_logp = [-1.0, -0.25, -0.5]
    adv = [1.0, -1.0]
    offsets = [0, 2, 3]
    kappa, N = 0.5, 5
    eps_lo, eps_hi = float(np.float32(0.2)), float(np.float32(0.2))
    tau = float(np.float32(0.99))
    bf = brute_force(hidden, W, targets, old_logp, adv, offsets, eps_lo, eps_hi, tau,
                     float(np.float32(0.35)), mode, mpt_mode, kappa, N)
    p = O.OracleParams(is_mode=mode, mpt_mode=mpt_mode, mpt_tau=0.99, entropy_target=0.35,
                       inv_temperature=kappa, norm_tokens=N)
    out = O.fwd_bwd(np.array(hidden, np.float32), np.array(W, np.float32),
                    np.array(targets, np.int32), np.array(old_logp, np.float32),
                    np.zeros(3, np.int32), np.array(adv, np.float32),
                    np.array(offsets, np.int32), p)
    assert np.allclose(out["logp"], bf[0], atol=1e-12)
    assert np.allclose(out["entropy"], bf[1], atol=1e-12)
    assert np.allclose(out["seq_entropy"], bf[2], atol=1e-7)       # float32 entropies enter the mean
    assert np.array_equal((out["flags"] & O.FLAG_MASKED) != 0, np.array(bf[5]))
    # token 1 (hidden (4,4), target 1) has probability above tau in a positive sequence
    assert bf[5][1] == (mpt_mode == "always" or (mpt_mode == "dynamic" and bf[2][0] < 0.35))
    assert abs(out["loss"] - bf[3]) < 1e-6
    assert np.allclose(out["grad_coef"], bf[4], rtol=1e-6, atol=1e-9)
    g_scale = np.array(out["grad_coef"]) / np.where(np.array(bf[4]) == 0, 1, np.array(bf[4]))
    g_scale = np.where(np.array(bf[4]) == 0, 1.0, g_scale)
    assert np.allclose(out["d_hidden"], np.array(bf[6]) * g_scale[:, None], atol=1e-12)
    assert np.allclose(out["d_W"], bf[7], rtol=1e-6, atol=1e-9)


# ------------------------------------------------------------------ ratio / clip / mask
def one_token_decide(r, A, **kw):
    """A single token whose ratio is r: logp32 = 0 - something, old = logp - ln r."""
    logp = np.float32(-1.0)
    old = np.float32(logp - np.float32(math.log(r)))
    p = O.OracleParams(is_mode="sais", mpt_mode="off", norm_tokens=1, **kw)
    return O.decide(np.array([logp]), np.array([1.0], np.float32), np.array([old]),
                    np.array([A], np.float32), np.array([0, 1]), np.zeros(1, np.int32), p)


@pytest.mark.parametrize("row", golden("clip"))
def test_clip_quadrants(row):
    r, A, s_expected, active = row
    out = one_token_decide(r, A)
    assert abs(out["surrogate"][0] - s_expected) < 2e-7
    assert abs(out["loss"] + s_expected) < 2e-7
    assert (out["grad_coef"][0] != 0.0) == bool(active)
    if active:
        assert abs(out["grad_coef"][0] + A * r) < 2e-7
    hi = bool(out["flags"][0] & O.FLAG_CLIP_HIGH)
    lo = bool(out["flags"][0] & O.FLAG_CLIP_LOW)
    assert hi == (A > 0 and r > 1.2 + 1e-6) and lo == (A < 0 and r < 0.8 - 1e-6)


def test_asymmetric_clip_bounds():
    out = one_token_decide(1.25, 1.0, clip_eps_low=0.2, clip_eps_high=0.28)
    assert out["grad_coef"][0] != 0.0 and abs(out["surrogate"][0] - 1.25) < 2e-7
    out = one_token_decide(1.3, 1.0, clip_eps_low=0.2, clip_eps_high=0.28)
    assert out["grad_coef"][0] == 0.0 and abs(out["surrogate"][0] - 1.28) < 2e-7
    out = one_token_decide(0.85, -1.0, clip_eps_low=0.1, clip_eps_high=0.28)
    assert out["grad_coef"][0] == 0.0 and abs(out["surrogate"][0] + 0.9) < 2e-7


def small_batch(seed=7, T=40, H=6, V=30, S=4):
    hidden, W, targets = rand_problem(T, H, V, seed, scale=1.5)
    offsets = np.array([0, 7, 19, 20, T], dtype=np.int32)[: S + 1]
    offsets[-1] = T
    adv = np.array([1.0, -1.0, 0.5, -2.0], dtype=np.float32)[:S]
    version = np.zeros(T, np.int32)
    return hidden, W, targets, offsets, adv, version


def test_ratio_one_when_old_equals_current_and_pois_equivalence():
    hidden, W, targets, offsets, adv, version = small_batch()
    logp, _, _ = O.token_stats(hidden, W, targets)
    old = logp.astype(np.float32)
    ps = O.OracleParams(is_mode="sais", mpt_mode="off")
    pp = O.OracleParams(is_mode="pois", mpt_mode="off")
    a = O.fwd_bwd(hidden, W, targets, old, version, adv, offsets, ps)
    b = O.fwd_bwd(hidden, W, targets, np.full_like(old, 123.0), version, adv, offsets, pp)
    assert np.array_equal(a["ratio"], np.ones(40))
    assert a["stats"]["n_clip_high"] == 0 and a["stats"]["n_clip_low"] == 0
    seq_of = np.repeat(np.arange(4), np.diff(offsets))
    assert abs(a["loss"] + adv[seq_of].astype(np.float64).sum() / 40) < 1e-12
    for k in ("loss", "grad_coef", "d_hidden", "d_W", "flags"):
        assert np.array_equal(np.asarray(a[k]), np.asarray(b[k]))


def planted_batch():
    """Rows 0..9 of a positive and of a negative sequence get a dominating target logit."""
    hidden, W, targets, offsets, adv, version = small_batch(seed=11)
    W[3] = 0.0
    W[3, 0] = 40.0
    for t in list(range(0, 5)) + list(range(7, 12)):
        targets[t] = 3
        hidden[t] = 0.0
        hidden[t, 0] = 1.0
    return hidden, W, targets, offsets, adv, version


def test_mask_invariants():
    hidden, W, targets, offsets, adv, version = planted_batch()
    logp, ent, _ = O.token_stats(hidden, W, targets)
    old = (logp + 0.01).astype(np.float32)
    run = lambda **kw: O.forward(hidden, W, targets, old, version, adv, offsets,
                                 O.OracleParams(is_mode="sais", **kw))
    always = run(mpt_mode="always")
    seq_of = np.repeat(np.arange(4), np.diff(offsets))
    A = adv[seq_of]
    masked = (always["flags"] & O.FLAG_MASKED) != 0
    p_tok = np.exp(logp)
    # negative (and zero) advantage tokens are never masked; their gradient is untouched
    assert not masked[A <= 0].any()
    off_run = run(mpt_mode="off")
    assert np.array_equal(always["grad_coef"][A <= 0], off_run["grad_coef"][A <= 0])
    # every positive token with p >= tau is masked and carries no gradient
    tau = float(np.float32(0.99))
    sure = (A > 0) & (p_tok >= tau + 1e-6)
    assert sure.sum() >= 5 and masked[sure].all() and (always["grad_coef"][sure] == 0).all()
    assert not masked[(A > 0) & (p_tok < tau - 1e-6)].any()
    # the gate: sigma = +inf is "always", sigma = -inf is "off"
    dyn_hi = run(mpt_mode="dynamic", entropy_target=float("inf"))
    dyn_lo = run(mpt_mode="dynamic", entropy_target=float("-inf"))
    assert np.array_equal(dyn_hi["flags"], always["flags"])
    assert np.array_equal(dyn_lo["flags"] & O.FLAG_MASKED, off_run["flags"] & O.FLAG_MASKED)
    assert np.array_equal(dyn_lo["grad_coef"], off_run["grad_coef"])
    # the gate flips exactly where H-bar crosses sigma (strict <)
    hbar0 = float(np.float32(always["seq_entropy"][0]))
    above = run(mpt_mode="dynamic", entropy_target=float(np.nextafter(np.float32(hbar0), np.float32(10))))
    at = run(mpt_mode="dynamic", entropy_target=hbar0)
    assert ((above["flags"][:7] & O.FLAG_MASKED) != 0).any()
    assert not ((at["flags"][:7] & O.FLAG_MASKED) != 0).any()
    # masked tokens still count in the normaliser: loss(off) - loss(always) = -(1/T) sum masked s
    diff = off_run["loss"] - always["loss"]
    assert abs(diff + off_run["surrogate"][masked].sum() / 40) < 1e-12


def test_threshold_strictness():
    p = O.OracleParams(is_mode="sais", mpt_mode="always", norm_tokens=1)
    ln_tau, ln_hi, ln_lo = O.decision_thresholds(p)
    one = np.array([1.0], np.float32)
    z = np.zeros(1, np.int32)
    # logp exactly at ln tau is an MPT (>=); one ulp below is not
    for lp, expect in ((ln_tau, True), (np.nextafter(ln_tau, np.float32(-1)), False)):
        out = O.decide(np.array([lp]), one, np.array([lp]), one, np.array([0, 1]), z, p)
        assert bool(out["flags"][0] & O.FLAG_MPT) == expect
    # d exactly at ln(1+eps) is not clipped (strict >)
    p2 = O.OracleParams(is_mode="sais", mpt_mode="off", norm_tokens=1)
    lp = np.float32(0.0)                                  # 0 - (-d) is exactly d
    for d, expect in ((ln_hi, False), (np.nextafter(ln_hi, np.float32(1)), True)):
        old = np.float32(lp - d)
        assert np.float32(lp - old) == d
        out = O.decide(np.array([lp]), one, np.array([old]), one, np.array([0, 1]), z, p2)
        assert bool(out["flags"][0] & O.FLAG_CLIP_HIGH) == expect
    for d, expect in ((ln_lo, False), (np.nextafter(ln_lo, np.float32(-1)), True)):
        old = np.float32(lp - d)
        assert np.float32(lp - old) == d
        out = O.decide(np.array([lp]), one, np.array([old]), -one, np.array([0, 1]), z, p2)
        assert bool(out["flags"][0] & O.FLAG_CLIP_LOW) == expect


def test_decision_thresholds_are_the_correctly_rounded_logarithms():
    """decision_thresholds against float32 bit patterns from a 60-digit decimal logarithm of the exact float32
    parameter (tests/golden/decision_thresholds.txt, written by make_decision_thresholds.py): the constants the
    bit-exact mask and clip decisions rest on have a value that does not come from libm."""
    seen = 0
    path = os.path.join(os.path.dirname(__file__), "golden", "decision_thresholds.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        kind, pbits, _, vbits, _ = line.split()
        param = float(np.array([int(pbits, 16)], dtype=np.uint32).view(np.float32)[0])
        want = np.array([int(vbits, 16)], dtype=np.uint32).view(np.float32)[0]
        if kind == "ln_tau":
            got = O.decision_thresholds(O.OracleParams(mpt_tau=param))[0]
        elif kind == "ln_1p_eps":
            got = O.decision_thresholds(O.OracleParams(clip_eps_high=param))[1]
        else:
            got = O.decision_thresholds(O.OracleParams(clip_eps_low=param))[2]
        assert got.dtype == np.float32 and got.view(np.uint32) == want.view(np.uint32), (kind, param, got, want)
        seen += 1
    assert seen == 9


def test_entropy_scopes_and_sequence_means():
    ent = np.array([0.5, 1.5, 0.25, 0.75, 4.0], np.float32)
    offsets = np.array([0, 2, 4, 5])
    seq_mean, batch_mean = O.sequence_mean_entropy(ent, offsets)
    assert np.allclose(seq_mean, [1.0, 0.5, 4.0], atol=0) and batch_mean == 1.4
    assert np.array_equal(O.gate_entropy(ent, offsets, "per_seq"), np.float32([1.0, 0.5, 4.0]))
    assert np.array_equal(O.gate_entropy(ent, offsets, "batch"), np.float32([1.4] * 3))
    assert np.array_equal(O.gate_entropy(ent, offsets, "supplied", [9, 8, 7]), np.float32([9, 8, 7]))


def test_normaliser_and_per_token_advantages():
    hidden, W, targets, offsets, adv, version = small_batch(seed=13)
    logp, _, _ = O.token_stats(hidden, W, targets)
    old = (logp - 0.05).astype(np.float32)
    a = O.forward(hidden, W, targets, old, version, adv, offsets, O.OracleParams(mpt_mode="off"))
    b = O.forward(hidden, W, targets, old, version, adv, offsets,
                  O.OracleParams(mpt_mode="off", norm_tokens=400))
    assert abs(a["loss"] / 10 - b["loss"]) < 1e-15
    assert np.allclose(a["grad_coef"] / 10, b["grad_coef"], rtol=1e-15)
    seq_of = np.repeat(np.arange(4), np.diff(offsets))
    c = O.forward(hidden, W, targets, old, version, adv[seq_of], offsets,
                  O.OracleParams(mpt_mode="off"), adv_per_token=True)
    assert c["loss"] == a["loss"] and np.array_equal(c["grad_coef"], a["grad_coef"])


def test_staleness_statistics():
    T = 6
    logp = np.float32([-1, -1, -1, -1, -1, -1])
    old = np.float32([-1, -1.5, -1, -0.5, -1, -1])      # ratios 1, e^.5 (clip hi), 1, e^-.5, 1, 1
    version = np.int32([3, 3, 2, 2, 0, 3])
    p = O.OracleParams(is_mode="sais", mpt_mode="off", current_version=3)
    out = O.decide(logp, np.float32([1.0]), old, np.float32([1.0]), np.array([0, T]), version, p)
    st = out["stats"]
    assert st["stale_tokens"][:4].tolist() == [3, 2, 0, 1]
    assert st["stale_clipped"][:4].tolist() == [1, 0, 0, 0]
    assert abs(st["stale_mean_abs_logratio"][0] - 0.5 / 3) < 1e-12
    assert abs(st["stale_mean_abs_logratio"][1] - 0.25) < 1e-12
    assert st["n_clip_high"] == 1 and st["n_clip_low"] == 0 and st["n_active"] == 5


# ------------------------------------------------------------------ gradients
def test_mean_nll_special_case():
    """A = 1, no mask, N = T, old = current: the gradients are those of the mean negative
    log-likelihood, dz = (p - onehot) / T (textbook)."""
    T, H, V = 12, 5, 9
    hidden, W, targets = rand_problem(T, H, V, 17)
    logp, _, _ = O.token_stats(hidden, W, targets)
    p = O.OracleParams(is_mode="sais", mpt_mode="off")
    out = O.fwd_bwd(hidden, W, targets, logp.astype(np.float32), np.zeros(T, np.int32),
                    np.ones(1, np.float32), np.array([0, T]), p)
    # float32 rounding of old_logp leaves r = 1 + O(1e-7); compare at 1e-6
    z = np.einsum("th,vh->tv", hidden.astype(np.float64), W.astype(np.float64))
    dz = scipy.special.softmax(z, axis=1)
    dz[np.arange(T), targets] -= 1.0
    dz /= T
    assert np.allclose(out["d_hidden"], dz @ W.astype(np.float64), atol=1e-6)
    assert np.allclose(out["d_W"], dz.T @ hidden.astype(np.float64), atol=1e-6)
    assert abs(out["loss"] + 1.0) < 1e-6


def test_dW_column_sums_vanish_and_dhidden_row_form():
    hidden, W, targets, offsets, adv, version = small_batch(seed=19)
    logp, _, lse = O.token_stats(hidden, W, targets, kappa=1.3)
    old = (logp + 0.03).astype(np.float32)
    p = O.OracleParams(mpt_mode="off", inv_temperature=1.3)
    out = O.fwd_bwd(hidden, W, targets, old, version, adv, offsets, p)
    assert np.abs(out["d_W"].sum(axis=0)).max() < 1e-12
    z = O.logits_rows(hidden, W, np.arange(40), kappa=1.3)
    prob = np.exp(z - lse[:, None])
    W64 = W.astype(np.float64)
    expect = 1.3 * out["grad_coef"][:, None] * (W64[targets] - prob @ W64)
    assert np.allclose(out["d_hidden"], expect, atol=1e-12)


def test_kl_estimate_closed_forms_and_expectation():
    """The per-token KL estimate of Eq. 5's term: zero at u = 0, non-negative, u^2 / 2 to second order, the
    hand values at u = +-ln 2 (2 - ln 2 - 1 and 1/2 + ln 2 - 1), and its mean under the policy equals the
    divergence D_KL[pi_theta || pi_ref] (SciPy's rel_entr) for every pair of small categorical distributions."""
    assert O.kl_estimate(0.0) == 0.0
    u = np.linspace(-3, 3, 61)
    assert (O.kl_estimate(u) >= 0).all() and (O.kl_estimate(u)[u != 0] > 0).all()
    assert abs(O.kl_estimate(1e-4) - 0.5e-8) < 1e-12
    assert abs(O.kl_estimate(0.6931471805599453) - 0.3068528194400547) < 1e-15
    assert abs(O.kl_estimate(-0.6931471805599453) - 0.1931471805599453) < 1e-15
    rng = np.random.default_rng(4)
    for V in (2, 5, 17):
        p_theta = rng.dirichlet(np.ones(V))
        p_ref = rng.dirichlet(np.ones(V))
        mean_k = float((p_theta * O.kl_estimate(np.log(p_ref) - np.log(p_theta))).sum())
        assert abs(mean_k - float(scipy.special.rel_entr(p_theta, p_ref).sum())) < 1e-12


def test_kl_term_in_the_decision_stage():
    """Eq. 5's objective s - beta k on hand cases: with A = 0 the loss is +beta k / N and the coefficient
    beta (1 - e^u) / N (it pulls logp towards the reference); a clipped token keeps the KL gradient; a masked
    token loses both terms; beta = 0 never reads ref_logp."""
    one, z = np.float32([1.0]), np.zeros(1, np.int32)
    ln2 = np.float32(0.6931471805599453)
    p = O.OracleParams(is_mode="sais", mpt_mode="off", norm_tokens=4, kl_beta=0.5)
    lp = np.float32([-1.0])
    out = O.decide(lp, one, lp, np.float32([0.0]), np.array([0, 1]), z, p, ref_logp=lp + ln2)
    k = 2.0 - float(np.float64(ln2)) - 1.0                       # u = ln 2 as the float32 difference gives it
    u = float(np.float64(np.float32(lp[0] + ln2)) - np.float64(lp[0]))
    assert abs(out["kl"][0] - (np.exp(u) - u - 1.0)) < 1e-15 and abs(out["kl"][0] - k) < 1e-6
    assert abs(out["loss"] - 0.5 * out["kl"][0] / 4) < 1e-15
    assert abs(out["grad_coef"][0] - 0.5 * (1.0 - np.exp(u)) / 4) < 1e-15 and out["grad_coef"][0] < 0
    # clipped (ratio e^0.5 > 1.2 with A > 0): the surrogate's gradient is gone, the KL one stays
    out = O.decide(lp, one, np.float32([-1.5]), one, np.array([0, 1]), z, p, ref_logp=lp - ln2)
    assert out["flags"][0] & O.FLAG_CLIP_HIGH
    u = float(np.float64(np.float32(lp[0] - ln2)) - np.float64(lp[0]))
    assert abs(out["grad_coef"][0] - 0.5 * (1.0 - np.exp(u)) / 4) < 1e-15 and out["grad_coef"][0] > 0
    assert abs(out["loss"] + (1.2 - 0.5 * out["kl"][0]) / 4) < 1e-8      # 1 + eps with eps = float32(0.2)
    # masked: nothing of the token is left
    pm = O.OracleParams(is_mode="sais", mpt_mode="always", norm_tokens=4, kl_beta=0.5)
    hi_lp = np.float32([-0.001])
    out = O.decide(hi_lp, one, hi_lp, one, np.array([0, 1]), z, pm, ref_logp=hi_lp - ln2)
    assert out["flags"][0] & O.FLAG_MASKED and out["loss"] == 0.0 and out["grad_coef"][0] == 0.0
    assert out["stats"]["mean_kl"] > 0            # the diagnostic still sees the token
    # beta = 0: the reference is not needed
    p0 = O.OracleParams(is_mode="sais", mpt_mode="off", norm_tokens=4)
    a = O.decide(lp, one, lp, one, np.array([0, 1]), z, p0)
    b = O.decide(lp, one, lp, one, np.array([0, 1]), z, p0, ref_logp=lp - ln2)
    assert a["loss"] == b["loss"] and a["grad_coef"][0] == b["grad_coef"][0] and b["stats"]["mean_kl"] == 0.0
    with pytest.raises(ValueError):
        O.decide(lp, one, lp, one, np.array([0, 1]), z, p)


@pytest.mark.parametrize("kappa,loss_norm,kl_beta", [(1.0, "tokens", 0.0), (1.0 / 0.85, "tokens", 0.0),
                                                    (1.0, "sequence", 0.0), (1.0, "tokens", 0.3),
                                                    (1.0 / 0.85, "sequence", 0.3)])
def test_finite_differences(kappa, loss_norm, kl_beta):
    """Central differences of the Eq. 10 objective (with Eq. 5's KL term when kl_beta > 0) in float64 on a
    tiny problem, with clipped, masked, negative-advantage and zero-advantage tokens present and every
    token at least 1e-2 away from each threshold."""
    T, H, V = 6, 4, 10
    rng = np.random.default_rng(23)
    hidden = rng.standard_normal((T, H))
    W = rng.standard_normal((V, H))
    targets = np.array([1, 4, 4, 9, 0, 2], np.int32)
    # make token 0 a mastered positive token
    hidden[0] = 0.0
    hidden[0, 1] = 1.0
    W[1] = 0.0
    W[1, 1] = 14.0
    offsets = np.array([0, 3, 5, 6], np.int32)
    adv = np.array([0.8, -1.2, 0.0], np.float32)
    logp, _, _ = O.token_stats(hidden, W, targets, kappa)
    shift = np.array([0.0, 0.4, -0.1, -0.5, 0.15, 0.0])     # clip-high on 1, clip-low on 3
    old = (logp - shift).astype(np.float32)
    p = O.OracleParams(is_mode="sais", mpt_mode="always", inv_temperature=kappa, norm_tokens=9, loss_norm=loss_norm,
                       norm_seqs=4, kl_beta=kl_beta)
    ref = (logp + np.array([0.3, -0.2, 0.5, -0.4, 0.1, 0.25])).astype(np.float32)
    out = O.fwd_bwd(hidden, W, targets, old, np.zeros(T, np.int32), adv, offsets, p, ref_logp=ref)
    fl = out["flags"]
    assert fl[0] & O.FLAG_MASKED and fl[1] & O.FLAG_CLIP_HIGH and fl[3] & O.FLAG_CLIP_LOW
    assert out["stats"]["n_active"] == (2 if kl_beta == 0 else 5)   # the KL gradient also flows through clipped and A = 0 tokens
    ln_tau, ln_hi, ln_lo = O.decision_thresholds(p)
    d = logp - old
    assert (np.abs(d - ln_hi) > 1e-2).all() and (np.abs(d - ln_lo) > 1e-2).all()
    assert (np.abs(logp - ln_tau) > 1e-2).all()
    masked = (fl & O.FLAG_MASKED) != 0
    f = lambda h, w: O.objective_value(h, w, targets, old, adv, offsets, masked, p, ref_logp=ref)
    # the oracle takes d from float32 log-probs, the smooth objective from float64 ones:
    # values agree to float32 rounding of logp (1e-7 relative), nothing coarser
    assert abs(f(hidden, W) - out["loss"]) < 1e-7
    step = 1e-6
    num_dH = np.zeros_like(hidden)
    for idx in np.ndindex(*hidden.shape):
        hp, hm = hidden.copy(), hidden.copy()
        hp[idx] += step
        hm[idx] -= step
        num_dH[idx] = (f(hp, W) - f(hm, W)) / (2 * step)
    num_dW = np.zeros_like(W)
    for idx in np.ndindex(*W.shape):
        wp, wm = W.copy(), W.copy()
        wp[idx] += step
        wm[idx] -= step
        num_dW[idx] = (f(hidden, wp) - f(hidden, wm)) / (2 * step)
    assert np.abs(out["d_hidden"]).max() > 1e-3
    assert np.allclose(out["d_hidden"], num_dH, rtol=1e-6, atol=1e-7)
    assert np.allclose(out["d_W"], num_dW, rtol=1e-6, atol=1e-7)


def test_backward_row_subset_and_grad_loss():
    hidden, W, targets, offsets, adv, version = small_batch(seed=29)
    g = np.random.default_rng(0).standard_normal(40) * 0.01
    dH, dW = O.backward(hidden, W, targets, g)
    rows = np.array([5, 39, 12])
    dH_s, dW_s = O.backward(hidden, W, targets, g, rows=rows, grad_loss=2.0)
    assert np.allclose(dH_s, 2.0 * dH[rows], atol=1e-14)
    g_only = np.zeros(40)
    g_only[rows] = g[rows]
    _, dW_o = O.backward(hidden, W, targets, g_only)
    assert np.allclose(dW_s, 2.0 * dW_o, atol=1e-14)
    # additivity of dW over a partition of the rows
    _, dW_a = O.backward(hidden, W, targets, g, rows=np.arange(0, 17))
    _, dW_b = O.backward(hidden, W, targets, g, rows=np.arange(17, 40))
    assert np.allclose(dW_a + dW_b, dW, atol=1e-13)


# ------------------------------------------------------------------ Eq. 5 per-sample normalisation
def test_sequence_normalisation_closed_forms():
    """With the ratio identically one and no mask the surrogate of a token is its advantage, so the two
    normalisations have closed forms: tokens -sum_i |o_i| A_i / T (Eq. 10's 1/sum|o_i|), sequence -(1/G) sum_i A_i
    (Eq. 5's (1/G) sum_i (1/|o_i|) sum_t), the second independent of the lengths."""
    off = np.array([0, 7, 9, 12], np.int32)
    adv = np.array([0.5, -2.0, 1.25], np.float32)
    T = 12
    lp = np.full(T, -1.0, np.float32)
    ent = np.ones(T, np.float32)
    kw = dict(is_mode="pois", mpt_mode="off")
    tok = O.decide(lp, ent[:3], None, adv, off, None, O.OracleParams(**kw))
    seq = O.decide(lp, ent[:3], None, adv, off, None, O.OracleParams(loss_norm="sequence", **kw))
    assert abs(tok["loss"] + (7 * 0.5 - 2 * 2.0 + 3 * 1.25) / 12) < 1e-15
    assert abs(seq["loss"] + (0.5 - 2.0 + 1.25) / 3) < 1e-15
    assert np.allclose(tok["grad_coef"], -np.repeat(adv, [7, 2, 3]) / 12, atol=1e-16)
    assert np.allclose(seq["grad_coef"], -np.repeat(adv / np.array([7, 2, 3]), [7, 2, 3]) / 3, atol=1e-16)
    assert np.array_equal(tok["flags"], seq["flags"])                   # decisions do not depend on the weights
    # G supplied by the caller (a micro-batch of a larger group)
    seq6 = O.decide(lp, ent[:3], None, adv, off, None, O.OracleParams(loss_norm="sequence", norm_seqs=6, **kw))
    assert abs(seq6["loss"] - seq["loss"] / 2) < 1e-15 and np.allclose(seq6["grad_coef"], seq["grad_coef"] / 2)
    # equal lengths: the two normalisations coincide
    off2 = np.array([0, 4, 8, 12], np.int32)
    a = O.decide(lp, ent[:3], None, adv, off2, None, O.OracleParams(**kw))
    b = O.decide(lp, ent[:3], None, adv, off2, None, O.OracleParams(loss_norm="sequence", **kw))
    assert abs(a["loss"] - b["loss"]) < 1e-15 and np.allclose(a["grad_coef"], b["grad_coef"], atol=1e-16)


# ------------------------------------------------------------------ Eq. 4 advantages
def test_group_advantages_closed_forms():
    # k correct of G with 0/1 rewards: mean p = k/G, std sqrt(p(1-p)); A(1) = sqrt((1-p)/p), A(0) = -sqrt(p/(1-p))
    r = np.array([1, 0, 0, 0, 1, 1, 1, 1, 0, 0, 0, 0], dtype=np.float32)
    adv, keep = O.group_advantages(r, 4)
    assert np.allclose(adv[:4], [math.sqrt(3.0), -math.sqrt(1 / 3), -math.sqrt(1 / 3), -math.sqrt(1 / 3)], atol=1e-15)
    assert np.array_equal(adv[4:], np.zeros(8))                  # all right / all wrong: no spread
    assert keep.tolist() == [1] * 4 + [0] * 8                     # Eq. 7: 0 < #correct < G
    # sign of the advantage is the correctness (Section 3.3); zero mean and unit spread within a kept group
    r = np.array([1, 1, 0, 1, 0, 0, 1, 0], dtype=np.float32)
    adv, keep = O.group_advantages(r, 8)
    assert ((adv > 0) == (r == 1)).all() and abs(adv.mean()) < 1e-15 and abs(adv.std() - 1.0) < 1e-15
    assert keep.all()
    # library second opinion
    ref = (r - r.mean()) / r.std()
    assert np.allclose(adv, ref, atol=1e-15)

"""Parity at the full workload sizes (V = 151936, H = 2048) in the launch configuration that
bench.py times.  The oracle cannot run 10^14 multiply-adds, so it computes a stratified sample of
token rows one by one (log-prob, entropy, dHidden row) and a sub-batch for dW; the rest is checked by
properties that hold at any size (decisions re-derived from the GPU's own log-probs, sequence means,
dW column sums, independence of dW from the backward panel size)."""
import numpy as np
import pytest
import torch

from oracle import ulorl_oracle as O
from paper_2507_19766_b200 import binding as B
from workloads import synth
from tests.helpers import TOL_GRAD, TOL_LOGP, both_params, rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def stratified_rows(batch, n_random=160, seed=0):
    wl = batch.workload
    T = wl.T
    rng = np.random.default_rng(seed)
    rows = {0, 1, 127, 128, 129, 255, 256, T - 129, T - 128, T - 1, 16383, 16384, 16385}
    off = batch.seq_offsets.numpy()
    for i in range(min(wl.S, 12)):                       # first and last token of some sequences
        rows.add(int(off[i]))
        rows.add(int(off[i + 1]) - 1)
    tg = batch.targets.numpy()
    tail = np.nonzero(tg >= (wl.V // 256) * 256)[0]       # target inside the last (partial) vocabulary tile
    rows.update(int(x) for x in tail[:8])
    ver = batch.segment_version.numpy()
    for v in np.unique(ver):                             # every policy version
        idx = np.nonzero(ver == v)[0]
        rows.update(int(x) for x in rng.choice(idx, size=min(4, idx.size), replace=False))
    planted = batch.planted_rows
    for sel in (planted, ~planted):
        idx = np.nonzero(sel)[0]
        if idx.size:
            rows.update(int(x) for x in rng.choice(idx, size=min(n_random // 2, idx.size), replace=False))
    rows = np.array(sorted(r for r in rows if 0 <= r < T), dtype=np.int64)
    return rows


@pytest.mark.parametrize("name", ["ultra", "ultra_open", "qwen", "mixed"])
def test_full_size_workload_against_sampled_oracle(name):
    wl = synth.WORKLOADS[name]
    batch = synth.make_batch(wl, device=DEV)
    gp, op = both_params(batch)
    b = batch.to(DEV)
    ws = B.alloc_workspace(gp, DEV)
    out = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages,
                           b.seq_offsets, workspace=ws)
    dH, dW = B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, workspace=ws)
    torch.cuda.synchronize()
    assert B.check_status(ws) == B.OK

    # ---- sampled rows: log-prob, entropy, lse one by one
    rows = stratified_rows(batch)
    rt = torch.from_numpy(rows)
    W_host = batch.host_f32("W")
    h_rows = batch.hidden[rt].float().numpy()
    y_rows = batch.targets[rt].numpy()
    logp_r, ent_r, lse_r = O.token_stats(h_rows, W_host, y_rows, op.inv_temperature)
    logp = out.logp.cpu().numpy()
    ent = out.entropy.cpu().numpy()
    assert np.abs(logp[rows] - logp_r).max() <= TOL_LOGP
    assert np.abs(ent[rows] - ent_r).max() <= TOL_LOGP
    assert np.abs(out.lse.cpu().numpy()[rows] - lse_r).max() <= TOL_LOGP
    assert np.isfinite(logp).all() and (ent >= 0).all() and (ent <= np.log(wl.V) + 1e-3).all() and (logp <= 1e-6).all()

    # ---- whole batch, properties that need no oracle: sequence means of the GPU's own entropies, and
    #      the mask bit is the MPT bit gated by the sequence's mean entropy
    off = batch.seq_offsets.numpy()
    lens = np.diff(off)
    seq_ent = out.seq_entropy.cpu().numpy()[: wl.S]
    assert np.allclose(seq_ent, np.add.reduceat(ent.astype(np.float64), off[:-1]) / lens, rtol=1e-6, atol=1e-9)
    st = out.stats_host()
    assert abs(st["mean_entropy"] - float(ent.astype(np.float64).mean())) <= 1e-6
    flags = out.flags.cpu().numpy()
    seq_of = np.repeat(np.arange(wl.S), lens)
    gate = np.ones(wl.S, bool) if op.mpt_mode == "always" else (seq_ent < np.float32(op.entropy_target))
    assert np.array_equal((flags & O.FLAG_MASKED) != 0, ((flags & O.FLAG_MPT) != 0) & gate[seq_of])
    g = out.grad_coef.cpu().numpy()
    assert st["n_tokens"] == wl.T and st["n_masked"] == int(((flags & O.FLAG_MASKED) != 0).sum())
    assert st["n_active"] == int(np.count_nonzero(g)) and st["n_mpt"] == int(((flags & O.FLAG_MPT) != 0).sum())
    assert st["n_clip_high"] == int(((flags & O.FLAG_CLIP_HIGH) != 0).sum())
    assert st["n_clip_low"] == int(((flags & O.FLAG_CLIP_LOW) != 0).sum())
    if name == "ultra":        # the recipe puts the mean entropy below sigma: the dynamic gate is open
        assert seq_ent[0] < wl.entropy_target and st["n_masked"] > wl.T // 2 and st["n_active"] > wl.T // 20
    if name == "ultra_open":   # weaker plants: mean entropy above sigma, the gate stays shut, MPTs are not masked
        assert seq_ent[0] > wl.entropy_target and st["n_masked"] == 0 and st["n_mpt"] > wl.T // 4
        assert st["n_active"] > wl.T // 2
    if name == "mixed":
        assert st["n_clip_high"] == 0 and st["n_clip_low"] == 0
    if name == "qwen":         # static masking: planted targets of positive sequences are masked
        assert st["n_mpt"] > 0 and st["n_masked"] == st["n_mpt"]

    # ---- sampled rows: the oracle's decisions and coefficients from its own log-probs.  The sampled rows of
    #      a sequence form a sub-sequence; the gate value of a sequence is the oracle's mean entropy over its
    #      sampled rows, which must be clear of sigma for the comparison to mean anything.
    sub_seq = seq_of[rows]
    present, sub_counts = np.unique(sub_seq, return_counts=True)
    sub_off = np.concatenate([[0], np.cumsum(sub_counts)]).astype(np.int32)
    gate_est = np.array([ent_r[sub_seq == i].mean() for i in present])
    trusted_seq = np.ones(present.shape[0], bool)
    if op.mpt_mode == "dynamic":
        # an estimate from few rows is only trusted when it is far from sigma
        far = np.abs(gate_est - op.entropy_target)
        trusted_seq = ((sub_counts >= 32) & (far > 0.04)) | (far > 1.0)
        assert trusted_seq.sum() >= 1
        # the GPU's gate (from its own full-sequence means) agrees with every trusted estimate
        assert np.array_equal((gate_est < op.entropy_target)[trusted_seq], gate[present][trusted_seq])
    trusted = np.repeat(trusted_seq, sub_counts)
    op_sub = O.OracleParams(**{**op.__dict__, "norm_tokens": wl.T})
    dec = O.decide(logp_r.astype(np.float32), gate_est.astype(np.float32), batch.old_logp.numpy()[rows],
                   batch.advantages.numpy()[present], sub_off, batch.segment_version.numpy()[rows], op_sub)
    ln_tau, ln_hi, ln_lo = (float(x) for x in O.decision_thresholds(op))
    d_r = logp_r - batch.old_logp.numpy()[rows].astype(np.float64)
    near = np.abs(logp_r - ln_tau) <= TOL_LOGP
    if op.is_mode == "sais":
        near |= (np.abs(d_r - ln_hi) <= TOL_LOGP) | (np.abs(d_r - ln_lo) <= TOL_LOGP)
    differ = flags[rows] != dec["flags"]
    assert not (differ & ~near & trusted).any()
    agree = ~differ & trusted
    assert np.allclose(g[rows][agree], dec["grad_coef"][agree], rtol=2 * TOL_LOGP, atol=1e-14)

    # ---- sampled rows of dHidden against the oracle's backward on the oracle's coefficients
    g_or = dec["grad_coef"]
    sel = agree & (g_or != 0)
    active = rows[sel]
    assert active.size >= 16
    dH_ref, _ = O.backward(h_rows[sel], W_host, y_rows[sel], g_or[sel], op.inv_temperature, want_dW=False)
    dH_gpu = dH[torch.from_numpy(active).to(DEV)].float().cpu().numpy()
    assert rel_l2(dH_gpu, dH_ref) <= TOL_GRAD
    # row by row.  dHidden[t] = kappa g_t ((1 - p_y) W_y - sum_{v != y} p_v W_v): a float32 error d in the row's
    # log-prob moves the first term by kappa |g_t| p_y d |W_y| whatever the size of 1 - p_y, so a row whose target
    # probability is close to one carries an absolute error that its own (tiny) norm cannot absorb.  With float32
    # accumulation over H = 2048 and logits up to ~40 that d is a few 1e-5 (the forward's contract allows 2e-3);
    # the bound takes 1e-4.
    row_err = np.linalg.norm(dH_gpu - dH_ref, axis=1)
    row_ref = np.linalg.norm(dH_ref, axis=1)
    w_y = np.linalg.norm(W_host[y_rows[sel]].astype(np.float64), axis=1)
    floor = op.inv_temperature * np.abs(g_or[sel]) * 1e-4 * w_y
    assert (row_err <= 3 * TOL_GRAD * row_ref + floor).all()
    inactive = rows[g[rows] == 0]
    if inactive.size:
        assert float(dH[torch.from_numpy(inactive).to(DEV)].float().abs().max()) == 0.0

    # ---- dW: properties at full size
    # column sums of d_W vanish up to the bf16 rounding of dz: six standard deviations of independent roundings
    # (2^-9 sqrt(2) |coef_t| per token) plus the float32 part that adds up linearly; the worst case behind it
    colsum = dW.double().sum(dim=0).abs()
    coef_t = out.grad_coef.abs().double() * op.inv_temperature
    stat = torch.zeros(wl.H, dtype=torch.float64, device=DEV)
    syst = torch.zeros(wl.H, dtype=torch.float64, device=DEV)
    for a in range(0, wl.T, 16384):
        ch = coef_t[a:a + 16384, None] * b.hidden[a:a + 16384].double().abs()
        stat += (ch * ch).sum(dim=0)
        syst += ch.sum(dim=0)
    bound = 6.0 * 2.0 ** -9 * np.sqrt(2.0) * stat.sqrt() + 4e-6 * syst + 1e-12
    assert bool((colsum <= bound).all()), float((colsum / bound).max())
    coef_sum = float(np.abs(g).sum()) * op.inv_temperature
    assert float(colsum.max()) <= 2.0 ** -8 * coef_sum * float(batch.hidden.float().abs().max()) + 1e-12
    print(f"{name}: d_W column sums at most {float((colsum / bound).max()):.3f} of the statistical bound")
    assert torch.isfinite(dW).all()
    dW_host = dW.cpu()
    del dW, dH
    gp2, _ = both_params(batch, bwd_panel_tokens=8192)
    ws2 = B.alloc_workspace(gp2, DEV)
    _, dW2 = B.token_loss_bwd(gp2, b.hidden, b.W, b.targets, out.lse, out.grad_coef, workspace=ws2)
    torch.cuda.synchronize()
    assert rel_l2(dW2.cpu().numpy(), dW_host.numpy()) <= 1e-4       # same sum, other panel boundaries
    del dW2, ws2
    # the compacted backward (rows with a zero coefficient dropped) gives the same gradients
    gp3, _ = both_params(batch, compact_rows=True)
    ws3c = B.alloc_workspace(gp3, DEV)
    dH3, dW3 = B.token_loss_bwd(gp3, b.hidden, b.W, b.targets, out.lse, out.grad_coef, workspace=ws3c)
    torch.cuda.synchronize()
    assert B.check_status(ws3c) == B.OK
    assert rel_l2(dW3.cpu().numpy(), dW_host.numpy()) <= 1e-4
    ta_all = torch.from_numpy(rows).to(DEV)
    assert rel_l2(dH3[ta_all].float().cpu().numpy()[sel], dH_ref) <= TOL_GRAD   # sel: sampled rows with a coefficient
    zero_rows = np.nonzero(g == 0)[0][:4096]
    if zero_rows.size:
        assert float(dH3[torch.from_numpy(zero_rows).to(DEV)].float().abs().max()) == 0.0
    del dH3, dW3, ws3c

    # ---- dW: sub-batch of the sampled active rows; the oracle's lse and coefficients are handed to the GPU
    n_sub = int(active.size)
    sub = B.Params(T=n_sub, H=wl.H, V=wl.V, num_seqs=1, dtype="bf16", is_mode=wl.is_mode, mpt_mode="off",
                   norm_tokens=wl.T, current_version=batch.current_version)
    ta = torch.from_numpy(active).to(DEV)
    ws3 = B.alloc_workspace(sub, DEV)
    f32 = lambda x: torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(DEV)
    dH_s, dW_s = B.token_loss_bwd(sub, b.hidden[ta].contiguous(), b.W, b.targets[ta].contiguous(),
                                  f32(lse_r[sel]), f32(g_or[sel]), workspace=ws3)
    torch.cuda.synchronize()
    _, dW_ref = O.backward(h_rows[sel], W_host, y_rows[sel], g_or[sel], op.inv_temperature)
    assert rel_l2(dW_s.cpu().numpy(), dW_ref) <= TOL_GRAD
    assert rel_l2(dH_s.float().cpu().numpy(), dH_ref) <= TOL_GRAD

"""Parity of the CUDA path (through the C ABI) against the fp64 oracle, element by element, on
seeded workloads the oracle finishes in seconds.  Tolerances: log-prob and entropy 2e-3 abs,
loss 1e-3 rel, gradients 1e-2 rel-L2; masks and clip flags exact on identical log-probs."""
import numpy as np
import pytest
import torch

from oracle import ulorl_oracle as O
from paper_2507_19766_b200 import binding as B
from workloads import synth
from tests.helpers import TOL_GRAD, TOL_LOGP, TOL_LOSS, both_params, near_threshold, oracle_inputs, rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

STAT_KEYS = ("n_tokens", "n_active", "n_mpt", "n_masked", "n_clip_high", "n_clip_low")
COLSUM_MARGINS = []      # largest |column sum of d_W| / statistical bound seen by each parity case (reported at the end)


def gpu_fwd_bwd(batch, gp, grad_loss=None, entropy_supplied=None):
    b = batch.to(DEV)
    ws = B.alloc_workspace(gp, DEV)
    es = None if entropy_supplied is None else torch.tensor(entropy_supplied, dtype=torch.float32, device=DEV)
    out = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages,
                           b.seq_offsets, entropy_supplied=es, workspace=ws)
    gl = None if grad_loss is None else torch.tensor([grad_loss], dtype=torch.float32, device=DEV)
    dH, dW = B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, grad_loss=gl, workspace=ws)
    torch.cuda.synchronize()
    assert B.check_status(ws) == B.OK
    return out, dH, dW


def check_against_oracle(batch, gp, op, grad_loss=None, check_grads=True):
    """Everything the oracle computes comes from the stored inputs only; data flows from the oracle
    to the GPU (its float32 log-probs into the decision kernel, its coefficients into the backward),
    never the other way."""
    out, dH, dW = gpu_fwd_bwd(batch, gp, grad_loss=grad_loss)
    oi = oracle_inputs(batch)
    S = batch.workload.S
    ref = O.forward(oi["hidden"], oi["W"], oi["targets"], oi["old_logp"], oi["segment_version"], oi["advantages"],
                    oi["seq_offsets"], op)
    logp = out.logp.cpu().numpy()
    ent = out.entropy.cpu().numpy()
    lse = out.lse.cpu().numpy()
    assert np.abs(logp - ref["logp"]).max() <= TOL_LOGP
    assert np.abs(ent - ref["entropy"]).max() <= TOL_LOGP
    assert np.abs(lse - ref["lse"]).max() <= TOL_LOGP
    seq_ent = out.seq_entropy.cpu().numpy()[:S]
    assert np.abs(seq_ent - ref["seq_entropy"]).max() <= TOL_LOGP
    st = out.stats_host()
    assert abs(st["mean_entropy"] - ref["mean_entropy"]) <= TOL_LOGP and st["device_status"] == 0

    # (1) fused path: decisions equal the oracle's wherever the oracle's own value is not within the
    #     tolerance of a threshold; coefficients of the tokens decided alike agree to the log-prob error
    flags = out.flags.cpu().numpy()
    near = near_threshold(ref["logp"], oi["old_logp"], ref["seq_entropy"], oi["seq_offsets"], op)
    differ = flags != ref["flags"]
    assert not (differ & ~near).any(), f"{int((differ & ~near).sum())} decisions differ away from any threshold"
    g = out.grad_coef.cpu().numpy()
    same = ~differ
    assert np.allclose(g[same], ref["grad_coef"][same], rtol=2 * TOL_LOGP, atol=1e-12)
    loss = float(out.loss.cpu()[0])
    N = float(op.norm_tokens) if op.norm_tokens > 0 else float(batch.workload.T)
    if op.loss_norm == "sequence":                                        # a token weighs at most 1/G there
        N = float(op.norm_seqs) if op.norm_seqs > 0 else float(S)
    flip_slack = float(np.abs(ref["surrogate"][differ]).sum()) / N        # what flipped tokens can move
    assert abs(loss - ref["loss"]) <= TOL_LOSS * max(abs(ref["loss"]), 1e-3) + flip_slack
    if not differ.any():
        for k in STAT_KEYS:
            assert st[k] == ref["stats"][k], k

    # (2) decision kernel alone on the oracle's float32 log-probs and entropies: bit-exact flags and counts
    t = lambda x, dt: torch.from_numpy(np.ascontiguousarray(x)).to(dt).to(DEV)
    b = batch.to(DEV)
    dec = B.token_loss_decide(gp, t(ref["logp"].astype(np.float32), torch.float32),
                              t(ref["entropy"].astype(np.float32), torch.float32), b.old_logp, b.segment_version,
                              b.advantages, b.seq_offsets)
    torch.cuda.synchronize()
    assert np.array_equal(dec.flags.cpu().numpy(), ref["flags"])
    assert np.allclose(dec.grad_coef.cpu().numpy(), ref["grad_coef"], rtol=2e-6, atol=1e-12)
    dst = dec.stats_host()
    for k in STAT_KEYS:
        assert dst[k] == ref["stats"][k], k
    assert dst["stale_tokens"] == ref["stats"]["stale_tokens"].tolist()
    assert dst["stale_clipped"] == ref["stats"]["stale_clipped"].tolist()
    assert np.allclose(dst["stale_mean_abs_logratio"], ref["stats"]["stale_mean_abs_logratio"], rtol=1e-5, atol=1e-7)
    assert abs(float(dec.loss.cpu()[0]) - ref["loss"]) <= 2e-6 * max(1.0, abs(ref["loss"]))
    assert np.allclose(dec.seq_entropy.cpu().numpy()[:S], ref["seq_entropy"], rtol=1e-6, atol=1e-9)

    if check_grads:
        gl = 1.0 if grad_loss is None else grad_loss
        dH_ref, dW_ref = O.backward(oi["hidden"], oi["W"], oi["targets"], ref["grad_coef"], op.inv_temperature,
                                    grad_loss=gl)
        if differ.any():
            # (3a) some near-threshold token was decided the other way: compare the backward kernels on the
            #      oracle's coefficients (the GPU's own are covered by (1))
            ws = B.alloc_workspace(gp, DEV)
            glt = None if grad_loss is None else torch.tensor([grad_loss], dtype=torch.float32, device=DEV)
            dH, dW = B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse,
                                      t(ref["grad_coef"].astype(np.float32), torch.float32), grad_loss=glt,
                                      workspace=ws)
            torch.cuda.synchronize()
        eh = rel_l2(dH.float().cpu().numpy(), dH_ref)
        ew = rel_l2(dW.cpu().numpy(), dW_ref)
        assert eh <= TOL_GRAD and ew <= TOL_GRAD, (eh, ew)
        # sum_v dz[t, v] = 0, so the column sums of d_W vanish up to the rounding of dz.  The tensor path stores dz in
        # bf16: every element carries an independent relative error of at most 2^-9, so the error of sum_v dz[t, v]
        # has a standard deviation below e_t = 2^-9 |dz_t|_2 <= 2^-9 sqrt(2) |coef_t|, and the column sum over T
        # tokens one below sqrt(sum_t (e_t hidden[t, h])^2).  Held to six of those, plus the systematic part that
        # does add up linearly: softmax rows that sum to one only to float32 (4e-6 sum_t |coef_t hidden[t, h]|).
        # The float32 path has no bf16 step (1e-6 in place of 2^-9).  The worst-case bound (all roundings aligned)
        # is kept behind it; it never binds.
        colsum = np.abs(dW.double().sum(dim=0).cpu().numpy())
        coef = np.abs(ref["grad_coef"]) * op.inv_temperature * abs(gl)
        habs = np.abs(oi["hidden"]).astype(np.float64)
        unit = 2.0 ** -9 * np.sqrt(2.0) if (gp.dtype == "bf16" and gp.kernel_path != "simt") else 1e-6
        stat = 6.0 * unit * np.sqrt(((coef[:, None] * habs) ** 2).sum(axis=0))
        syst = 4e-6 * (coef[:, None] * habs).sum(axis=0)
        assert (colsum <= stat + syst + 1e-12).all(), float((colsum / (stat + syst + 1e-12)).max())
        worst = 2.0 ** -8 if (gp.dtype == "bf16" and gp.kernel_path != "simt") else 1e-5
        assert colsum.max() <= worst * float(coef.sum()) * 1.01 * float(habs.max()) + 1e-12
        COLSUM_MARGINS.append(float((colsum / (stat + syst + 1e-12)).max()))
    return out, ref


# --------------------------------------------------------------------------- named workloads
def test_tiny_f32():
    wl = synth.WORKLOADS["tiny"]
    batch = synth.make_batch(wl)
    gp, op = both_params(batch)
    out, ref = check_against_oracle(batch, gp, op)


def test_tiny_f32_old_logp_from_oracle():
    """The 'tiny' recipe as stated: old_logp = the oracle's current log-prob + N(0, 0.05)."""
    wl = synth.WORKLOADS["tiny"]
    b0 = synth.make_batch(wl)
    oi = oracle_inputs(b0)
    logp, _, _ = O.token_stats(oi["hidden"], oi["W"], oi["targets"])
    batch = synth.make_batch(wl, base_logp=logp.astype(np.float32))
    gp, op = both_params(batch)
    check_against_oracle(batch, gp, op)


@pytest.mark.parametrize("mpt_mode", ["always", "dynamic", "off"])
def test_tiny_planted_mask_fires(mpt_mode):
    wl = synth.WORKLOADS["tiny"].scaled(planted=0.5, beta_planted=(120.0, 220.0), mpt_mode=mpt_mode,
                                        entropy_target=5.0)
    batch = synth.make_batch(wl, seed=77)
    gp, op = both_params(batch)
    out, ref = check_against_oracle(batch, gp, op)
    if mpt_mode != "off":
        assert ref["stats"]["n_masked"] > 20
    assert ref["stats"]["n_mpt"] > 20


@pytest.mark.parametrize("path", ["tensor", "tensor_1cta", "simt"])
def test_bf16_mini_ragged(path):
    """bf16, several token tiles with a ragged tail, vocabulary not a multiple of any tile width,
    hidden size not a multiple of the 64-element pipeline stage, two backward panels."""
    wl = synth.WORKLOADS["small"].scaled(T=700, S=5, H=328, V=3001, lengths="lognormal:100:400",
                                         segment_len=64, planted=0.3, beta_planted=(80.0, 160.0),
                                         mpt_mode="dynamic", entropy_target=6.0)
    batch = synth.make_batch(wl, seed=5)
    gp, op = both_params(batch, kernel_path=path, bwd_panel_tokens=384)
    check_against_oracle(batch, gp, op)


@pytest.mark.parametrize("path", ["tensor", "tensor_1cta"])
def test_odd_staging_tile_counts_across_units(path):
    """The dz and d_W epilogues hand tiles to the copy engine through two alternating staging buffers.
    Here the last column tile of a unit ends after an odd number of copies (ceil(V / 64) = 301 = 1 mod 4 for
    dz, H / 32 = 11 chunks for d_W) and every persistent worker runs more than one unit (3 x 76 dz units,
    76 d_W units on 74 or 148 workers), so a worker's next unit starts right behind an odd count."""
    wl = synth.WORKLOADS["small"].scaled(T=600, S=4, H=352, V=19264, lengths="lognormal:100:300", segment_len=64,
                                         planted=0.3, beta_planted=(80.0, 160.0), mpt_mode="dynamic",
                                         entropy_target=6.0)
    batch = synth.make_batch(wl, seed=51)
    gp, op = both_params(batch, kernel_path=path, bwd_panel_tokens=512)
    check_against_oracle(batch, gp, op)


def test_bf16_temperature_and_grad_loss():
    wl = synth.WORKLOADS["small"].scaled(T=512, S=4, H=256, V=2048, lengths="tiny", segment_len=100)
    batch = synth.make_batch(wl, seed=9)
    gp, op = both_params(batch, inv_temperature=1.0 / 0.85, norm_tokens=4096)
    check_against_oracle(batch, gp, op, grad_loss=0.5)


def test_small_bf16_full():
    """The 'small' workload in full: T=16384, H=1024, V=32768 (oracle: tens of seconds)."""
    wl = synth.WORKLOADS["small"]
    batch = synth.make_batch(wl)
    gp, op = both_params(batch)
    check_against_oracle(batch, gp, op)


def test_pois_path():
    wl = synth.WORKLOADS["small"].scaled(T=640, S=6, H=256, V=4096, lengths="lognormal:100:300", segment_len=50,
                                         is_mode="pois", planted=0.4, beta_planted=(100.0, 200.0), noise="stale:0.02",
                                         mpt_mode="always")
    batch = synth.make_batch(wl, seed=3)
    gp, op = both_params(batch)
    out, ref = check_against_oracle(batch, gp, op)
    assert ref["stats"]["n_clip_high"] == 0 and ref["stats"]["n_clip_low"] == 0
    # POIS does not read old_logp: NULL is accepted and gives the same result
    b = batch.to(DEV)
    out2 = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, None, b.segment_version, b.advantages, b.seq_offsets)
    assert torch.equal(out2.grad_coef, out.grad_coef) and torch.equal(out2.loss, out.loss)


# --------------------------------------------------------------------------- tensor path vs SIMT path
def test_tensor_path_matches_simt_path():
    wl = synth.WORKLOADS["small"].scaled(T=1000, S=3, H=512, V=5000, lengths="lognormal:300:600", segment_len=128)
    batch = synth.make_batch(wl, seed=21)
    res = {}
    for path in ("tensor", "tensor_1cta", "simt"):
        gp, _ = both_params(batch, kernel_path=path)
        res[path] = gpu_fwd_bwd(batch, gp)
    b = res["simt"]
    for path in ("tensor", "tensor_1cta"):
        a = res[path]
        assert (a[0].logp - b[0].logp).abs().max() <= 1e-4
        assert (a[0].entropy - b[0].entropy).abs().max() <= 1e-4
        assert rel_l2(a[1].float().cpu().numpy(), b[1].float().cpu().numpy()) <= 1e-2
        assert rel_l2(a[2].cpu().numpy(), b[2].cpu().numpy()) <= 1e-2
    # the two tensor-core variants differ only in how the vocabulary is split and merged
    assert (res["tensor"][0].logp - res["tensor_1cta"][0].logp).abs().max() <= 1e-5
    assert rel_l2(res["tensor"][1].float().cpu().numpy(), res["tensor_1cta"][1].float().cpu().numpy()) <= 1e-3


# --------------------------------------------------------------------------- decision stage, bit exact
@pytest.mark.parametrize("mode,mpt,scope", [("sais", "dynamic", "per_seq"), ("sais", "always", "per_seq"),
                                            ("pois", "dynamic", "batch"), ("sais", "dynamic", "supplied"),
                                            ("sais", "off", "per_seq")])
def test_decide_bit_exact_on_oracle_logp(mode, mpt, scope):
    """Feed the elementwise kernel the oracle's float32 log-probs and entropies: flags and counts
    must match bit for bit, values to float32 rounding."""
    rng = np.random.default_rng(12)
    T, S = 5000, 7
    cuts = np.sort(rng.choice(np.arange(1, T), size=S - 1, replace=False))
    offsets = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    logp = (-np.abs(rng.standard_normal(T)) * 0.02).astype(np.float32)        # many tokens near ln(0.99)
    logp[rng.random(T) < 0.3] -= np.float32(3.0)
    ent = np.abs(rng.standard_normal(T)).astype(np.float32) * 0.25
    old = (logp + rng.standard_normal(T).astype(np.float32) * 0.15).astype(np.float32)
    adv = rng.choice(np.float32([1.0, -1.0, 0.0, 0.7]), size=S).astype(np.float32)
    version = rng.integers(0, 9, size=T).astype(np.int32)
    supplied = rng.random(S).astype(np.float32) * 0.4
    kw = dict(is_mode=mode, mpt_mode=mpt, ent_scope=scope, entropy_target=0.2, current_version=8,
              clip_eps_low=0.2, clip_eps_high=0.28)
    op = O.OracleParams(**kw)
    gp = B.Params(T=T, H=8, V=16, num_seqs=S, dtype="f32", **kw)
    gate = O.gate_entropy(ent, offsets, scope, supplied)
    ref = O.decide(logp, gate, old, adv, offsets, version, op)
    t = lambda x: torch.from_numpy(x).to(DEV)
    out = B.token_loss_decide(gp, t(logp), t(ent), t(old), t(version), t(adv), t(offsets),
                              entropy_supplied=t(supplied))
    torch.cuda.synchronize()
    assert np.array_equal(out.flags.cpu().numpy(), ref["flags"])
    st = out.stats_host()
    for k in STAT_KEYS:
        assert st[k] == ref["stats"][k], k
    assert st["stale_tokens"] == ref["stats"]["stale_tokens"].tolist()
    assert st["stale_clipped"] == ref["stats"]["stale_clipped"].tolist()
    assert np.allclose(out.grad_coef.cpu().numpy(), ref["grad_coef"], rtol=1e-6, atol=0)
    assert abs(float(out.loss.cpu()[0]) - ref["loss"]) <= 1e-6 * max(1.0, abs(ref["loss"]))
    seq_mean, batch_mean = O.sequence_mean_entropy(ent, offsets)
    assert np.allclose(out.seq_entropy.cpu().numpy()[:S], seq_mean, rtol=1e-6)
    assert abs(st["mean_entropy"] - batch_mean) <= 1e-6
    if mpt != "off":
        assert ref["stats"]["n_masked"] > 0
    if mode == "sais":
        assert ref["stats"]["n_clip_high"] > 0 and ref["stats"]["n_clip_low"] > 0


# --------------------------------------------------------------------------- edge cases
def test_single_token_and_length_one_sequences():
    wl = synth.WORKLOADS["small"].scaled(T=3, S=3, H=64, V=256, lengths="tiny", segment_len=1)
    batch = synth.make_batch(wl, seed=2)
    gp, op = both_params(batch)
    check_against_oracle(batch, gp, op)
    wl1 = synth.WORKLOADS["tiny"].scaled(T=1, S=1, H=64, V=100, lengths="single")
    b1 = synth.make_batch(wl1, seed=4)
    gp, op = both_params(b1)
    check_against_oracle(b1, gp, op)


def test_all_tokens_masked_gives_zero_loss_and_gradients():
    wl = synth.WORKLOADS["small"].scaled(T=300, S=2, H=128, V=1024, lengths="tiny", planted=1.0,
                                         beta_planted=(400.0, 500.0), adv="plus1", mpt_mode="always")
    batch = synth.make_batch(wl, seed=6)
    gp, op = both_params(batch)
    out, dH, dW = gpu_fwd_bwd(batch, gp)
    st = out.stats_host()
    assert st["n_masked"] == 300 and st["n_active"] == 0
    assert float(out.loss.cpu()[0]) == 0.0
    assert float(dH.float().abs().max()) == 0.0 and float(dW.abs().max()) == 0.0


def test_zero_advantage_sequences_contribute_nothing():
    wl = synth.WORKLOADS["small"].scaled(T=256, S=4, H=128, V=512, lengths="tiny", adv="bern:0.0:4")
    batch = synth.make_batch(wl, seed=8)
    assert float(batch.advantages.abs().max()) == 0.0
    gp, op = both_params(batch)
    out, dH, dW = gpu_fwd_bwd(batch, gp)
    assert float(out.loss.cpu()[0]) == 0.0 and out.stats_host()["n_active"] == 0
    assert float(dW.abs().max()) == 0.0


def test_target_in_last_vocabulary_column_and_tail_tile():
    wl = synth.WORKLOADS["small"].scaled(T=200, S=2, H=128, V=1187, lengths="tiny")
    batch = synth.make_batch(wl, seed=10)
    batch.targets[::3] = 1186
    batch.targets[1::3] = 1024
    gp, op = both_params(batch)
    check_against_oracle(batch, gp, op)


def test_dw_accumulate_and_panel_additivity():
    wl = synth.WORKLOADS["small"].scaled(T=600, S=3, H=128, V=1500, lengths="tiny")
    batch = synth.make_batch(wl, seed=14)
    gp1, _ = both_params(batch, bwd_panel_tokens=128)
    gp2, _ = both_params(batch, bwd_panel_tokens=1024)
    _, dH1, dW1 = gpu_fwd_bwd(batch, gp1)
    _, dH2, dW2 = gpu_fwd_bwd(batch, gp2)
    assert torch.equal(dH1, dH2)
    assert rel_l2(dW1.cpu().numpy(), dW2.cpu().numpy()) <= 1e-5
    gp3, _ = both_params(batch, dw_accumulate=True)
    b = batch.to(DEV)
    out = B.token_loss_fwd(gp3, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets)
    dW = torch.ones(wl.V, wl.H, dtype=torch.float32, device=DEV)
    B.token_loss_bwd(gp3, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_W=dW)
    assert rel_l2((dW - 1.0).cpu().numpy(), dW2.cpu().numpy()) <= 1e-4


def test_empty_batch_and_bad_arguments():
    p = B.Params(T=0, H=64, V=128, num_seqs=0, dtype="bf16")
    ws = torch.empty(B.workspace_bytes(p), dtype=torch.uint8, device=DEV)
    e = lambda n, dt=torch.float32: torch.zeros(n, dtype=dt, device=DEV)
    out = B.token_loss_fwd(p, e(0, torch.bfloat16).reshape(0, 64), e(128 * 64, torch.bfloat16), e(0, torch.int32),
                           e(0), e(0, torch.int32), e(0), e(1, torch.int32), workspace=ws)
    torch.cuda.synchronize()
    assert float(out.loss.cpu()[0]) == 0.0
    bad = B.Params(T=8, H=60, V=128, num_seqs=1, dtype="bf16")           # H not a multiple of 8
    with pytest.raises(B.UlorlError):
        B.workspace_bytes(bad)
    ok = B.Params(T=8, H=64, V=128, num_seqs=1, dtype="bf16")
    small_ws = torch.empty(16, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.UlorlError, match="workspace"):
        B.token_loss_fwd(ok, e(8 * 64, torch.bfloat16), e(128 * 64, torch.bfloat16), e(8, torch.int32), e(8),
                         e(8, torch.int32), e(1), torch.tensor([0, 8], dtype=torch.int32, device=DEV),
                         workspace=small_ws)


def test_out_of_range_target_is_clamped_and_reported():
    wl = synth.WORKLOADS["small"].scaled(T=130, S=1, H=64, V=300, lengths="single")
    batch = synth.make_batch(wl, seed=16)
    batch.targets[5] = 300
    batch.targets[77] = -4
    for path in ("tensor", "simt"):
        gp, _ = both_params(batch, kernel_path=path)
        b = batch.to(DEV)
        ws = B.alloc_workspace(gp, DEV)
        out = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages,
                               b.seq_offsets, workspace=ws)
        assert B.check_status(ws) == -6
        assert torch.isfinite(out.logp).all()


def test_repeated_runs_are_bit_identical():
    wl = synth.WORKLOADS["small"].scaled(T=900, S=4, H=256, V=4000, lengths="tiny")
    batch = synth.make_batch(wl, seed=18)
    gp, _ = both_params(batch)
    a = gpu_fwd_bwd(batch, gp)
    b = gpu_fwd_bwd(batch, gp)
    assert torch.equal(a[0].logp, b[0].logp) and torch.equal(a[0].loss, b[0].loss)
    assert torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])


# --------------------------------------------------------------------------- active-row compaction
@pytest.mark.parametrize("panel,path", [(0, "auto"), (256, "auto"), (256, "tensor_1cta")])
def test_compacted_backward_matches_dense_and_oracle(panel, path):
    """Rows with a zero coefficient (masked, clipped, zero advantage) are dropped from the backward
    contractions; the gradients must not change."""
    wl = synth.WORKLOADS["small"].scaled(T=1500, S=6, H=256, V=3000, lengths="lognormal:200:500", segment_len=64,
                                         planted=0.5, beta_planted=(100.0, 220.0), mpt_mode="always",
                                         noise="const:0.15", adv="bern:0.5:3")
    batch = synth.make_batch(wl, seed=33)
    gp_d, op = both_params(batch, bwd_panel_tokens=panel, kernel_path=path)
    gp_c, _ = both_params(batch, bwd_panel_tokens=panel, compact_rows=True, kernel_path=path)
    out_d, dH_d, dW_d = gpu_fwd_bwd(batch, gp_d)
    out_c, dH_c, dW_c = gpu_fwd_bwd(batch, gp_c)
    st = out_c.stats_host()
    assert 0 < st["n_active"] < wl.T - 100 and st["n_masked"] > 20 and st["n_clip_high"] + st["n_clip_low"] > 0
    assert torch.equal(out_d.grad_coef, out_c.grad_coef)
    assert torch.equal(dH_d, dH_c)                       # a row's reduction over V does not depend on its position
    assert rel_l2(dW_c.cpu().numpy(), dW_d.cpu().numpy()) <= 1e-5
    inactive = (out_c.grad_coef == 0)
    assert float(dH_c[inactive].float().abs().max()) == 0.0
    check_against_oracle(batch, gp_c, op)


def test_compacted_backward_with_nothing_active_and_with_accumulation():
    wl = synth.WORKLOADS["small"].scaled(T=300, S=2, H=128, V=1024, lengths="tiny", planted=1.0,
                                         beta_planted=(400.0, 500.0), adv="plus1", mpt_mode="always")
    batch = synth.make_batch(wl, seed=6)
    gp, _ = both_params(batch, compact_rows=True)
    out, dH, dW = gpu_fwd_bwd(batch, gp)
    assert out.stats_host()["n_active"] == 0
    assert float(dH.float().abs().max()) == 0.0 and float(dW.abs().max()) == 0.0
    # accumulation into a caller's d_W
    wl2 = synth.WORKLOADS["small"].scaled(T=600, S=3, H=128, V=1500, lengths="tiny", planted=0.4,
                                          beta_planted=(300.0, 500.0), mpt_mode="always")
    b2 = synth.make_batch(wl2, seed=14)
    gp_d, _ = both_params(b2)
    gp_a, _ = both_params(b2, compact_rows=True, dw_accumulate=True)
    _, _, dW_ref = gpu_fwd_bwd(b2, gp_d)
    b = b2.to(DEV)
    ws = B.alloc_workspace(gp_a, DEV)
    out = B.token_loss_fwd(gp_a, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets,
                           workspace=ws)
    dW = torch.ones(wl2.V, wl2.H, dtype=torch.float32, device=DEV)
    B.token_loss_bwd(gp_a, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_W=dW, workspace=ws)
    assert rel_l2((dW - 1.0).cpu().numpy(), dW_ref.cpu().numpy()) <= 1e-4


# --------------------------------------------------------------------------- bf16 d_W, d_W slab by slab
@pytest.mark.parametrize("path,panel,compact", [("tensor", 0, False), ("tensor", 384, False), ("tensor", 384, True),
                                                ("tensor_1cta", 384, False), ("simt", 384, False)])
def test_bf16_dw_output_matches_the_oracle_and_the_rounded_f32_result(path, panel, compact):
    """dw_dtype = bf16: the sum over tokens is still taken in float32 and rounded once when final, so the
    result is the float32 d_W rounded to bf16 (bit for bit), and it keeps the gradient tolerance to the oracle."""
    wl = synth.WORKLOADS["small"].scaled(T=700, S=5, H=328, V=3001, lengths="lognormal:100:400",
                                         segment_len=64, planted=0.3, beta_planted=(80.0, 160.0),
                                         mpt_mode="dynamic", entropy_target=6.0)
    batch = synth.make_batch(wl, seed=5)
    import dataclasses
    gp32, op = both_params(batch, kernel_path=path, bwd_panel_tokens=panel, compact_rows=compact)
    gp16 = dataclasses.replace(gp32, dw_dtype="bf16")
    assert B.workspace_bytes(gp16) >= B.workspace_bytes(gp32) + 4 * wl.V * wl.H
    out, dH32, dW32 = gpu_fwd_bwd(batch, gp32)
    _, dH16, dW16 = gpu_fwd_bwd(batch, gp16)
    assert dW16.dtype == torch.bfloat16 and torch.equal(dH16, dH32)
    assert torch.equal(dW16, dW32.to(torch.bfloat16))
    oi = oracle_inputs(batch)
    _, dW_ref = O.backward(oi["hidden"], oi["W"], oi["targets"], out.grad_coef.cpu().numpy().astype(np.float64))
    assert rel_l2(dW16.float().cpu().numpy(), dW_ref) <= TOL_GRAD
    # accumulation into the caller's bf16 array: old + sum, rounded once
    gp_acc = dataclasses.replace(gp16, dw_accumulate=True)
    b = batch.to(DEV)
    ws = B.alloc_workspace(gp_acc, DEV)
    old = (torch.randn(wl.V, wl.H, device=DEV) * dW32.abs().mean()).to(torch.bfloat16)
    dW = old.clone()
    B.token_loss_bwd(gp_acc, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_W=dW, workspace=ws)
    assert torch.equal(dW, (old.float() + dW32).to(torch.bfloat16))


@pytest.mark.parametrize("path,V,panel,dw_dtype,compact", [("tensor", 40000, 512, "f32", False),
                                                           ("tensor", 40000, 512, "bf16", False),
                                                           ("tensor", 40000, 512, "f32", True),
                                                           ("tensor", 2500, 0, "f32", False),
                                                           ("simt", 2500, 256, "f32", False)])
def test_backward_reports_dw_slab_by_slab(path, V, panel, dw_dtype, compact):
    """ulorl_token_loss_bwd_slabs: the callback sees ascending slabs that cover [0, V) once, the rows it is told
    about are final when the work queued before the callback has run (an event recorded inside the callback
    orders a copy on a second stream), and the results are those of the plain backward bit for bit."""
    wl = synth.WORKLOADS["small"].scaled(T=900, S=4, H=256, V=V, lengths="tiny", planted=0.3,
                                         beta_planted=(100.0, 200.0), mpt_mode="always")
    batch = synth.make_batch(wl, seed=41)
    gp, _ = both_params(batch, kernel_path=path, bwd_panel_tokens=panel, compact_rows=compact)
    import dataclasses
    gp = dataclasses.replace(gp, dw_dtype=dw_dtype)
    out, dH, dW = gpu_fwd_bwd(batch, gp)
    b = batch.to(DEV)
    ws = B.alloc_workspace(gp, DEV)
    dW2 = torch.full((wl.V, wl.H), 7.0, dtype=gp.dw_torch_dtype, device=DEV)
    copy = torch.zeros_like(dW2)
    side = torch.cuda.Stream()
    slabs = []

    def on_slab(first_row, rows):
        slabs.append((first_row, rows))
        ev = torch.cuda.Event()
        ev.record()                                   # behind the launches that make these rows final
        side.wait_event(ev)
        with torch.cuda.stream(side):
            copy[first_row:first_row + rows].copy_(dW2[first_row:first_row + rows], non_blocking=True)

    dH2, _ = B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_W=dW2, workspace=ws,
                              on_dw_slab=on_slab)
    torch.cuda.synchronize()
    assert slabs[0][0] == 0 and sum(r for _, r in slabs) == wl.V
    assert all(slabs[i][0] + slabs[i][1] == slabs[i + 1][0] for i in range(len(slabs) - 1))
    if path == "tensor" and V == 40000:
        assert len(slabs) > 1                          # several waves of vocabulary row tiles
    assert torch.equal(dW2, dW) and torch.equal(dH2, dH) and torch.equal(copy, dW)
    # an exception raised inside the callback stops the pass and reaches the caller
    def boom(first_row, rows):
        raise ValueError("stop here")
    with pytest.raises(ValueError, match="stop here"):
        B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_W=dW2, workspace=ws, on_dw_slab=boom)
    torch.cuda.synchronize()


def test_sequence_entropy_tables_edge_cases():
    """The exact per-sequence entropy tables: identity ids, pieces of one sequence inside one call, ids out of
    range reported and skipped, and the means of an unsplit call reproduced."""
    rng = np.random.default_rng(8)
    T, S = 3000, 5
    ent = torch.from_numpy((rng.random(T) * 3.0).astype(np.float32)).to(DEV)
    off = torch.tensor([0, 10, 10, 1500, 2999, 3000], dtype=torch.int32, device=DEV)     # one empty sequence
    p = B.Params(T=T, H=8, V=16, num_seqs=S, dtype="f32")
    table = B.sequence_entropy_partials(p, ent, off, None, S)
    fixed = np.rint(ent.cpu().numpy().astype(np.float64) * 2.0 ** 34).astype(np.int64)
    o = off.cpu().numpy()
    assert table[:, 0].cpu().tolist() == [int(fixed[o[i]:o[i + 1]].sum()) for i in range(S)]
    assert table[:, 1].cpu().tolist() == np.diff(o).tolist()
    means, batch = B.sequence_entropy_combine(table, None, S, want_batch=True)
    dec = B.token_loss_decide(p, ent.clone(), ent, ent, None, torch.ones(S, device=DEV), off)
    assert torch.equal(means, dec.seq_entropy[:S]) and float(means[1]) == 0.0
    assert float(batch[0]) == dec.stats_host()["mean_entropy"]
    # two pieces of sequence 3 and one of sequence 0 in one call of a 6-sequence step; id 9 is out of range
    ids = torch.tensor([3, 0, 3, 9, 5], dtype=torch.int32, device=DEV)
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    t2 = B.sequence_entropy_partials(p, ent, off, ids, 6, workspace=ws)
    assert t2[3].cpu().tolist() == [int(fixed[0:10].sum() + fixed[10:1500].sum()), 1500]
    assert t2[0].cpu().tolist() == [0, 0] and t2[5].cpu().tolist() == [int(fixed[2999]), 1]
    assert t2[[1, 2, 4]].abs().sum().item() == 0
    assert B.check_status(ws) == -1


# --------------------------------------------------------------------------- host-buffer step, timing aid, bad offsets
@pytest.mark.parametrize("V,panel,compact,dw_dtype", [(2500, 0, False, "f32"), (40000, 512, False, "f32"),
                                                      (40000, 512, True, "f32"), (40000, 512, False, "bf16")])
def test_host_buffer_step_matches_device_calls(V, panel, compact, dw_dtype):
    # the second case has two backward panels and a vocabulary of several d_W slabs: on the last panel the
    # host-buffer step computes d_W slab by slab, ahead of d_hidden, and copies each slab out as it is done
    wl = synth.WORKLOADS["small"].scaled(T=900, S=4, H=256, V=V, lengths="tiny", planted=0.3,
                                         beta_planted=(100.0, 200.0), mpt_mode="always")
    batch = synth.make_batch(wl, seed=41)
    gp, _ = both_params(batch, bwd_panel_tokens=panel, compact_rows=compact)
    import dataclasses
    gp = dataclasses.replace(gp, dw_dtype=dw_dtype)
    out, dH, dW = gpu_fwd_bwd(batch, gp)
    arena = torch.empty(B.host_step_arena_bytes(gp), dtype=torch.uint8, device=DEV)
    pin = lambda t: t.contiguous().pin_memory()
    ho = dict(logp=torch.empty(wl.T).pin_memory(), entropy=torch.empty(wl.T).pin_memory(),
              flags=torch.empty(wl.T, dtype=torch.uint8).pin_memory(), seq_entropy=torch.empty(wl.S).pin_memory(),
              loss=torch.empty(1).pin_memory(), stats=torch.empty(out.stats.numel(), dtype=torch.uint8).pin_memory(),
              d_hidden=torch.empty(wl.T, wl.H, dtype=torch.bfloat16).pin_memory(),
              d_W=torch.empty(wl.V, wl.H, dtype=gp.dw_torch_dtype).pin_memory())
    for _ in range(2):                                   # the arena is reusable across calls
        B.token_loss_step_host(gp, arena, pin(batch.hidden), pin(batch.W), pin(batch.targets), pin(batch.old_logp),
                               pin(batch.segment_version), pin(batch.advantages), pin(batch.seq_offsets), **ho)
        torch.cuda.synchronize()
    assert torch.equal(ho["logp"], out.logp.cpu()) and torch.equal(ho["entropy"], out.entropy.cpu())
    assert torch.equal(ho["flags"], out.flags.cpu()) and torch.equal(ho["loss"], out.loss.cpu())
    assert torch.equal(ho["d_hidden"], dH.cpu()) and torch.equal(ho["d_W"], dW.cpu())
    assert B.decode_stats(ho["stats"]) == out.stats_host()
    with pytest.raises(B.UlorlError, match="workspace"):
        B.token_loss_step_host(gp, arena[:1024], pin(batch.hidden), pin(batch.W), pin(batch.targets),
                               pin(batch.old_logp), pin(batch.segment_version), pin(batch.advantages),
                               pin(batch.seq_offsets), **ho)


@pytest.mark.parametrize("path", ["tensor", "tensor_1cta"])
def test_kernel_timing_counts_the_tensor_core_launches(path):
    wl = synth.WORKLOADS["small"].scaled(T=700, S=2, H=256, V=2048, lengths="tiny")
    batch = synth.make_batch(wl, seed=43)
    gp, _ = both_params(batch, bwd_panel_tokens=256, kernel_path=path)
    n0 = B.launch_count()
    B.kernel_timing_begin()
    gpu_fwd_bwd(batch, gp)
    kt = B.kernel_timing_end()
    panels = -(-wl.T // B_panel_rows(gp))
    assert kt["stats"][1] == 1 and kt["dz"][1] == panels and kt["d_hidden"][1] == panels and kt["d_W"][1] == panels
    assert all(ms > 0 for ms, n in kt.values())
    assert B.launch_count() - n0 == 1 + 1 + 4 + 3 * panels      # stats, merge, decision stage (4), three per panel


def B_panel_rows(gp):
    # panels are whole row tiles of the kernels in use (256 tokens for CTA pairs, 128 otherwise)
    unit = 128 if gp.kernel_path == "tensor_1cta" else 256
    return -(-gp.bwd_panel_tokens // unit) * unit


def test_inconsistent_sequence_offsets_are_reported_not_followed():
    wl = synth.WORKLOADS["small"].scaled(T=300, S=3, H=64, V=512, lengths="tiny")
    batch = synth.make_batch(wl, seed=45)
    gp, _ = both_params(batch)
    b = batch.to(DEV)
    ws = B.alloc_workspace(gp, DEV)
    bad = b.seq_offsets.clone()
    bad[2] = 5000                                        # beyond T
    out = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, bad,
                           workspace=ws)
    assert B.check_status(ws) == -1
    assert torch.isfinite(out.seq_entropy).all()
    out = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets,
                           workspace=ws)
    assert B.check_status(ws) == B.OK


def test_group_advantages_match_the_oracle():
    rng = np.random.default_rng(3)
    for S, G, p in ((1024, 8, 0.3), (37, 16, 0.5), (5, 8, 0.9), (64, 4, 0.0)):
        r = (rng.random(S) < p).astype(np.float32)
        adv, keep = B.group_advantages(torch.from_numpy(r).to(DEV), G)
        ref_adv, ref_keep = O.group_advantages(r, G)
        assert np.array_equal(keep.cpu().numpy(), ref_keep)
        assert np.allclose(adv.cpu().numpy(), ref_adv, rtol=1e-6, atol=1e-7)


def test_token_range_split_with_entropy_exchange_matches_the_unsplit_batch():
    """Two token ranges of one batch, run one after the other as two ranks would run them: forward on each
    range, the library's exact per-sequence (entropy sum, count) tables added as an int64 all-reduce would add
    them, the means taken on the device, decision stage with the means supplied, backward accumulating into
    one d_W.  The mean entropy of every sequence is the unsplit run's bit for bit, so with sigma one float32
    step above, at, and one step below a split sequence's H-bar the flags, loss and gradients equal the
    unsplit run's."""
    import dataclasses
    from paper_2507_19766_b200 import dp
    wl = synth.WORKLOADS["small"].scaled(T=1500, S=4, H=128, V=1500, lengths="fixed:700,400,300,100", planted=0.6,
                                         beta_planted=(200.0, 450.0), mpt_mode="dynamic", adv="bern:0.5:3")
    batch = synth.make_batch(wl, seed=26)
    gp0, op0 = both_params(batch)
    oi = oracle_inputs(batch)
    ref = O.forward(oi["hidden"], oi["W"], oi["targets"], oi["old_logp"], oi["segment_version"], oi["advantages"],
                    oi["seq_offsets"], op0)
    b = batch.to(DEV)
    off = batch.seq_offsets.numpy()
    ranges = dp.shard_token_ranges(wl.T, 2, align=256)
    assert ranges == [(0, 768), (768, 1500)]                   # sequence 1 (tokens 700..1100) is split
    base, _, _ = gpu_fwd_bwd(batch, gp0)
    hbar = base.seq_entropy.cpu().numpy()[:wl.S].astype(np.float32)
    assert np.abs(hbar - ref["seq_entropy"]).max() <= TOL_LOGP
    split_seq = 1
    up, down = np.nextafter(hbar[split_seq], np.float32(np.inf)), np.nextafter(hbar[split_seq], np.float32(-np.inf))
    masked_counts = []
    for sigma in (float(up), float(hbar[split_seq]), float(down)):
        gp, _ = both_params(batch, entropy_target=sigma)
        full, dH_full, dW_full = gpu_fwd_bwd(batch, gp)
        pieces = []
        table = torch.zeros(wl.S, 2, dtype=torch.int64, device=DEV)
        for lo, hi in ranges:
            ids, loff = dp.local_sequence_pieces(off, lo, hi)
            lp = dataclasses.replace(gp, T=hi - lo, num_seqs=len(ids), norm_tokens=wl.T, ent_scope="supplied",
                                     dw_accumulate=True)
            loff_t = torch.tensor(loff, dtype=torch.int32, device=DEV)
            ids_t = torch.tensor(ids, dtype=torch.int32, device=DEV)
            adv = b.advantages[ids_t.long()].contiguous()
            dummy = torch.zeros(len(ids), dtype=torch.float32, device=DEV)
            sl = slice(lo, hi)
            f = B.token_loss_fwd(lp, b.hidden[sl], b.W, b.targets[sl], b.old_logp[sl], b.segment_version[sl], adv,
                                 loff_t, entropy_supplied=dummy)
            table += B.sequence_entropy_partials(lp, f.entropy, loff_t, ids_t, wl.S)   # what the all-reduce sums
            pieces.append((sl, ids_t, lp, loff_t, adv, f))
        dp.all_reduce_sequence_entropy(table)                   # no process group here: returns the table as is
        dW = torch.zeros(wl.V, wl.H, dtype=torch.float32, device=DEV)
        dH = torch.empty_like(b.hidden)
        loss, flags = 0.0, np.zeros(wl.T, dtype=np.uint8)
        for sl, ids_t, lp, loff_t, adv, f in pieces:
            gate = B.sequence_entropy_combine(table, ids_t, ids_t.numel())
            d = B.token_loss_decide(lp, f.logp, f.entropy, b.old_logp[sl], b.segment_version[sl], adv, loff_t,
                                    entropy_supplied=gate)
            B.token_loss_bwd(lp, b.hidden[sl], b.W, b.targets[sl], f.lse, d.grad_coef, d_hidden=dH[sl], d_W=dW)
            loss += float(d.loss.cpu()[0])
            flags[sl] = d.flags.cpu().numpy()
        torch.cuda.synchronize()
        gate_all, batch_mean = B.sequence_entropy_combine(table, None, wl.S, want_batch=True)
        assert torch.equal(gate_all, full.seq_entropy[:wl.S])      # bit for bit, split or not
        assert float(batch_mean.cpu()[0]) == full.stats_host()["mean_entropy"]
        assert table[:, 1].cpu().tolist() == np.diff(off).tolist()
        assert np.array_equal(flags, full.flags.cpu().numpy())
        assert abs(loss - float(full.loss.cpu()[0])) <= 1e-5 * max(1e-3, abs(loss))
        assert torch.equal(dH, dH_full)                            # rows are independent of the split
        assert rel_l2(dW.cpu().numpy(), dW_full.cpu().numpy()) <= 1e-4
        seq_of = np.repeat(np.arange(wl.S), np.diff(off))
        masked_counts.append(int(((flags & O.FLAG_MASKED) != 0)[seq_of == split_seq].sum()))
    # one float32 step of sigma across the split sequence's H-bar opens and shuts its gate (H-bar < sigma, strict)
    assert masked_counts[0] > 0 and masked_counts[1] == 0 and masked_counts[2] == 0


@pytest.mark.parametrize("path,norm_seqs", [("tensor", 0), ("simt", 9)])
def test_per_sample_normalisation_matches_the_oracle(path, norm_seqs):
    """Eq. 5's (1/G) sum_i (1/|o_i|) weights instead of Eq. 10's 1/N: loss, coefficients and both gradients
    against the oracle on ragged sequence lengths; the decisions are those of the token-normalised run."""
    wl = synth.WORKLOADS["small"].scaled(T=700, S=5, H=328, V=3001, lengths="lognormal:100:400",
                                         segment_len=64, planted=0.3, beta_planted=(80.0, 160.0),
                                         mpt_mode="dynamic", entropy_target=6.0)
    batch = synth.make_batch(wl, seed=5)
    gp, op = both_params(batch, kernel_path=path, loss_norm="sequence", norm_seqs=norm_seqs)
    out, ref = check_against_oracle(batch, gp, op)
    gp_t, _ = both_params(batch, kernel_path=path)
    out_t, _, _ = gpu_fwd_bwd(batch, gp_t)
    assert torch.equal(out.flags, out_t.flags)
    lens = np.diff(batch.seq_offsets.numpy())
    G = norm_seqs if norm_seqs else wl.S
    scale = np.repeat(wl.T / (G * lens.astype(np.float64)), lens)          # (1/(G|o_i|)) / (1/T)
    assert np.allclose(out.grad_coef.cpu().numpy(), out_t.grad_coef.cpu().numpy() * scale, rtol=1e-6, atol=1e-12)


def test_slab_wise_all_reduce_on_a_one_rank_nccl_group():
    """The data-parallel step as bench.py runs it, on a process group of one rank: the backward hands d_W to
    dp.SlabAllReduce slab by slab, each slab is all-reduced asynchronously on the backend's stream behind the
    launches that made it final, and finish() joins them.  With one rank the sum is the rank's own d_W, which
    must be the plain backward's bit for bit; what this exercises is the ordering between the compute stream
    and the collective's stream."""
    import torch.distributed as dist
    from paper_2507_19766_b200 import dp
    wl = synth.WORKLOADS["small"].scaled(T=900, S=4, H=256, V=40000, lengths="tiny", planted=0.3,
                                         beta_planted=(100.0, 200.0), mpt_mode="always")
    batch = synth.make_batch(wl, seed=41)
    gp, _ = both_params(batch, bwd_panel_tokens=512)
    out, dH, dW = gpu_fwd_bwd(batch, gp)
    b = batch.to(DEV)
    ws = B.alloc_workspace(gp, DEV)
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{dp.free_port()}", rank=0, world_size=1,
                                device_id=torch.device(DEV))
    try:
        dW2 = torch.full((wl.V, wl.H), 3.0, device=DEV)
        red = dp.SlabAllReduce(dW2)
        red.active = True                    # a one-rank group would otherwise skip the collective
        dH2, _ = B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_W=dW2, workspace=ws,
                                  on_dw_slab=red)
        assert len(red.works) > 1
        covered = red.finish()
        torch.cuda.synchronize()
        assert covered[0][0] == 0 and sum(r for _, r in covered) == wl.V
        assert torch.equal(dW2, dW) and torch.equal(dH2, dH)
    finally:
        if created:
            dist.destroy_process_group()


def test_zz_report_colsum_margins():
    """Not a check of its own: prints how close the d_W column sums came to their statistical bound."""
    if COLSUM_MARGINS:
        print(f"d_W column sums: largest fraction of the statistical bound over {len(COLSUM_MARGINS)} cases = "
              f"{max(COLSUM_MARGINS):.3f}")
        assert max(COLSUM_MARGINS) <= 1.0


def test_decision_stage_on_unaligned_arrays_matches_the_vector_path():
    """The decision kernel moves a thread's four tokens as one 128-bit vector when every per-token array is
    16-byte aligned; arrays that start one element into an allocation take the scalar accesses.  Same flags,
    coefficients, loss and statistics, with per-token advantages and a ragged token count."""
    rng = np.random.default_rng(19)
    T, S = 4099, 5
    cuts = np.sort(rng.choice(np.arange(1, T), size=S - 1, replace=False))
    offsets = torch.from_numpy(np.concatenate([[0], cuts, [T]]).astype(np.int32)).to(DEV)
    mk = lambda x: torch.from_numpy(x).to(DEV)
    logp = mk((-np.abs(rng.standard_normal(T + 1)) * 0.02).astype(np.float32))
    ent = mk((np.abs(rng.standard_normal(T + 1)) * 0.25).astype(np.float32))
    old = mk((logp.cpu().numpy() + rng.standard_normal(T + 1).astype(np.float32) * 0.15).astype(np.float32))
    ver = mk(rng.integers(0, 6, size=T + 1).astype(np.int32))
    adv = mk(rng.choice(np.float32([1.0, -1.0, 0.0, 0.6]), size=T + 1).astype(np.float32))
    p = B.Params(T=T, H=8, V=16, num_seqs=S, dtype="f32", adv_per_token=True, current_version=5, entropy_target=0.2)
    outs = []
    for shift in (0, 1):
        cut = lambda x: x[1:] if shift else x[1:].clone()          # same values; the clone starts aligned
        o = B.alloc_fwd_outputs(p, DEV)
        if shift:
            o.grad_coef = torch.empty(T + 1, device=DEV)[1:]
            o.flags = torch.empty(T + 1, dtype=torch.uint8, device=DEV)[1:]
        outs.append(B.token_loss_decide(p, cut(logp), cut(ent), cut(old), cut(ver), cut(adv), offsets, out=o))
    torch.cuda.synchronize()
    a, b = outs
    assert torch.equal(a.flags, b.flags) and torch.equal(a.grad_coef, b.grad_coef) and torch.equal(a.loss, b.loss)
    assert a.stats_host() == b.stats_host()
    ref = O.decide(logp.cpu().numpy()[1:], O.gate_entropy(ent.cpu().numpy()[1:], offsets.cpu().numpy(), "per_seq", None),
                   old.cpu().numpy()[1:], adv.cpu().numpy()[1:], offsets.cpu().numpy(), ver.cpu().numpy()[1:],
                   O.OracleParams(current_version=5, entropy_target=0.2), adv_per_token=True)
    assert np.array_equal(a.flags.cpu().numpy(), ref["flags"])
    for k in STAT_KEYS:
        assert a.stats_host()[k] == ref["stats"][k], k


# --------------------------------------------------------------------------- KL-to-reference term of Eq. 5
def kl_reference(batch, seed):
    """A recorded reference log-prob per token: the rollout record moved by N(0, 0.3)."""
    rng = np.random.default_rng(seed)
    return (batch.old_logp.numpy() + 0.3 * rng.standard_normal(batch.workload.T).astype(np.float32)).astype(np.float32)


@pytest.mark.parametrize("path,loss_norm", [("tensor", "tokens"), ("simt", "sequence")])
def test_kl_term_matches_the_oracle(path, loss_norm):
    """Eq. 5's objective s - beta k through the whole path: forward (loss, coefficients, mean KL) and both
    gradients against the oracle; the decision kernel on the oracle's float32 log-probs to 2e-6."""
    wl = synth.WORKLOADS["small"].scaled(T=700, S=5, H=328, V=3001, lengths="lognormal:100:400", segment_len=64,
                                         planted=0.3, beta_planted=(80.0, 160.0), mpt_mode="always")
    batch = synth.make_batch(wl, seed=5)
    ref_lp = kl_reference(batch, 77)
    gp, op = both_params(batch, kernel_path=path, kl_beta=0.25, loss_norm=loss_norm)
    oi = oracle_inputs(batch)
    ref = O.fwd_bwd(oi["hidden"], oi["W"], oi["targets"], oi["old_logp"], oi["segment_version"], oi["advantages"],
                    oi["seq_offsets"], op, ref_logp=ref_lp)
    b = batch.to(DEV)
    rl = torch.from_numpy(ref_lp).to(DEV)
    ws = B.alloc_workspace(gp, DEV)
    out = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets,
                           workspace=ws, ref_logp=rl)
    torch.cuda.synchronize()
    near = near_threshold(ref["logp"], oi["old_logp"], ref["seq_entropy"], oi["seq_offsets"], op)
    differ = out.flags.cpu().numpy() != ref["flags"]
    assert not (differ & ~near).any()
    st = out.stats_host()
    assert abs(st["mean_kl"] - ref["stats"]["mean_kl"]) <= 1e-3 * max(ref["stats"]["mean_kl"], 1e-3)
    assert ref["stats"]["mean_kl"] > 0.01 and ref["stats"]["n_clip_high"] + ref["stats"]["n_clip_low"] > 0
    # the oracle's float32 log-probs through the decision kernel: same decisions, coefficients and loss to float32
    t32 = lambda x: torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(DEV)
    dec = B.token_loss_decide(gp, t32(ref["logp"]), t32(ref["entropy"]), b.old_logp, b.segment_version, b.advantages,
                              b.seq_offsets, ref_logp=rl)
    assert np.array_equal(dec.flags.cpu().numpy(), ref["flags"])
    assert np.allclose(dec.grad_coef.cpu().numpy(), ref["grad_coef"], rtol=2e-6, atol=1e-12)
    assert abs(float(dec.loss.cpu()[0]) - ref["loss"]) <= 2e-6 * max(1.0, abs(ref["loss"]))
    assert abs(dec.stats_host()["mean_kl"] - ref["stats"]["mean_kl"]) <= 1e-6
    assert dec.stats_host()["n_active"] == ref["stats"]["n_active"]
    # clipped tokens are active now (their KL gradient flows); masked ones are not
    clipped = (ref["flags"] & (O.FLAG_CLIP_HIGH | O.FLAG_CLIP_LOW)) != 0
    masked = (ref["flags"] & O.FLAG_MASKED) != 0
    g = dec.grad_coef.cpu().numpy()
    assert (g[clipped & ~masked] != 0).all() and (g[masked] == 0).all()
    # backward on the oracle's coefficients
    dH, dW = B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, t32(ref["grad_coef"]), workspace=ws)
    torch.cuda.synchronize()
    assert rel_l2(dH.float().cpu().numpy(), ref["d_hidden"]) <= TOL_GRAD
    assert rel_l2(dW.cpu().numpy(), ref["d_W"]) <= TOL_GRAD
    if not differ.any():
        assert abs(float(out.loss.cpu()[0]) - ref["loss"]) <= TOL_LOSS * max(abs(ref["loss"]), 1e-3)
    # beta > 0 without a reference is refused; beta = 0 ignores one
    with pytest.raises(B.UlorlError):
        B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets,
                         workspace=ws)
    gp0, _ = both_params(batch, kernel_path=path, loss_norm=loss_norm)
    a0 = B.token_loss_fwd(gp0, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets)
    a1 = B.token_loss_fwd(gp0, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets,
                          ref_logp=rl)
    assert torch.equal(a0.grad_coef, a1.grad_coef) and torch.equal(a0.loss, a1.loss) and a1.stats_host()["mean_kl"] == 0.0


def test_kl_term_through_the_host_buffer_step():
    wl = synth.WORKLOADS["small"].scaled(T=900, S=4, H=256, V=2500, lengths="tiny", planted=0.3,
                                         beta_planted=(100.0, 200.0), mpt_mode="always")
    batch = synth.make_batch(wl, seed=41)
    ref_lp = kl_reference(batch, 78)
    gp, _ = both_params(batch, kl_beta=0.1)
    b = batch.to(DEV)
    ws = B.alloc_workspace(gp, DEV)
    out = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets,
                           workspace=ws, ref_logp=torch.from_numpy(ref_lp).to(DEV))
    dH, dW = B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, workspace=ws)
    arena = torch.empty(B.host_step_arena_bytes(gp), dtype=torch.uint8, device=DEV)
    pin = lambda t: t.contiguous().pin_memory()
    ho = dict(loss=torch.empty(1).pin_memory(), stats=torch.empty(out.stats.numel(), dtype=torch.uint8).pin_memory(),
              d_hidden=torch.empty(wl.T, wl.H, dtype=torch.bfloat16).pin_memory(), d_W=torch.empty(wl.V, wl.H).pin_memory())
    B.token_loss_step_host(gp, arena, pin(batch.hidden), pin(batch.W), pin(batch.targets), pin(batch.old_logp),
                           pin(batch.segment_version), pin(batch.advantages), pin(batch.seq_offsets),
                           ref_logp=pin(torch.from_numpy(ref_lp)), **ho)
    torch.cuda.synchronize()
    assert torch.equal(ho["loss"], out.loss.cpu()) and torch.equal(ho["d_W"], dW.cpu()) and torch.equal(ho["d_hidden"], dH.cpu())
    assert B.decode_stats(ho["stats"]) == out.stats_host() and out.stats_host()["mean_kl"] > 0

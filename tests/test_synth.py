"""The workload generator: determinism and the structure the recipes promise."""
import numpy as np
import pytest

from workloads import synth


def test_batches_are_a_pure_function_of_workload_and_seed():
    wl = synth.WORKLOADS["tiny"]
    a, b = synth.make_batch(wl), synth.make_batch(wl)
    for k in ("hidden", "W", "targets", "old_logp", "segment_version", "advantages", "seq_offsets"):
        assert (getattr(a, k) == getattr(b, k)).all()
    c = synth.make_batch(wl, seed=1)
    assert not (a.hidden == c.hidden).all()


def test_tiny_structure():
    b = synth.make_batch(synth.WORKLOADS["tiny"])
    assert b.seq_offsets.tolist() == [0, 64, 160, 288, 512]
    assert sorted(b.advantages.tolist()) == [-1.0, -1.0, 1.0, 1.0]
    v = b.segment_version.numpy()
    off = b.seq_offsets.numpy()
    for i in range(4):
        seg = v[off[i]:off[i + 1]]
        assert set(seg.tolist()) == {0, 1} and (np.diff(seg) >= 0).all() and seg[-1] == b.current_version
    assert b.hidden.dtype.is_floating_point and b.hidden.element_size() == 4
    assert 0 <= int(b.targets.min()) and int(b.targets.max()) < 4096


@pytest.mark.parametrize("name,T,S", [("small", 16384, 16), ("qwen", 65536, 32), ("mixed", 262144, 64),
                                      ("ultra", 131072, 1)])
def test_sequence_structure_of_named_workloads(name, T, S):
    wl = synth.WORKLOADS[name]
    rng = np.random.Generator(np.random.Philox(synth.BASE_SEED + wl.index))
    lengths = synth._sequence_lengths(wl, rng)
    assert lengths.sum() == T and lengths.shape[0] == S and lengths.min() >= 1
    version, current = synth._segments(wl, lengths)
    assert version.min() >= 0 and version.max() == current
    pos = 0
    for L in lengths:
        seg = version[pos:pos + L]
        assert (np.diff(seg) >= 0).all() and seg[-1] == current
        pos += L
    if name == "ultra":
        assert np.bincount(version).tolist() == [16384] * 8
    if name == "qwen":
        assert (lengths <= 1024).mean() >= 0.85 and lengths.max() <= 32768 and lengths.max() > 8192
    if name == "mixed":
        assert lengths.max() <= 131072 and np.median(lengths) < lengths.mean()
    if name == "small":
        assert lengths.max() <= 4096


def test_group_normalised_advantages():
    wl = synth.WORKLOADS["small"]
    b = synth.make_batch(wl.scaled(T=2048, H=64, V=512))
    a = b.advantages.numpy().reshape(2, 8)
    for g in a:
        if np.any(g != 0):
            assert abs(g.mean()) < 1e-6 and abs(g.std() - 1.0) < 1e-5
            assert len(set(np.round(g, 5))) == 2          # 0/1 rewards give two advantage values


def test_planted_rows_are_the_argmax_with_high_probability():
    wl = synth.WORKLOADS["small"].scaled(T=400, S=2, H=256, V=2048, lengths="tiny", planted=0.5,
                                         beta_planted=(100.0, 200.0))
    b = synth.make_batch(wl, seed=3)
    logp, amax, _ = synth.rollout_logp(b.hidden, b.W, b.targets)
    planted = b.planted_rows
    assert 120 < planted.sum() < 280
    assert (amax.numpy()[planted] == b.targets.numpy()[planted]).all()
    p = np.exp(logp.numpy())
    assert (p[planted] > 0.5).mean() > 0.9 and (p[~planted] < 0.1).all()
    assert ((p[planted] >= 0.99).sum() > 10) and ((p[planted] < 0.99).sum() > 0)


def test_softmax_sampled_targets_follow_the_row_distribution():
    wl = synth.WORKLOADS["ultra"].scaled(T=512, H=128, V=1024, segment_len=64, planted=0.0, sampled=1.0,
                                         beta_sampled=(150.0, 250.0))
    b = synth.make_batch(wl, seed=5)
    logp, amax, _ = synth.rollout_logp(b.hidden, b.W, b.targets)
    hit = (amax.numpy() == b.targets.numpy()).mean()
    assert 0.5 < hit <= 1.0
    assert np.isfinite(logp.numpy()).all()
    # stale segments carry more old_logp noise, the newest segment none
    v = b.segment_version.numpy()
    assert np.all(b.old_logp_noise[v == b.current_version] == 0)
    assert np.abs(b.old_logp_noise[v == 0]).mean() > np.abs(b.old_logp_noise[v == b.current_version - 1]).mean()

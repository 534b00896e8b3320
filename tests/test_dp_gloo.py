"""The data-parallel decomposition on two CPU ranks (gloo): sequences sharded across ranks, the
global normaliser, and the summed head gradient and loss reproduce the single-process result.  The
per-rank arithmetic here is the oracle's; the GPU path is launched the same way by bench.py."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2507_19766_b200 import dp


def test_shard_sequences_balances_and_covers():
    lengths = [131072, 900, 40000, 17, 65000, 3000, 800, 12000]
    shards = dp.shard_sequences(lengths, 3)
    flat = sorted(i for s in shards for i in s)
    assert flat == list(range(len(lengths)))
    loads = [sum(lengths[i] for i in s) for s in shards]
    assert max(loads) == 131072                       # the longest sequence cannot be split
    assert abs(loads[1] - loads[2]) <= 20000
    assert dp.shard_sequences([5, 5], 2) == [[0], [1]]
    assert dp.shard_sequences([7], 2) == [[0], []]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, result_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import ulorl_oracle as O
        from paper_2507_19766_b200 import synth
        wl = synth.WORKLOADS["small"].scaled(T=96, S=6, H=16, V=64, lengths="lognormal:16:40", segment_len=8,
                                             planted=0.3, beta_planted=(30.0, 60.0), mpt_mode="always")
        batch = synth.make_batch(wl, seed=11)          # every rank builds the same global batch
        off = batch.seq_offsets.numpy()
        lengths = np.diff(off)
        mine = dp.shard_sequences(lengths, world)[rank]
        rows = np.concatenate([np.arange(off[i], off[i + 1]) for i in mine])
        local_off = np.concatenate([[0], np.cumsum(lengths[mine])]).astype(np.int32)
        n_global = dp.global_token_count(rows.size)
        assert n_global == wl.T
        kw = dict(is_mode="sais", mpt_mode="always", current_version=batch.current_version, norm_tokens=n_global)
        h, w = batch.host_f32("hidden"), batch.host_f32("W")
        out = O.fwd_bwd(h[rows], w, batch.targets.numpy()[rows], batch.old_logp.numpy()[rows],
                        batch.segment_version.numpy()[rows], batch.advantages.numpy()[mine], local_off,
                        O.OracleParams(**kw))
        d_W = torch.from_numpy(out["d_W"].copy())
        loss = torch.tensor([out["loss"]], dtype=torch.float64)
        counters = torch.tensor([out["stats"]["n_masked"], out["stats"]["n_active"]], dtype=torch.int64)
        dp.reduce_step_outputs(d_W, loss, counters)
        if rank == 0:
            full = O.fwd_bwd(h, w, batch.targets.numpy(), batch.old_logp.numpy(), batch.segment_version.numpy(),
                             batch.advantages.numpy(), off, O.OracleParams(**dict(kw, norm_tokens=0)))
            assert np.allclose(d_W.numpy(), full["d_W"], rtol=1e-12, atol=1e-15)
            assert abs(float(loss) - full["loss"]) < 1e-14
            assert counters.tolist() == [full["stats"]["n_masked"], full["stats"]["n_active"]]
            assert np.allclose(out["d_hidden"], full["d_hidden"][rows], rtol=1e-12, atol=1e-15)
            open(os.path.join(result_dir, "ok"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_two_rank_data_parallel_matches_single_process(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok").exists()


def _token_range_worker(rank, world, port, result_dir):
    """Token-range sharding: sequences straddle the two ranks; the (sum, count) exchange gives both the
    same per-sequence mean entropy and the dynamic mask, loss and gradients of the unsplit batch."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import ulorl_oracle as O
        from paper_2507_19766_b200 import synth
        wl = synth.WORKLOADS["small"].scaled(T=90, S=3, H=16, V=64, lengths="fixed:50,25,15", segment_len=8,
                                             planted=0.6, beta_planted=(1500.0, 4000.0), mpt_mode="dynamic")   # H = 16: |W_y|^2 is tiny
        batch = synth.make_batch(wl, seed=14)
        off = batch.seq_offsets.numpy()
        lo, hi = dp.shard_token_ranges(wl.T, world, align=8)[rank]
        assert (lo, hi) == ((0, 48), (48, 90))[rank]                 # sequence 0 (50 tokens) is split
        ids, loff = dp.local_sequence_pieces(off, lo, hi)
        assert ids == ([0], [0, 1, 2])[rank]
        rows = np.arange(lo, hi)
        h, w = batch.host_f32("hidden"), batch.host_f32("W")
        tg, ol, sv = batch.targets.numpy(), batch.old_logp.numpy(), batch.segment_version.numpy()
        _, ent, _ = O.token_stats(h[rows], w, tg[rows], 1.0)
        ent32 = ent.astype(np.float32)
        means = torch.tensor([ent32[loff[k]:loff[k + 1]].astype(np.float64).mean() for k in range(len(ids))])
        cnts = torch.tensor(np.diff(loff))
        gate = dp.exchange_sequence_entropy(means, cnts, ids, wl.S).numpy()
        # sigma between the sequences' mean entropies, so that the gate is open for some and shut for others
        full_fwd = O.forward(h, w, tg, ol, sv, batch.advantages.numpy(), off, O.OracleParams())
        hbar = np.sort(full_fwd["seq_entropy"])
        sigma = float(0.5 * (hbar[0] + hbar[1]))
        kw = dict(is_mode="sais", mpt_mode="dynamic", entropy_target=sigma, current_version=batch.current_version)
        out = O.fwd_bwd(h[rows], w, tg[rows], ol[rows], sv[rows], batch.advantages.numpy()[ids],
                        np.asarray(loff, dtype=np.int32), O.OracleParams(ent_scope="supplied", norm_tokens=wl.T, **kw),
                        entropy_supplied=gate)
        d_W = torch.from_numpy(out["d_W"].copy())
        loss = torch.tensor([out["loss"]], dtype=torch.float64)
        counters = torch.tensor([out["stats"]["n_masked"], out["stats"]["n_active"]], dtype=torch.int64)
        dp.reduce_step_outputs(d_W, loss, counters)
        full = O.fwd_bwd(h, w, tg, ol, sv, batch.advantages.numpy(), off, O.OracleParams(**kw))
        assert np.allclose(gate, full["seq_entropy"][ids].astype(np.float32), rtol=1e-6)
        assert np.array_equal(out["flags"], full["flags"][rows])
        assert np.allclose(out["d_hidden"], full["d_hidden"][rows], rtol=1e-12, atol=1e-15)
        # the step-wide gate: both ranks obtain the batch mean entropy of the unsplit call
        step_gate = dp.step_entropy_gate([float(ent32.astype(np.float64).mean())], [rows.size])
        assert abs(step_gate - full["mean_entropy"]) < 1e-12
        if rank == 0:
            assert 0 < full["stats"]["n_masked"] < np.count_nonzero(full["flags"] & O.FLAG_MPT)   # both gate states
            assert np.allclose(d_W.numpy(), full["d_W"], rtol=1e-12, atol=1e-15)
            assert abs(float(loss) - full["loss"]) < 1e-14
            assert counters.tolist() == [full["stats"]["n_masked"], full["stats"]["n_active"]]
            open(os.path.join(result_dir, "ok"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_token_range_sharding_with_entropy_exchange(tmp_path):
    port = _free_port()
    mp.spawn(_token_range_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok").exists()

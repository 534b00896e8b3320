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
        from workloads import synth
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
        from workloads import synth
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
        # the exchange format of the library, restated: per sequence (sum of the float32 entropies in units of
        # 2^-34 nats as int64, token count); integer sums are exact, so the all-reduce reproduces the unsplit sums
        to_fixed = lambda e: np.rint(e.astype(np.float64) * 2.0 ** 34).astype(np.int64)
        table = torch.zeros(wl.S, 2, dtype=torch.int64)
        for k, i in enumerate(ids):
            table[i, 0] = int(to_fixed(ent32[loff[k]:loff[k + 1]]).sum())
            table[i, 1] = int(loff[k + 1] - loff[k])
        dp.all_reduce_sequence_entropy(table)
        _, ent_all, _ = O.token_stats(h, w, tg, 1.0)
        fixed_all = to_fixed(ent_all.astype(np.float32))
        assert table[:, 0].tolist() == [int(fixed_all[off[i]:off[i + 1]].sum()) for i in range(wl.S)]
        assert table[:, 1].tolist() == np.diff(off).tolist()
        gate = (table[ids, 0].numpy().astype(np.float64) * 2.0 ** -34 / table[ids, 1].numpy()).astype(np.float32)
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
        # the step-wide gate: the same summed table gives both ranks the token mean entropy of the unsplit call
        step_gate = float(table[:, 0].sum().item()) * 2.0 ** -34 / float(table[:, 1].sum().item())
        assert abs(step_gate - full["mean_entropy"]) < 1e-9
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


def test_launch_ranks_starts_the_world_it_is_asked_for(tmp_path):
    """bench.py --gpus N starts its own ranks through dp.launch_ranks; here two CPU ranks."""
    import sys
    probe = os.path.join(os.path.dirname(os.path.abspath(__file__)), "rank_probe.py")
    rc = dp.launch_ranks(probe, [str(tmp_path), "2"], 2)
    assert rc == 0
    for r in range(2):
        world, local_rank, total = (tmp_path / f"rank{r}").read_text().split()
        assert (int(world), int(local_rank), int(total)) == (2, r, 3)
    # a launcher whose world differs from what the script was asked for is an error, not a silent 1-rank run
    rc = dp.launch_ranks(probe, [str(tmp_path), "3"], 2)
    assert rc != 0
    os.environ.pop("WORLD_SIZE", None)
    assert dp.world_from_env(4) is None


def _slab_worker(rank, world, port, result_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        V, H = 1000, 24
        for dtype, exact in ((torch.float64, True), (torch.float32, False)):
            g = torch.Generator().manual_seed(100 + rank)
            mine = torch.randn(V, H, generator=g, dtype=torch.float64).to(dtype)
            one_shot = mine.clone()
            dist.all_reduce(one_shot)
            by_slab = mine.clone()
            red = dp.SlabAllReduce(by_slab)
            # the slab schedule of the backward: ascending, covering [0, V) once, last slab ragged
            for v0 in range(0, V, 296):
                red(v0, min(296, V - v0))
            covered = red.finish()
            assert covered == [(0, 296), (296, 296), (592, 296), (888, 112)]
            if exact:
                assert torch.equal(by_slab, one_shot)
            else:
                assert torch.allclose(by_slab, one_shot, rtol=1e-6, atol=0) and torch.equal(by_slab, one_shot)
        if rank == 0:
            open(os.path.join(result_dir, "ok"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_slab_wise_reduction_equals_the_one_shot_sum(tmp_path):
    port = _free_port()
    mp.spawn(_slab_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok").exists()

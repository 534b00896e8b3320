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

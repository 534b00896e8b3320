"""The data-parallel step with two ranks on real device buffers.  Only one GPU is at hand, so both ranks
share cuda:0 and the process group is gloo (which moves CUDA tensors through the host): no kernel of one
rank ever waits for the other, the ranks only meet in host-side collectives.  What this covers that the CPU
tests cannot: the library's own outputs going through the sharding, the global normaliser, the slab-wise
d_W all-reduce started from inside the backward call, and the exact entropy tables of the token-range split,
against the same batch run unsplit on the same GPU."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _batch():
    from workloads import synth
    wl = synth.WORKLOADS["small"].scaled(T=2300, S=7, H=256, V=40000, lengths="lognormal:200:700", segment_len=128,
                                         planted=0.5, beta_planted=(100.0, 220.0), mpt_mode="dynamic",
                                         adv="plus1")
    return wl, synth.make_batch(wl, seed=61)


def _params(B, wl, batch, **kw):
    base = dict(T=wl.T, H=wl.H, V=wl.V, num_seqs=wl.S, dtype="bf16", is_mode="sais", mpt_mode="dynamic",
                entropy_target=wl.entropy_target, current_version=batch.current_version, bwd_panel_tokens=512)
    base.update(kw)
    return B.Params(**base)


def _unsplit(B, wl, batch, sigma):
    b = batch.to(DEV)
    gp = _params(B, wl, batch, entropy_target=sigma)
    out = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets)
    dH, dW = B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef)
    torch.cuda.synchronize()
    return out, dH, dW


def _sigma(B, wl, batch):
    # between the sequences' mean entropies, so that the gate is open for some sequences and shut for others
    out, _, _ = _unsplit(B, wl, batch, 0.2)
    hbar = np.sort(out.seq_entropy.cpu().numpy()[:wl.S])
    return float(0.5 * (hbar[wl.S // 2 - 1] + hbar[wl.S // 2]))


def _sequence_worker(rank, world, port, result_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2507_19766_b200 import binding as B, dp
        torch.cuda.set_device(0)
        wl, batch = _batch()
        sigma = _sigma(B, wl, batch)
        off = batch.seq_offsets.numpy()
        lengths = np.diff(off)
        mine = dp.shard_sequences(lengths, world)[rank]
        rows = torch.from_numpy(np.concatenate([np.arange(off[i], off[i + 1]) for i in mine])).to(DEV)
        local_off = torch.tensor(np.concatenate([[0], np.cumsum(lengths[mine])]), dtype=torch.int32, device=DEV)
        n_global = dp.global_token_count(int(rows.numel()))
        assert n_global == wl.T
        b = batch.to(DEV)
        gp = _params(B, wl, batch, T=int(rows.numel()), num_seqs=len(mine), norm_tokens=n_global, entropy_target=sigma)
        hidden = b.hidden[rows].contiguous()
        out = B.token_loss_fwd(gp, hidden, b.W, b.targets[rows].contiguous(), b.old_logp[rows].contiguous(),
                               b.segment_version[rows].contiguous(),
                               b.advantages[torch.tensor(mine, device=DEV)].contiguous(), local_off)
        d_W = torch.empty(wl.V, wl.H, device=DEV)
        red = dp.SlabAllReduce(d_W)
        assert red.active
        dH, _ = B.token_loss_bwd(gp, hidden, b.W, b.targets[rows].contiguous(), out.lse, out.grad_coef, d_W=d_W,
                                 on_dw_slab=red)
        dist.all_reduce(out.loss)
        covered = red.finish()
        torch.cuda.synchronize()
        assert covered[0][0] == 0 and sum(r for _, r in covered) == wl.V and len(covered) > 1
        full, dH_full, dW_full = _unsplit(B, wl, batch, sigma)
        assert torch.equal(dH, dH_full[rows])                       # rows do not depend on the sharding
        assert torch.equal(out.flags, full.flags[rows]) and torch.equal(out.grad_coef, full.grad_coef[rows])
        err = float((d_W - dW_full).norm() / dW_full.norm())
        assert err <= 1e-5, err                                     # same sum, other grouping of the tokens
        assert abs(float(out.loss) - float(full.loss)) <= 1e-5 * max(1e-3, abs(float(full.loss)))
        masked = int((full.flags & 1).sum())
        assert 0 < masked < int((full.flags & 8).ne(0).sum())       # both gate states occur
        open(os.path.join(result_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def _token_range_worker(rank, world, port, result_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import dataclasses
        from paper_2507_19766_b200 import binding as B, dp
        torch.cuda.set_device(0)
        wl, batch = _batch()
        sigma = _sigma(B, wl, batch)
        off = batch.seq_offsets.numpy()
        lo, hi = dp.shard_token_ranges(wl.T, world, align=256)[rank]
        ids, loff = dp.local_sequence_pieces(off, lo, hi)
        b = batch.to(DEV)
        sl = slice(lo, hi)
        lp = _params(B, wl, batch, T=hi - lo, num_seqs=len(ids), norm_tokens=wl.T, ent_scope="supplied",
                     entropy_target=sigma)
        loff_t = torch.tensor(loff, dtype=torch.int32, device=DEV)
        ids_t = torch.tensor(ids, dtype=torch.int32, device=DEV)
        adv = b.advantages[ids_t.long()].contiguous()
        f = B.token_loss_fwd(lp, b.hidden[sl], b.W, b.targets[sl], b.old_logp[sl], b.segment_version[sl], adv, loff_t,
                             entropy_supplied=torch.zeros(len(ids), device=DEV))
        table = B.sequence_entropy_partials(lp, f.entropy, loff_t, ids_t, wl.S)
        dp.all_reduce_sequence_entropy(table)                       # the one exchange of the split
        gate = B.sequence_entropy_combine(table, ids_t, len(ids))
        d = B.token_loss_decide(lp, f.logp, f.entropy, b.old_logp[sl], b.segment_version[sl], adv, loff_t,
                                entropy_supplied=gate)
        d_W = torch.empty(wl.V, wl.H, device=DEV)
        red = dp.SlabAllReduce(d_W)
        dH, _ = B.token_loss_bwd(lp, b.hidden[sl], b.W, b.targets[sl], f.lse, d.grad_coef, d_W=d_W, on_dw_slab=red)
        dist.all_reduce(d.loss)
        red.finish()
        torch.cuda.synchronize()
        full, dH_full, dW_full = _unsplit(B, wl, batch, sigma)
        gate_all = B.sequence_entropy_combine(table, None, wl.S)
        assert torch.equal(gate_all, full.seq_entropy[:wl.S])       # bit for bit the unsplit means
        assert torch.equal(d.flags, full.flags[sl]) and torch.equal(dH, dH_full[sl])
        assert float((d_W - dW_full).norm() / dW_full.norm()) <= 1e-5
        assert abs(float(d.loss) - float(full.loss)) <= 1e-5 * max(1e-3, abs(float(full.loss)))
        open(os.path.join(result_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("worker", [_sequence_worker, _token_range_worker])
def test_two_ranks_on_device_buffers_match_the_unsplit_batch(worker, tmp_path):
    from paper_2507_19766_b200 import dp
    mp.spawn(worker, args=(2, dp.free_port(), str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok0").exists() and (tmp_path / "ok1").exists()

"""Failure reporting and memory discipline of the CUDA path, without faulting or stalling the GPU:
the bounded wait that every tensor-core kernel uses is made to run out in a block of its own, and
every buffer the library writes is fenced with guard bytes that must survive all passes."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2507_19766_b200 import binding as B
from workloads import synth
from tests.helpers import both_params

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GUARD = 4096
PATTERN = 0xA5


def test_bounded_wait_gives_up_and_reports_a_timeout():
    """A wait on a barrier that nothing signals ends after its cycle limit, the kernel returns normally, the
    status word says DEVICE_TIMEOUT, and the next ordinary call on the same workspace is clean."""
    wl = synth.WORKLOADS["small"].scaled(T=300, S=2, H=128, V=1024, lengths="tiny")
    batch = synth.make_batch(wl, seed=3)
    gp, _ = both_params(batch)
    ws = B.alloc_workspace(gp, DEV)
    ws.zero_()
    assert B.selftest_bounded_wait(ws, 1_000_000) == B.OK
    assert B.check_status(ws) == -5
    assert "wait" in B.status_string(-5)
    b = batch.to(DEV)
    out = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets,
                           workspace=ws)
    B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, workspace=ws)
    assert B.check_status(ws) == B.OK and out.stats_host()["device_status"] == 0
    # limits outside the accepted range are refused on the host, nothing is launched
    assert B.selftest_bounded_wait(ws, 10) == -1 and B.selftest_bounded_wait(ws, 10 ** 12) == -1


class Guarded:
    """Device buffers with GUARD bytes of a pattern on both sides."""

    def __init__(self):
        self.raw = []

    def alloc(self, n_elems, dtype):
        nbytes = n_elems * torch.empty(0, dtype=dtype).element_size()
        pad = (-nbytes) % 256
        raw = torch.full((GUARD + nbytes + pad + GUARD,), PATTERN, dtype=torch.uint8, device=DEV)
        self.raw.append((raw, nbytes))
        return raw[GUARD:GUARD + nbytes].view(dtype)

    def intact(self):
        for raw, nbytes in self.raw:
            if not bool((raw[:GUARD] == PATTERN).all()) or not bool((raw[GUARD + nbytes:] == PATTERN).all()):
                return False
        return True


@pytest.mark.parametrize("path,compact,dw_dtype", [("tensor", False, "f32"), ("tensor", True, "f32"),
                                                   ("tensor", False, "bf16"), ("tensor_1cta", True, "bf16"),
                                                   ("simt", False, "f32")])
def test_guard_bytes_around_every_buffer_survive_all_passes(path, compact, dw_dtype):
    """Ragged sizes (T = 700, V = 3001, H = 328, two backward panels): forward, backward and the host-buffer step
    write the workspace, the arena and every output only inside their bounds."""
    wl = synth.WORKLOADS["small"].scaled(T=700, S=5, H=328, V=3001, lengths="lognormal:100:400", segment_len=64,
                                         planted=0.3, beta_planted=(80.0, 160.0), mpt_mode="dynamic",
                                         entropy_target=6.0)
    batch = synth.make_batch(wl, seed=5)
    gp, _ = both_params(batch, kernel_path=path, bwd_panel_tokens=384, compact_rows=compact)
    gp = dataclasses.replace(gp, dw_dtype=dw_dtype)
    b = batch.to(DEV)
    G = Guarded()
    T, S, H, V = wl.T, wl.S, wl.H, wl.V
    f32 = torch.float32
    out = B.FwdOut(logp=G.alloc(T, f32), entropy=G.alloc(T, f32), lse=G.alloc(T, f32), grad_coef=G.alloc(T, f32),
                   flags=G.alloc(T, torch.uint8), seq_entropy=G.alloc(S, f32), loss=G.alloc(1, f32),
                   stats=G.alloc(B.alloc_fwd_outputs(gp, DEV).stats.numel(), torch.uint8))
    ws = G.alloc(B.workspace_bytes(gp), torch.uint8)
    d_hidden = G.alloc(T * H, torch.bfloat16).view(T, H)
    d_W = G.alloc(V * H, gp.dw_torch_dtype).view(V, H)
    table = G.alloc(2 * S, torch.int64)
    for _ in range(2):
        B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets,
                         out=out, workspace=ws)
        B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_hidden=d_hidden, d_W=d_W, workspace=ws)
    code = B.load_library().ulorl_sequence_entropy_partials(
        __import__("ctypes").byref(gp.to_c()), B._ptr(out.entropy), B._ptr(b.seq_offsets), None, S, B._ptr(table), None,
        B._stream())
    assert code == B.OK
    torch.cuda.synchronize()
    assert B.check_status(ws) == B.OK
    assert G.intact()
    assert torch.isfinite(d_hidden.float()).all() and torch.isfinite(d_W.float()).all()
    # host-buffer step: the arena is the only device memory it is given
    arena = G.alloc(B.host_step_arena_bytes(gp), torch.uint8)
    pin = lambda t: t.contiguous().pin_memory()
    ho = dict(logp=torch.empty(T).pin_memory(), entropy=torch.empty(T).pin_memory(),
              flags=torch.empty(T, dtype=torch.uint8).pin_memory(), seq_entropy=torch.empty(S).pin_memory(),
              loss=torch.empty(1).pin_memory(), stats=torch.empty(out.stats.numel(), dtype=torch.uint8).pin_memory(),
              d_hidden=torch.empty(T, H, dtype=torch.bfloat16).pin_memory(),
              d_W=torch.empty(V, H, dtype=gp.dw_torch_dtype).pin_memory())
    B.token_loss_step_host(gp, arena, pin(batch.hidden), pin(batch.W), pin(batch.targets), pin(batch.old_logp),
                           pin(batch.segment_version), pin(batch.advantages), pin(batch.seq_offsets), **ho)
    torch.cuda.synchronize()
    assert G.intact()
    assert torch.equal(ho["d_W"], d_W.cpu()) and torch.equal(ho["d_hidden"], d_hidden.cpu())
    assert torch.equal(ho["logp"], out.logp.cpu())


def test_decision_stage_with_many_short_and_empty_sequences():
    """20000 sequences of 0..3 tokens: every thread of the decision kernel steps through several sequence
    boundaries (and over empty sequences) inside its four tokens, the per-sequence sums take the token-by-token
    path in every block.  Flags, counts and sequence means against the oracle."""
    from oracle import ulorl_oracle as O
    rng = np.random.default_rng(23)
    S = 20000
    lens = rng.integers(0, 4, size=S)
    lens[-1] = max(lens[-1], 1)
    T = int(lens.sum())
    offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    logp = (-np.abs(rng.standard_normal(T)) * 0.02).astype(np.float32)
    logp[rng.random(T) < 0.3] -= np.float32(3.0)
    ent = (np.abs(rng.standard_normal(T)) * 0.25).astype(np.float32)
    old = (logp + rng.standard_normal(T).astype(np.float32) * 0.15).astype(np.float32)
    adv = rng.choice(np.float32([1.0, -1.0, 0.0, 0.7]), size=S).astype(np.float32)
    version = rng.integers(0, 9, size=T).astype(np.int32)
    kw = dict(is_mode="sais", mpt_mode="dynamic", entropy_target=0.2, current_version=8)
    ref = O.decide(logp, O.gate_entropy(ent, offsets, "per_seq", None), old, adv, offsets, version, O.OracleParams(**kw))
    t = lambda x: torch.from_numpy(x).to(DEV)
    out = B.token_loss_decide(B.Params(T=T, H=8, V=16, num_seqs=S, dtype="f32", **kw), t(logp), t(ent), t(old),
                              t(version), t(adv), t(offsets))
    torch.cuda.synchronize()
    assert np.array_equal(out.flags.cpu().numpy(), ref["flags"])
    st = out.stats_host()
    for k in ("n_tokens", "n_active", "n_mpt", "n_masked", "n_clip_high", "n_clip_low"):
        assert st[k] == ref["stats"][k], k
    assert st["device_status"] == 0 and ref["stats"]["n_masked"] > 0
    seq_mean, batch_mean = O.sequence_mean_entropy(ent, offsets)
    got = out.seq_entropy.cpu().numpy()[:S]
    assert np.allclose(got, seq_mean, rtol=1e-6, atol=1e-9) and (got[lens == 0] == 0).all()
    assert abs(st["mean_entropy"] - batch_mean) <= 1e-6
    assert np.allclose(out.grad_coef.cpu().numpy(), ref["grad_coef"], rtol=1e-6, atol=0)


def test_first_calls_from_two_host_threads_at_once():
    """Two host threads, each with its own stream, workspace and outputs, make their calls at the same time
    (ctypes releases the interpreter lock for the duration of a call): the lazily created per-device tables are
    built under one mutex, and the results are those of the same calls made one after the other."""
    import threading
    wl = synth.WORKLOADS["small"].scaled(T=900, S=4, H=256, V=4000, lengths="tiny", planted=0.3,
                                         beta_planted=(100.0, 200.0), mpt_mode="always")
    batch = synth.make_batch(wl, seed=18)
    b = batch.to(DEV)
    results, errors = {}, []

    def work(name, path):
        try:
            gp, _ = both_params(batch, kernel_path=path)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                ws = B.alloc_workspace(gp, DEV)
                for _ in range(10):
                    out = B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages,
                                           b.seq_offsets, workspace=ws)
                    dH, dW = B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, workspace=ws)
                stream.synchronize()
                assert B.check_status(ws) == B.OK
            results[name] = (out.logp.clone(), out.loss.clone(), dH.clone(), dW.clone())
        except BaseException as exc:      # surfaced in the main thread below
            errors.append(exc)

    torch.cuda.synchronize()
    threads = [threading.Thread(target=work, args=(f"t{i}", p)) for i, p in enumerate(("tensor", "tensor_1cta", "tensor", "simt"))]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors
    work("serial_tensor", "tensor")
    work("serial_1cta", "tensor_1cta")
    for a, c in (("t0", "serial_tensor"), ("t2", "serial_tensor"), ("t1", "serial_1cta")):
        for x, y in zip(results[a], results[c]):
            assert torch.equal(x, y)

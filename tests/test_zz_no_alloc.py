"""ulorl_token_loss_decide_static: the elementwise stage for callers that cannot allocate device
memory when they call (a frozen allocator inside a host framework's step, a plugin that only gets
its op's tensors, a process whose device budget was handed out at start-up).  Its scratch is a
fixed array inside the library, so it takes no workspace; results must be those of
ulorl_token_loss_decide.  Collected last on purpose: a run that stops at the first failure has
then already exercised everything else."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2507_19766_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def make_case(seed, T, S):
    rng = np.random.default_rng(seed)
    cuts = np.sort(rng.choice(np.arange(1, T), size=S - 1, replace=False))
    offsets = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    logp = (-np.abs(rng.standard_normal(T)) * 0.02).astype(np.float32)
    logp[rng.random(T) < 0.3] -= np.float32(2.5)
    ent = (np.abs(rng.standard_normal(T)) * 0.25).astype(np.float32)
    old = (logp + rng.standard_normal(T).astype(np.float32) * 0.15).astype(np.float32)
    adv = rng.choice(np.float32([1.0, -1.0, 0.0, 0.6]), size=S).astype(np.float32)
    version = rng.integers(0, 6, size=T).astype(np.int32)
    t = lambda x: torch.from_numpy(x).to(DEV)
    return tuple(t(x) for x in (logp, ent, old, version, adv, offsets))


def same(a: B.FwdOut, b: B.FwdOut, S):
    assert torch.equal(a.flags, b.flags)
    assert torch.equal(a.grad_coef, b.grad_coef)
    assert torch.equal(a.loss, b.loss)
    assert torch.equal(a.seq_entropy[:S], b.seq_entropy[:S])
    sa, sb = a.stats_host(), b.stats_host()
    assert sa == sb


def test_static_scratch_variant_matches_workspace_variant_twice_in_a_row():
    # two calls in a row with different sizes and modes: the second sees the first's leftovers
    cases = [(31, 70001, 9, dict(is_mode="sais", mpt_mode="dynamic", entropy_target=0.2, current_version=5)),
             (32, 1237, 3, dict(is_mode="pois", mpt_mode="always", ent_scope="batch", current_version=5))]
    for seed, T, S, kw in cases:
        logp, ent, old, version, adv, offsets = make_case(seed, T, S)
        p = B.Params(T=T, H=8, V=16, num_seqs=S, dtype="f32", **kw)
        ref = B.token_loss_decide(p, logp, ent, old, version, adv, offsets)
        out = B.alloc_fwd_outputs(p, DEV)            # outputs belong to the caller, as in the C ABI
        got = B.token_loss_decide_static(p, logp, ent, old, version, adv, offsets, out=out)
        torch.cuda.synchronize()
        same(got, ref, S)
        assert got.stats_host()["n_tokens"] == T and got.stats_host()["device_status"] == 0


def test_static_scratch_variant_reports_bad_offsets_through_its_own_status_word():
    # this caller has no workspace to ask: the finding is in the built-in array's status word
    logp, ent, old, version, adv, offsets = make_case(33, 500, 3)
    p = B.Params(T=500, H=8, V=16, num_seqs=3, dtype="f32", current_version=5)
    out = B.alloc_fwd_outputs(p, DEV)
    bad = offsets.clone()
    bad[1] = 9999
    B.token_loss_decide_static(p, logp, ent, old, version, adv, bad, out=out)
    assert B.check_status(None) == -1 and out.stats_host()["device_status"] != 0
    B.token_loss_decide_static(p, logp, ent, old, version, adv, offsets, out=out)
    assert B.check_status(None) == B.OK and out.stats_host()["device_status"] == 0


def test_static_scratch_variant_rejects_batches_beyond_its_limit():
    lib = B.load_library()
    for T, S in ((B.STATIC_MAX_TOKENS + 1, 1), (B.STATIC_MAX_SEQS + 1, B.STATIC_MAX_SEQS + 1)):
        p = B.Params(T=T, H=8, V=16, num_seqs=S, dtype="f32").to_c()
        code = lib.ulorl_token_loss_decide_static(ctypes.byref(p), *([None] * 13), None)
        assert code == -7
    assert "scratch" in B.status_string(-7)

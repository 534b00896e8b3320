"""ctypes binding of libulorl.so: argument marshalling only.

Every step of the token-loss path runs inside the CUDA library; this module turns torch
tensors into device pointers, fills the parameter struct and checks return codes.  There is
no CPU fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libulorl.so")

OK = 0
F32, BF16 = 0, 1
IS_SAIS, IS_POIS = 0, 1
MPT_OFF, MPT_ALWAYS, MPT_DYNAMIC = 0, 1, 2
ENT_PER_SEQ, ENT_BATCH, ENT_SUPPLIED = 0, 1, 2
PATH_AUTO, PATH_SIMT, PATH_TENSOR, PATH_TENSOR_1CTA = 0, 1, 2, 3
FLAG_MASKED, FLAG_CLIP_HIGH, FLAG_CLIP_LOW, FLAG_MPT = 1, 2, 4, 8
N_STALENESS = 16

_IS = {"sais": IS_SAIS, "pois": IS_POIS}
_MPT = {"off": MPT_OFF, "always": MPT_ALWAYS, "dynamic": MPT_DYNAMIC}
_ENT = {"per_seq": ENT_PER_SEQ, "batch": ENT_BATCH, "supplied": ENT_SUPPLIED}
_NORM = {"tokens": 0, "sequence": 1}
_PATH = {"auto": PATH_AUTO, "simt": PATH_SIMT, "tensor": PATH_TENSOR, "tensor_1cta": PATH_TENSOR_1CTA}


class UlorlError(RuntimeError):
    pass


class CParams(ctypes.Structure):
    _fields_ = [
        ("T", ctypes.c_int32), ("H", ctypes.c_int32), ("V", ctypes.c_int32), ("num_seqs", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("is_mode", ctypes.c_int32), ("mpt_mode", ctypes.c_int32),
        ("ent_scope", ctypes.c_int32), ("adv_per_token", ctypes.c_int32),
        ("clip_eps_low", ctypes.c_float), ("clip_eps_high", ctypes.c_float), ("mpt_tau", ctypes.c_float),
        ("entropy_target", ctypes.c_float), ("inv_temperature", ctypes.c_float),
        ("norm_tokens", ctypes.c_int64), ("current_version", ctypes.c_int32),
        ("dw_accumulate", ctypes.c_int32), ("kernel_path", ctypes.c_int32), ("bwd_panel_tokens", ctypes.c_int32),
        ("compact_rows", ctypes.c_int32), ("loss_norm", ctypes.c_int32), ("norm_seqs", ctypes.c_int32),
        ("dw_dtype", ctypes.c_int32), ("kl_beta", ctypes.c_float),
    ]


class CStats(ctypes.Structure):
    _fields_ = [
        ("loss", ctypes.c_float), ("mean_entropy", ctypes.c_float),
        ("n_tokens", ctypes.c_int32), ("n_active", ctypes.c_int32), ("n_mpt", ctypes.c_int32),
        ("n_masked", ctypes.c_int32), ("n_clip_high", ctypes.c_int32), ("n_clip_low", ctypes.c_int32),
        ("stale_tokens", ctypes.c_int32 * N_STALENESS), ("stale_clipped", ctypes.c_int32 * N_STALENESS),
        ("stale_mean_abs_logratio", ctypes.c_float * N_STALENESS),
        ("device_status", ctypes.c_int32), ("mean_kl", ctypes.c_float), ("reserved", ctypes.c_int32 * 2),
    ]


EXPORTS = ("ulorl_workspace_bytes", "ulorl_token_loss_fwd", "ulorl_token_loss_decide", "ulorl_token_loss_bwd",
           "ulorl_token_loss_bwd_slabs",
           "ulorl_check_status", "ulorl_status_string", "ulorl_launch_count", "ulorl_kernel_timing_begin",
           "ulorl_kernel_timing_end", "ulorl_host_step_arena_bytes", "ulorl_token_loss_step_host",
           "ulorl_token_loss_decide_static", "ulorl_group_advantages", "ulorl_sequence_entropy_partials",
           "ulorl_sequence_entropy_combine", "ulorl_decision_thresholds", "ulorl_selftest_bounded_wait")
STATIC_MAX_TOKENS, STATIC_MAX_SEQS = 1 << 20, 1 << 16
KERNEL_KINDS = ("stats", "dz", "d_hidden", "d_W")

DW_SLAB_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32)

_lib = None


def load_library() -> ctypes.CDLL:
    """Load libulorl.so (built in-tree by paper_2507_19766_b200/build.py).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise UlorlError(f"{LIB_PATH} is missing: build it with `python -m paper_2507_19766_b200.build` "
                         "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, cp = ctypes.c_void_p, ctypes.POINTER(CParams)
    lib.ulorl_workspace_bytes.restype = ctypes.c_size_t
    lib.ulorl_workspace_bytes.argtypes = [cp]
    lib.ulorl_token_loss_fwd.restype = ctypes.c_int
    lib.ulorl_token_loss_fwd.argtypes = [cp] + [vp] * 17 + [vp, ctypes.c_size_t, vp]
    lib.ulorl_token_loss_decide.restype = ctypes.c_int
    lib.ulorl_token_loss_decide.argtypes = [cp] + [vp] * 13 + [vp, ctypes.c_size_t, vp]
    lib.ulorl_token_loss_decide_static.restype = ctypes.c_int
    lib.ulorl_token_loss_decide_static.argtypes = [cp] + [vp] * 13 + [vp]
    lib.ulorl_group_advantages.restype = ctypes.c_int
    lib.ulorl_group_advantages.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, vp, vp, vp]
    lib.ulorl_sequence_entropy_partials.restype = ctypes.c_int
    lib.ulorl_sequence_entropy_partials.argtypes = [cp, vp, vp, vp, ctypes.c_int32, vp, vp, vp]
    lib.ulorl_sequence_entropy_combine.restype = ctypes.c_int
    lib.ulorl_sequence_entropy_combine.argtypes = [vp, ctypes.c_int32, vp, ctypes.c_int32, vp, vp, vp]
    lib.ulorl_selftest_bounded_wait.restype = ctypes.c_int
    lib.ulorl_selftest_bounded_wait.argtypes = [vp, ctypes.c_int64, vp]
    lib.ulorl_decision_thresholds.restype = ctypes.c_int
    lib.ulorl_decision_thresholds.argtypes = [cp, ctypes.POINTER(ctypes.c_float)]
    lib.ulorl_token_loss_bwd.restype = ctypes.c_int
    lib.ulorl_token_loss_bwd.argtypes = [cp] + [vp] * 8 + [vp, ctypes.c_size_t, vp]
    lib.ulorl_token_loss_bwd_slabs.restype = ctypes.c_int
    lib.ulorl_token_loss_bwd_slabs.argtypes = [cp] + [vp] * 8 + [DW_SLAB_FN, vp] + [vp, ctypes.c_size_t, vp]
    lib.ulorl_check_status.restype = ctypes.c_int
    lib.ulorl_check_status.argtypes = [vp, vp]
    lib.ulorl_status_string.restype = ctypes.c_char_p
    lib.ulorl_status_string.argtypes = [ctypes.c_int]
    lib.ulorl_launch_count.restype = ctypes.c_int64
    lib.ulorl_launch_count.argtypes = []
    lib.ulorl_kernel_timing_begin.restype = ctypes.c_int
    lib.ulorl_kernel_timing_begin.argtypes = []
    lib.ulorl_kernel_timing_end.restype = ctypes.c_int
    lib.ulorl_kernel_timing_end.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int64)]
    lib.ulorl_host_step_arena_bytes.restype = ctypes.c_size_t
    lib.ulorl_host_step_arena_bytes.argtypes = [cp]
    lib.ulorl_token_loss_step_host.restype = ctypes.c_int
    lib.ulorl_token_loss_step_host.argtypes = [cp] + [vp] * 17 + [vp, ctypes.c_size_t, vp]
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().ulorl_status_string(code).decode()


def _check(code: int, what: str):
    if code != OK:
        raise UlorlError(f"{what} failed: {status_string(code)} ({code})")


@dataclass
class Params:
    """Mirror of ulorl_params_t with the paper's names (Eq. 7-10, Section 4.1)."""
    T: int
    H: int
    V: int
    num_seqs: int
    dtype: str = "bf16"
    is_mode: str = "sais"
    mpt_mode: str = "dynamic"
    ent_scope: str = "per_seq"
    adv_per_token: bool = False
    clip_eps_low: float = 0.2
    clip_eps_high: float = 0.2
    mpt_tau: float = 0.99
    entropy_target: float = 0.2
    inv_temperature: float = 1.0
    norm_tokens: int = 0
    current_version: int = 0
    dw_accumulate: bool = False
    kernel_path: str = "auto"
    bwd_panel_tokens: int = 0
    compact_rows: bool = False
    loss_norm: str = "tokens"
    norm_seqs: int = 0
    dw_dtype: str = "f32"
    kl_beta: float = 0.0

    @property
    def dw_torch_dtype(self):
        return torch.bfloat16 if self.dw_dtype == "bf16" else torch.float32

    def to_c(self) -> CParams:
        return CParams(self.T, self.H, self.V, self.num_seqs, BF16 if self.dtype == "bf16" else F32,
                       _IS[self.is_mode], _MPT[self.mpt_mode], _ENT[self.ent_scope], int(self.adv_per_token),
                       self.clip_eps_low, self.clip_eps_high, self.mpt_tau, self.entropy_target,
                       self.inv_temperature, self.norm_tokens, self.current_version, int(self.dw_accumulate),
                       _PATH[self.kernel_path], self.bwd_panel_tokens, int(self.compact_rows),
                       _NORM[self.loss_norm], self.norm_seqs, BF16 if self.dw_dtype == "bf16" else F32,
                       self.kl_beta)


def workspace_bytes(p: Params) -> int:
    n = load_library().ulorl_workspace_bytes(ctypes.byref(p.to_c()))
    if n == 0:
        raise UlorlError("ulorl_workspace_bytes: invalid parameters")
    return int(n)


def decision_thresholds(p: Params):
    """(ln tau, ln(1 + eps_high), ln(1 - eps_low)) as the float32 values the decision kernel compares with."""
    out = (ctypes.c_float * 3)()
    _check(load_library().ulorl_decision_thresholds(ctypes.byref(p.to_c()), out), "ulorl_decision_thresholds")
    return tuple(float(x) for x in out)


def launch_count() -> int:
    return int(load_library().ulorl_launch_count())


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise UlorlError("tensors must be contiguous CUDA tensors")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _want(t: torch.Tensor, dtype, n: int, name: str):
    if t.dtype != dtype or t.numel() != n:
        raise UlorlError(f"{name}: expected {n} elements of {dtype}, got {t.numel()} of {t.dtype}")


@dataclass
class FwdOut:
    logp: torch.Tensor
    entropy: torch.Tensor
    lse: torch.Tensor
    grad_coef: torch.Tensor
    flags: torch.Tensor
    seq_entropy: torch.Tensor
    loss: torch.Tensor
    stats: torch.Tensor      # raw bytes of ulorl_stats_t on the device

    def stats_host(self) -> dict:
        return decode_stats(self.stats)


def decode_stats(stats: torch.Tensor) -> dict:
    raw = bytes(stats.cpu().numpy().tobytes())
    s = CStats.from_buffer_copy(raw)
    return dict(loss=s.loss, mean_entropy=s.mean_entropy, n_tokens=s.n_tokens, n_active=s.n_active, n_mpt=s.n_mpt,
                n_masked=s.n_masked, n_clip_high=s.n_clip_high, n_clip_low=s.n_clip_low,
                stale_tokens=list(s.stale_tokens), stale_clipped=list(s.stale_clipped),
                stale_mean_abs_logratio=list(s.stale_mean_abs_logratio), device_status=s.device_status,
                mean_kl=s.mean_kl)


def alloc_workspace(p: Params, device) -> torch.Tensor:
    return torch.empty(workspace_bytes(p), dtype=torch.uint8, device=device)


def alloc_fwd_outputs(p: Params, device) -> FwdOut:
    f = dict(dtype=torch.float32, device=device)
    return FwdOut(logp=torch.empty(p.T, **f), entropy=torch.empty(p.T, **f), lse=torch.empty(p.T, **f),
                  grad_coef=torch.empty(p.T, **f), flags=torch.empty(p.T, dtype=torch.uint8, device=device),
                  seq_entropy=torch.empty(max(p.num_seqs, 1), **f), loss=torch.empty(1, **f),
                  stats=torch.empty(ctypes.sizeof(CStats), dtype=torch.uint8, device=device))


def token_loss_fwd(p: Params, hidden, W, targets, old_logp, segment_version, advantages, seq_offsets,
                   entropy_supplied=None, out: Optional[FwdOut] = None, workspace: Optional[torch.Tensor] = None,
                   ref_logp=None) -> FwdOut:
    """ulorl_token_loss_fwd on the current CUDA stream."""
    lib = load_library()
    dev = hidden.device
    tdt = torch.bfloat16 if p.dtype == "bf16" else torch.float32
    _want(hidden, tdt, p.T * p.H, "hidden")
    _want(W, tdt, p.V * p.H, "W")
    _want(targets, torch.int32, p.T, "targets")
    _want(seq_offsets, torch.int32, p.num_seqs + 1, "seq_offsets")
    _want(advantages, torch.float32, p.T if p.adv_per_token else p.num_seqs, "advantages")
    if old_logp is not None:
        _want(old_logp, torch.float32, p.T, "old_logp")
    if segment_version is not None:
        _want(segment_version, torch.int32, p.T, "segment_version")
    out = out or alloc_fwd_outputs(p, dev)
    workspace = workspace if workspace is not None else alloc_workspace(p, dev)
    code = lib.ulorl_token_loss_fwd(
        ctypes.byref(p.to_c()), _ptr(hidden), _ptr(W), _ptr(targets), _ptr(old_logp), _ptr(ref_logp),
        _ptr(segment_version),
        _ptr(advantages), _ptr(seq_offsets), _ptr(entropy_supplied), _ptr(out.logp), _ptr(out.entropy), _ptr(out.lse),
        _ptr(out.grad_coef), _ptr(out.flags), _ptr(out.seq_entropy), _ptr(out.loss), _ptr(out.stats),
        _ptr(workspace), workspace.numel(), _stream())
    _check(code, "ulorl_token_loss_fwd")
    return out


def token_loss_decide(p: Params, logp, entropy, old_logp, segment_version, advantages, seq_offsets,
                      entropy_supplied=None, out: Optional[FwdOut] = None,
                      workspace: Optional[torch.Tensor] = None, ref_logp=None) -> FwdOut:
    """ulorl_token_loss_decide: the elementwise stage on given per-token log-probs and entropies."""
    lib = load_library()
    dev = logp.device
    _want(logp, torch.float32, p.T, "logp")
    _want(entropy, torch.float32, p.T, "entropy")
    out = out or alloc_fwd_outputs(p, dev)
    out.logp, out.entropy = logp, entropy
    workspace = workspace if workspace is not None else alloc_workspace(p, dev)
    code = lib.ulorl_token_loss_decide(
        ctypes.byref(p.to_c()), _ptr(logp), _ptr(entropy), _ptr(old_logp), _ptr(ref_logp), _ptr(segment_version),
        _ptr(advantages),
        _ptr(seq_offsets), _ptr(entropy_supplied), _ptr(out.grad_coef), _ptr(out.flags), _ptr(out.seq_entropy),
        _ptr(out.loss), _ptr(out.stats), _ptr(workspace), workspace.numel(), _stream())
    _check(code, "ulorl_token_loss_decide")
    return out


def token_loss_decide_static(p: Params, logp, entropy, old_logp, segment_version, advantages, seq_offsets,
                             entropy_supplied=None, out: Optional[FwdOut] = None, ref_logp=None) -> FwdOut:
    """ulorl_token_loss_decide_static: the elementwise stage with no workspace argument, for callers
    that cannot allocate device memory; its scratch is a fixed array inside the library (at most
    STATIC_MAX_TOKENS tokens and STATIC_MAX_SEQS sequences).  `out` must be given by such a caller;
    when omitted this wrapper allocates the outputs with torch for convenience."""
    lib = load_library()
    _want(logp, torch.float32, p.T, "logp")
    _want(entropy, torch.float32, p.T, "entropy")
    out = out or alloc_fwd_outputs(p, logp.device)
    out.logp, out.entropy = logp, entropy
    code = lib.ulorl_token_loss_decide_static(
        ctypes.byref(p.to_c()), _ptr(logp), _ptr(entropy), _ptr(old_logp), _ptr(ref_logp), _ptr(segment_version),
        _ptr(advantages),
        _ptr(seq_offsets), _ptr(entropy_supplied), _ptr(out.grad_coef), _ptr(out.flags), _ptr(out.seq_entropy),
        _ptr(out.loss), _ptr(out.stats), _stream())
    _check(code, "ulorl_token_loss_decide_static")
    return out


def token_loss_bwd(p: Params, hidden, W, targets, lse, grad_coef, grad_loss=None, d_hidden=None, d_W=None,
                   workspace: Optional[torch.Tensor] = None, on_dw_slab=None):
    """ulorl_token_loss_bwd on the current CUDA stream.  Returns (d_hidden, d_W).  With on_dw_slab (a callable
    (first_row, rows) -> None) the call goes through ulorl_token_loss_bwd_slabs: the callable runs on this
    thread each time the launches that make a slab of rows of d_W final have been queued."""
    lib = load_library()
    dev = hidden.device
    if d_hidden is None:
        d_hidden = torch.empty_like(hidden)
    if d_W is None:
        d_W = (torch.zeros if p.dw_accumulate else torch.empty)(p.V, p.H, dtype=p.dw_torch_dtype, device=dev)
    _want(d_W, p.dw_torch_dtype, p.V * p.H, "d_W")
    workspace = workspace if workspace is not None else alloc_workspace(p, dev)
    head = (ctypes.byref(p.to_c()), _ptr(hidden), _ptr(W), _ptr(targets), _ptr(lse), _ptr(grad_coef), _ptr(grad_loss),
            _ptr(d_hidden), _ptr(d_W))
    tail = (_ptr(workspace), workspace.numel(), _stream())
    if on_dw_slab is None:
        code = lib.ulorl_token_loss_bwd(*head, *tail)
    else:
        failure = []

        def trampoline(_user, first_row, rows):
            try:
                on_dw_slab(int(first_row), int(rows))
                return 0
            except BaseException as exc:       # an exception cannot cross the C frames: stop the pass, re-raise below
                failure.append(exc)
                return -4
        code = lib.ulorl_token_loss_bwd_slabs(*head, DW_SLAB_FN(trampoline), None, *tail)
        if failure:
            raise failure[0]
    _check(code, "ulorl_token_loss_bwd")
    return d_hidden, d_W


def check_status(workspace: Optional[torch.Tensor]) -> int:
    """ulorl_check_status; workspace=None reads the status word of the no-allocation entry point's built-in scratch."""
    return int(load_library().ulorl_check_status(_ptr(workspace), _stream()))


def selftest_bounded_wait(workspace: torch.Tensor, limit_cycles: int = 1_000_000) -> int:
    """ulorl_selftest_bounded_wait: returns the launch status; the timeout shows up in check_status(workspace)."""
    return int(load_library().ulorl_selftest_bounded_wait(_ptr(workspace), limit_cycles, _stream()))


def kernel_timing_begin():
    _check(load_library().ulorl_kernel_timing_begin(), "ulorl_kernel_timing_begin")


def kernel_timing_end() -> dict:
    """Per tensor-core kernel: (total milliseconds, launches) since kernel_timing_begin()."""
    ms = (ctypes.c_float * 4)()
    n = (ctypes.c_int64 * 4)()
    _check(load_library().ulorl_kernel_timing_end(ms, n), "ulorl_kernel_timing_end")
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_KINDS)}


def host_step_arena_bytes(p: Params) -> int:
    n = load_library().ulorl_host_step_arena_bytes(ctypes.byref(p.to_c()))
    if n == 0:
        raise UlorlError("ulorl_host_step_arena_bytes: invalid parameters")
    return int(n)


def _hptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise UlorlError("host-step tensors must be contiguous CPU tensors")
    return ctypes.c_void_p(t.data_ptr())


def token_loss_step_host(p: Params, arena: torch.Tensor, hidden, W, targets, old_logp, segment_version, advantages,
                         seq_offsets, entropy_supplied=None, logp=None, entropy=None, flags=None, seq_entropy=None,
                         loss=None, stats=None, d_hidden=None, d_W=None, ref_logp=None):
    """ulorl_token_loss_step_host: every tensor except `arena` lives in host memory (pinned for
    asynchronous copies).  Asynchronous on the current stream."""
    code = load_library().ulorl_token_loss_step_host(
        ctypes.byref(p.to_c()), _hptr(hidden), _hptr(W), _hptr(targets), _hptr(old_logp), _hptr(ref_logp),
        _hptr(segment_version), _hptr(advantages), _hptr(seq_offsets), _hptr(entropy_supplied), _hptr(logp), _hptr(entropy), _hptr(flags),
        _hptr(seq_entropy), _hptr(loss), _hptr(stats), _hptr(d_hidden), _hptr(d_W), _ptr(arena), arena.numel(),
        _stream())
    _check(code, "ulorl_token_loss_step_host")


def sequence_entropy_partials(p: Params, entropy: torch.Tensor, seq_offsets: torch.Tensor, seq_ids, total_seqs: int,
                              workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """ulorl_sequence_entropy_partials: int64 [total_seqs, 2] (entropy sum in 2^-34 nats, token count) of the
    call's pieces of sequences, zero for the sequences it holds nothing of."""
    _want(entropy, torch.float32, p.T, "entropy")
    _want(seq_offsets, torch.int32, p.num_seqs + 1, "seq_offsets")
    if seq_ids is not None:
        _want(seq_ids, torch.int32, p.num_seqs, "seq_ids")
    table = torch.empty(total_seqs, 2, dtype=torch.int64, device=entropy.device)
    code = load_library().ulorl_sequence_entropy_partials(ctypes.byref(p.to_c()), _ptr(entropy), _ptr(seq_offsets),
                                                          _ptr(seq_ids), total_seqs, _ptr(table), _ptr(workspace),
                                                          _stream())
    _check(code, "ulorl_sequence_entropy_partials")
    return table


def sequence_entropy_combine(table: torch.Tensor, seq_ids, num_seqs: int, want_batch: bool = False):
    """ulorl_sequence_entropy_combine: float32 mean entropy of the sequences seq_ids (None: the first num_seqs)
    from a summed table; with want_batch also the token mean over the whole table."""
    _want(table, torch.int64, table.numel(), "table")
    if seq_ids is not None:
        _want(seq_ids, torch.int32, num_seqs, "seq_ids")
    out = torch.empty(max(num_seqs, 1), dtype=torch.float32, device=table.device)
    batch = torch.empty(1, dtype=torch.float32, device=table.device) if want_batch else None
    code = load_library().ulorl_sequence_entropy_combine(_ptr(table), table.shape[0], _ptr(seq_ids), num_seqs,
                                                         _ptr(out), _ptr(batch), _stream())
    _check(code, "ulorl_sequence_entropy_combine")
    return (out[:num_seqs], batch) if want_batch else out[:num_seqs]


def group_advantages(rewards: torch.Tensor, group_size: int):
    """ulorl_group_advantages: Eq. 4 advantages and the Eq. 7 keep flag per response (device tensors)."""
    _want(rewards, torch.float32, rewards.numel(), "rewards")
    adv = torch.empty_like(rewards)
    keep = torch.empty(rewards.numel(), dtype=torch.uint8, device=rewards.device)
    code = load_library().ulorl_group_advantages(_ptr(rewards), rewards.numel(), group_size, _ptr(adv), _ptr(keep),
                                                 _stream())
    _check(code, "ulorl_group_advantages")
    return adv, keep

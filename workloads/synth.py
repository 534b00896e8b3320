"""Seeded synthetic inputs with the shape and structure of UloRL policy-update batches.

This module only *produces inputs*.  It is the one piece shared by the CUDA path's
tests, the CPU oracle's tests and the benchmark; it imports neither of them.  The
workloads stand in for the paper's Qwen3-30B-A3B batches (Section 4.1: 128 prompts x 8
responses, up to 128k response tokens in 8 segments of 16k): packed response tokens,
long-tailed sequence lengths, a policy version per segment (Section 3.1.2, the map f of
Eq. 8), 0/1 rewards turned into group-normalised advantages (Eq. 4), and a share of
sharply peaked rows so that well-mastered positive tokens (Eq. 9) actually occur.

Random numbers come from NumPy's counter-based Philox generator; a batch is a pure
function of (workload, seed).

Two recipes imitate what the parts of the training loop upstream of the policy update hand
over; they are input recipes, not implementations anyone is checked against.  `rollout_logp`
stands in for the rollout engine's record of the log-prob of each generated token (library
matmul + logsumexp in float32) and for its sampler (inverse-CDF draw from the row softmax with
supplied uniforms); per-segment noise is added on top, and a caller may hand in log-probs from
elsewhere as the noise's base.  `_advantages` stands in for the reward model followed by the
group normalisation of Eq. 4 (library mean and standard deviation).  No expected value of any
test comes from either: the oracle and the CUDA path both just receive the arrays.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional

import numpy as np
import torch

BASE_SEED = 20250719


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                    # position in the list of named workloads (seed offset)
    T: int
    S: int
    H: int
    V: int
    dtype: str                    # "f32" | "bf16"
    lengths: str                  # recipe name, see _sequence_lengths
    segment_len: int              # tokens per segment; 0 = two halves per sequence
    max_segments: int
    noise: str                    # "const:<sigma>" | "stale:<sigma per version>"
    adv: str                      # "pm1" | "bern:<p>:<group>" | "plus1"
    planted: float                # share of rows whose target is a planted row argmax
    sampled: float                # share of rows whose target is drawn from the row softmax
    is_mode: str = "sais"
    mpt_mode: str = "dynamic"
    beta_planted: tuple = (18.0, 30.0)
    beta_sampled: tuple = (8.0, 16.0)
    clip_eps_low: float = 0.2
    clip_eps_high: float = 0.2
    mpt_tau: float = 0.99
    entropy_target: float = 0.2

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    "tiny": Workload("tiny", 0, T=512, S=4, H=256, V=4096, dtype="f32", lengths="tiny",
                     segment_len=0, max_segments=2, noise="const:0.05", adv="pm1",
                     planted=0.0, sampled=0.0, mpt_mode="always"),
    "small": Workload("small", 1, T=16384, S=16, H=1024, V=32768, dtype="bf16",
                      lengths="lognormal:512:4096", segment_len=1024, max_segments=4,
                      noise="const:0.1", adv="bern:0.5:8", planted=0.0, sampled=0.0,
                      mpt_mode="always"),
    "qwen": Workload("qwen", 2, T=65536, S=32, H=2048, V=151936, dtype="bf16",
                     lengths="longtail:1024:32768", segment_len=8192, max_segments=4,
                     noise="const:0.1", adv="bern:0.3:16", planted=0.4, sampled=0.0,
                     mpt_mode="always"),      # static masking (Section 3.2.1), so that the planted rows are masked
    "mixed": Workload("mixed", 3, T=262144, S=64, H=2048, V=151936, dtype="bf16",
                      lengths="pareto:1.2:131072", segment_len=16384, max_segments=8,
                      noise="stale:0.02", adv="bern:0.3:16", planted=0.4, sampled=0.0,
                      is_mode="pois", mpt_mode="dynamic"),
    "ultra": Workload("ultra", 4, T=131072, S=1, H=2048, V=151936, dtype="bf16",
                      lengths="single", segment_len=16384, max_segments=8,
                      noise="stale:0.02", adv="plus1", planted=0.7, sampled=0.3,
                      mpt_mode="dynamic", beta_planted=(18.5, 32.0), beta_sampled=(18.5, 32.0)),
    # the same batch shape with weaker plants: mean entropy above sigma, so the dynamic gate stays shut
    "ultra_open": Workload("ultra_open", 5, T=131072, S=1, H=2048, V=151936, dtype="bf16",
                           lengths="single", segment_len=16384, max_segments=8,
                           noise="stale:0.02", adv="plus1", planted=0.7, sampled=0.3,
                           mpt_mode="dynamic", beta_planted=(17.0, 29.0), beta_sampled=(17.0, 29.0)),
}


@dataclass
class Batch:
    workload: Workload
    hidden: torch.Tensor           # [T, H] f32 or bf16
    W: torch.Tensor                # [V, H]
    targets: torch.Tensor          # [T] int32
    old_logp: torch.Tensor         # [T] f32
    segment_version: torch.Tensor  # [T] int32
    advantages: torch.Tensor       # [S] f32
    seq_offsets: torch.Tensor      # [S+1] int32
    current_version: int
    planted_rows: np.ndarray       # bool [T]
    old_logp_noise: np.ndarray     # f32 [T]

    def to(self, device) -> "Batch":
        kw = {}
        for k in ("hidden", "W", "targets", "old_logp", "segment_version", "advantages",
                  "seq_offsets"):
            kw[k] = getattr(self, k).to(device)
        return replace(self, **kw)

    def host_f32(self, name: str) -> np.ndarray:
        """The stored values of `hidden` or `W` widened exactly to float32 on the host."""
        return getattr(self, name).detach().to("cpu", torch.float32).numpy()


# ------------------------------------------------------------------ structure of a batch
def _rescale_to_sum(raw: np.ndarray, total: int, cap: int) -> np.ndarray:
    """Positive integer lengths proportional to `raw`, each in [1, cap], summing to total."""
    n = raw.shape[0]
    assert n <= total <= n * cap
    w = raw.astype(np.float64) / raw.sum()
    x = np.clip(np.floor(w * total), 1, cap).astype(np.int64)
    order = np.argsort(-raw, kind="stable")
    guard = 0
    while x.sum() != total:
        diff = int(total - x.sum())
        step = 1 if diff > 0 else -1
        moved = 0
        for j in order:
            if moved == abs(diff):
                break
            if step > 0 and x[j] < cap:
                room = min(cap - x[j], abs(diff) - moved, max(1, abs(diff) // n))
                x[j] += room
                moved += room
            elif step < 0 and x[j] > 1:
                room = min(x[j] - 1, abs(diff) - moved, max(1, abs(diff) // n))
                x[j] -= room
                moved += room
        guard += 1
        assert guard < 10000 and moved > 0
    return x


def _sequence_lengths(wl: Workload, rng: np.random.Generator) -> np.ndarray:
    kind = wl.lengths.split(":")
    if kind[0] == "tiny":
        base = np.array([64, 96, 128, 224], dtype=np.float64)
        reps = int(np.ceil(wl.S / 4))
        raw = np.tile(base, reps)[: wl.S]
        return _rescale_to_sum(raw, wl.T, wl.T)
    if kind[0] == "single":
        assert wl.S == 1
        return np.array([wl.T], dtype=np.int64)
    if kind[0] == "lognormal":
        median, cap = float(kind[1]), int(kind[2])
        raw = np.exp(np.log(median) + 1.0 * rng.standard_normal(wl.S))
        return _rescale_to_sum(raw, wl.T, min(cap, wl.T))
    if kind[0] == "longtail":
        short_cap, cap = int(kind[1]), int(kind[2])
        n_long = max(1, int(round(0.1 * wl.S)))
        n_short = wl.S - n_long
        short = rng.integers(64, short_cap + 1, size=n_short).astype(np.float64)
        scale = wl.T / 65536.0
        short = np.maximum(1, np.floor(short * min(1.0, scale))).astype(np.int64)
        rest = wl.T - int(short.sum())
        raw_long = rng.uniform(0.5, 1.0, size=n_long)
        longs = _rescale_to_sum(raw_long, rest, max(int(cap * scale), rest // n_long + 1))
        x = np.concatenate([short, longs])
        return x[rng.permutation(wl.S)]
    if kind[0] == "pareto":
        alpha, cap = float(kind[1]), int(kind[2])
        raw = (1.0 - rng.random(wl.S)) ** (-1.0 / alpha)
        return _rescale_to_sum(raw, wl.T, min(cap, wl.T))
    if kind[0] == "fixed":                       # "fixed:50,25,15": the lengths as given (tests)
        x = np.array([int(v) for v in kind[1].split(",")], dtype=np.int64)
        assert x.shape[0] == wl.S and int(x.sum()) == wl.T
        return x
    raise ValueError(wl.lengths)


def _segments(wl: Workload, lengths: np.ndarray):
    """Per-token policy version (the map f of Eq. 8).  The last segment of every sequence
    was generated by the current policy, earlier ones by earlier versions."""
    T = int(lengths.sum())
    seg_idx = np.empty(T, dtype=np.int64)
    n_seg = np.empty(T, dtype=np.int64)
    pos = 0
    for L in lengths:
        L = int(L)
        k = np.arange(L)
        if wl.segment_len == 0:
            s = (k >= L // 2).astype(np.int64) if L > 1 else np.zeros(L, dtype=np.int64)
        else:
            s = np.minimum(k // wl.segment_len, wl.max_segments - 1)
        seg_idx[pos:pos + L] = s
        n_seg[pos:pos + L] = int(s[-1]) + 1
        pos += L
    current_version = int(n_seg.max()) - 1
    version = current_version - (n_seg - 1 - seg_idx)
    return version.astype(np.int32), current_version


def _advantages(wl: Workload, rng: np.random.Generator) -> np.ndarray:
    kind = wl.adv.split(":")
    if kind[0] == "plus1":
        return np.ones(wl.S, dtype=np.float32)
    if kind[0] == "pm1":
        a = np.where(np.arange(wl.S) % 2 == 0, 1.0, -1.0)
        return a.astype(np.float32)
    if kind[0] == "bern":
        prob, group = float(kind[1]), int(kind[2])
        rewards = (rng.random(wl.S) < prob).astype(np.float64)
        adv = np.zeros(wl.S)
        for a in range(0, wl.S, group):
            r = rewards[a:a + group]
            sd = r.std()
            adv[a:a + group] = 0.0 if sd == 0.0 else (r - r.mean()) / sd   # Eq. 4
        return adv.astype(np.float32)
    raise ValueError(wl.adv)


# ------------------------------------------------------------------ rollout stand-in
@torch.no_grad()
def rollout_logp(hidden: torch.Tensor, W: torch.Tensor, targets: Optional[torch.Tensor],
                 kappa: float = 1.0, chunk: int = 2048, sample_u: Optional[torch.Tensor] = None,
                 sample_rows: Optional[torch.Tensor] = None):
    """What a rollout engine would have recorded: log-prob of the target per row (library
    matmul + logsumexp, float32 accumulate) and the row argmax.  With `sample_u` given,
    rows flagged in `sample_rows` get their target replaced by an inverse-CDF draw from
    the row's softmax using the supplied uniforms.  Returns (logp, argmax, targets)."""
    T = hidden.shape[0]
    dev = hidden.device
    logp = torch.empty(T, dtype=torch.float32, device=dev)
    amax = torch.empty(T, dtype=torch.int64, device=dev)
    tg = targets.to(torch.int64).clone() if targets is not None else torch.zeros(T, dtype=torch.int64, device=dev)
    Wc = W if dev.type == "cuda" else W.float()
    for a in range(0, T, chunk):
        h = hidden[a:a + chunk]
        h = h if dev.type == "cuda" else h.float()
        z = (h @ Wc.t()).float() * kappa
        lse = torch.logsumexp(z, dim=1)
        amax[a:a + chunk] = z.argmax(dim=1)
        if sample_u is not None:
            sel = sample_rows[a:a + chunk]
            if bool(sel.any()):
                cdf = torch.softmax(z[sel].double(), dim=1).cumsum(dim=1)
                u = sample_u[a:a + chunk][sel].double().unsqueeze(1)
                draw = torch.searchsorted(cdf, u).squeeze(1).clamp_(max=z.shape[1] - 1)
                idx = torch.nonzero(sel).squeeze(1) + a
                tg[idx] = draw
        logp[a:a + chunk] = z.gather(1, tg[a:a + chunk].unsqueeze(1)).squeeze(1) - lse
    return logp, amax, tg


# ------------------------------------------------------------------ the generator
def make_batch(wl: Workload, seed: Optional[int] = None, device: str = "cpu",
               base_logp: Optional[np.ndarray] = None) -> Batch:
    """Generate one batch of the workload.  `device` is where the rollout stand-in's
    matmuls run (the batch itself is returned on the host; use Batch.to)."""
    seed = BASE_SEED + wl.index if seed is None else seed
    rng = np.random.Generator(np.random.Philox(seed))
    T, H, V, S = wl.T, wl.H, wl.V, wl.S
    tdt = torch.float32 if wl.dtype == "f32" else torch.bfloat16

    lengths = _sequence_lengths(wl, rng)
    assert lengths.sum() == T and lengths.shape[0] == S and lengths.min() >= 1
    seq_offsets = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    version, current_version = _segments(wl, lengths)
    adv = _advantages(wl, rng)

    W = torch.from_numpy((0.02 * rng.standard_normal((V, H), dtype=np.float32))).to(tdt)
    hidden = torch.from_numpy(rng.standard_normal((T, H), dtype=np.float32))
    targets = rng.integers(0, V, size=T).astype(np.int64)

    # planted rows: the target becomes the row argmax with probability around tau
    kind = rng.random(T)
    planted = kind < wl.planted
    sampled = (~planted) & (kind < wl.planted + wl.sampled)
    beta = np.zeros(T, dtype=np.float32)
    beta[planted] = rng.uniform(*wl.beta_planted, size=int(planted.sum())).astype(np.float32)
    beta[sampled] = rng.uniform(*wl.beta_sampled, size=int(sampled.sum())).astype(np.float32)
    nz = np.nonzero(beta)[0]
    if nz.size:
        tgt_t = torch.from_numpy(targets[nz])
        for a in range(0, nz.size, 8192):
            rows = torch.from_numpy(nz[a:a + 8192])
            hidden[rows] += torch.from_numpy(beta[nz[a:a + 8192]]).unsqueeze(1) * W[tgt_t[a:a + 8192]].float()
    hidden = hidden.to(tdt)
    sample_u = rng.random(T).astype(np.float32)
    noise = rng.standard_normal(T).astype(np.float32)

    nk = wl.noise.split(":")
    if nk[0] == "const":
        sigma_t = np.full(T, float(nk[1]), dtype=np.float32)
    else:
        sigma_t = (float(nk[1]) * (current_version - version)).astype(np.float32)
    noise = noise * sigma_t

    tg = torch.from_numpy(targets)
    if base_logp is None or wl.sampled > 0:
        dev = torch.device(device)
        lp, amax, tg_dev = rollout_logp(
            hidden.to(dev), W.to(dev), tg.to(dev), 1.0,
            sample_u=torch.from_numpy(sample_u).to(dev) if wl.sampled > 0 else None,
            sample_rows=torch.from_numpy(sampled).to(dev) if wl.sampled > 0 else None)
        tg = tg_dev.cpu()
        if base_logp is None:
            base_logp = lp.cpu().numpy()
    old_logp = (np.asarray(base_logp, dtype=np.float32) + noise).astype(np.float32)

    return Batch(
        workload=wl, hidden=hidden, W=W, targets=tg.to(torch.int32),
        old_logp=torch.from_numpy(old_logp), segment_version=torch.from_numpy(version),
        advantages=torch.from_numpy(adv), seq_offsets=torch.from_numpy(seq_offsets),
        current_version=current_version, planted_rows=planted, old_logp_noise=noise)

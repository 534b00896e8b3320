"""Benchmark of the fused UloRL token-loss path (forward + backward) on synthetic batches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload ultra] [--impl ours|reference]

One step = one forward and one backward pass of the whole path over one batch.  The headline
workload is the ultra-long single response (T=131072 tokens, H=2048, V=151936, bf16) with the
entropy gate of Eq. 10 open; the same line carries the gate-shut state of that workload, the other
named workloads, the run with active-row compaction, the end-to-end run from host buffers and the
CPU oracle on a bounded sample.  With --gpus N > 1 and no launcher around it the script starts its
own N ranks (one per GPU); rank 0 prints one JSON line.  `--impl reference` times the fp64 CPU
oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2507_19766_b200 import binding as B  # noqa: E402
from paper_2507_19766_b200 import dp  # noqa: E402
from workloads import synth  # noqa: E402

METRIC = "fused loss fwd+bwd tokens/sec at H=2048,V=151936; % of B200 bf16 tensor peak"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic_per_launch.txt")
KERNEL_SOURCE = os.path.join(ROOT, "paper_2507_19766_b200", "csrc", "umma_gemm.cuh")
LEG_SECONDS = 5.0          # timed length of each secondary leg: 25 clock samples at 200 ms


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


def load_traffic(workload: str, kernel: str):
    """DRAM bytes (read + write) per launch of a tensor-core kernel, from the tracked table of ncu counters.
    The table names the kernel source it was measured on by hash; if the source has changed since, the
    counters no longer describe the kernel and None is returned."""
    if not os.path.exists(TRAFFIC_FILE):
        return None
    with open(KERNEL_SOURCE, "rb") as f:
        current = hashlib.sha256(f.read()).hexdigest()[:16]
    measured_on, value = None, None
    for line in open(TRAFFIC_FILE):
        parts = line.split()
        if not parts or parts[0].startswith("#"):
            continue
        if parts[0] == "kernel_source_sha256_16":
            measured_on = parts[1]
        elif parts[0] == workload and parts[1] == kernel:
            value = None if parts[2] == "null" else float(parts[2])
    return value if measured_on == current else None


# ------------------------------------------------------------------ clocks during a timed region
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "200",
                 "-i", str(self.gpu_index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        return self

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, power = [], [], []
        reasons = set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.file.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.file.close()
        os.unlink(self.file.name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "power_w_median": float(np.median(power)),
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------ the CPU oracle on a bounded sample
def oracle_sample_run(hidden_rows, W_host, targets_rows, old_rows, version_rows, adv_value, params_kw):
    """Steps 1-8 of the oracle on a sub-batch made of the sampled rows (one sequence)."""
    from oracle import ulorl_oracle as O
    n = hidden_rows.shape[0]
    op = O.OracleParams(**params_kw)
    out = O.fwd_bwd(hidden_rows, W_host, targets_rows, old_rows, version_rows, np.float32([adv_value]),
                    np.array([0, n], dtype=np.int32), op)
    return out


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 0) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count() or 1


def oracle_params_kw(wl, current_version):
    return dict(is_mode=wl.is_mode, mpt_mode=wl.mpt_mode, ent_scope="per_seq", clip_eps_low=wl.clip_eps_low,
                clip_eps_high=wl.clip_eps_high, mpt_tau=wl.mpt_tau, entropy_target=wl.entropy_target,
                current_version=current_version)


def cpu_baseline(batch, n_rows: int) -> dict:
    wl = batch.workload
    rows = np.linspace(0, wl.T - 1, n_rows).astype(np.int64)
    rt = torch.from_numpy(rows)
    h = batch.hidden[rt].float().numpy()
    Wh = batch.W.float().numpy()
    t0 = time.perf_counter()
    oracle_sample_run(h, Wh, batch.targets[rt].numpy(), batch.old_logp[rt].numpy(),
                      batch.segment_version[rt].numpy(), float(batch.advantages[0]),
                      oracle_params_kw(wl, batch.current_version))
    dt = time.perf_counter() - t0
    return {"value": n_rows / dt, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
            "sample": f"{n_rows} evenly spaced token rows of the {wl.name} workload as one sub-batch, "
                      f"full V={wl.V}, fp64 forward+backward, {dt:.1f} s"}


def run_reference(args):
    """The reference arm: the fp64 oracle as it stands, on host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl_full = synth.WORKLOADS[args.workload]
    n_rows = args.ref_rows
    wl = wl_full.scaled(T=n_rows, S=1, lengths="single",
                        segment_len=max(1, n_rows // wl_full.max_segments))
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    batch = synth.make_batch(wl, device=dev)
    h = batch.host_f32("hidden")
    Wh = batch.host_f32("W")
    kw = oracle_params_kw(wl, batch.current_version)
    run = lambda: oracle_sample_run(h, Wh, batch.targets.numpy(), batch.old_logp.numpy(),
                                    batch.segment_version.numpy(), float(batch.advantages[0]), kw)
    for _ in range(min(args.warmup, 1)):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = time.perf_counter() - t0
    value = n_rows * args.steps / dt
    sample = (f"each step = fp64 oracle forward+backward on a {n_rows}-token batch of the {wl_full.name} recipe "
              f"(H={wl.H}, V={wl.V}); {args.steps} steps in {dt:.1f} s")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl_full.name, "T_per_step": n_rows, "H": wl.H, "V": wl.V},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------ the CUDA path
class Context:
    """What every leg needs: the device, the process group (or None), the measured peaks."""

    def __init__(self, world, rank, local_rank):
        self.world, self.rank, self.local_rank = world, rank, local_rank
        self.dev = torch.device("cuda", local_rank)
        self.dist = None
        self.peaks = load_peaks()

    def fence(self):
        torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
            torch.cuda.synchronize()

    def max_over_ranks(self, x: float) -> float:
        t = torch.tensor([x], dtype=torch.float64, device=self.dev)
        if self.dist is not None:
            self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())


class Leg:
    """One workload resident on the device with everything a step needs."""

    def __init__(self, ctx: Context, wl, panel=0, compact=False, dw_dtype="f32"):
        self.ctx, self.wl = ctx, wl
        dev = ctx.dev
        self.host_batch = synth.make_batch(wl, seed=synth.BASE_SEED + wl.index + 1000 * ctx.rank, device=str(dev))
        self.b = self.host_batch.to(dev)
        self.gp = B.Params(T=wl.T, H=wl.H, V=wl.V, num_seqs=wl.S, dtype=wl.dtype, is_mode=wl.is_mode,
                           mpt_mode=wl.mpt_mode, clip_eps_low=wl.clip_eps_low, clip_eps_high=wl.clip_eps_high,
                           mpt_tau=wl.mpt_tau, entropy_target=wl.entropy_target,
                           current_version=self.host_batch.current_version, bwd_panel_tokens=panel,
                           compact_rows=compact, dw_dtype=dw_dtype,
                           norm_tokens=dp.global_token_count(wl.T, dev) if ctx.world > 1 else 0)
        self.ws = B.alloc_workspace(self.gp, dev)
        self.out = B.alloc_fwd_outputs(self.gp, dev)
        self.d_hidden = torch.empty_like(self.b.hidden)
        self.d_W = torch.empty(wl.V, wl.H, dtype=self.gp.dw_torch_dtype, device=dev)

    def with_params(self, **kw):
        """The same batch under other parameters (its own workspace)."""
        other = object.__new__(Leg)
        other.__dict__.update(self.__dict__)
        other.gp = dataclasses.replace(self.gp, **kw)
        other.ws = B.alloc_workspace(other.gp, self.ctx.dev)
        other.d_hidden = torch.empty_like(self.d_hidden)          # its own gradients: this leg's stay as they are
        other.d_W = torch.empty(self.wl.V, self.wl.H, dtype=other.gp.dw_torch_dtype, device=self.ctx.dev)
        return other

    def step(self, reduce=True):
        b, gp, out = self.b, self.gp, self.out
        B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets,
                         out=out, workspace=self.ws)
        if self.ctx.dist is not None and reduce:
            # data-parallel exchange: d_W summed over ranks slab by slab while the last panel is still computed
            red = dp.SlabAllReduce(self.d_W)
            B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_hidden=self.d_hidden,
                             d_W=self.d_W, workspace=self.ws, on_dw_slab=red)
            self.ctx.dist.all_reduce(out.loss)
            red.finish()
        else:
            B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_hidden=self.d_hidden,
                             d_W=self.d_W, workspace=self.ws)

    def timed(self, steps, warmup, reduce=True, per_kernel=False, clocks=True, min_seconds=0.0):
        """`warmup` untimed steps, then `steps` timed ones (at least `min_seconds` of them when given) between
        two CUDA events on the launching stream, barrier and synchronize on both sides, maximum over ranks."""
        ctx = self.ctx
        for _ in range(warmup):
            self.step(reduce)
        ctx.fence()
        assert B.check_status(self.ws) == B.OK, "device status word is set"
        if min_seconds > 0:             # size the leg from two more untimed steps
            p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            p0.record()
            self.step(reduce)
            self.step(reduce)
            p1.record()
            ctx.fence()
            est = ctx.max_over_ranks(p0.elapsed_time(p1) / 2)
            steps = int(min(5000, max(steps, math.ceil(min_seconds * 1e3 / max(est, 1e-3)))))
        sampler = ClockSampler(ctx.local_rank).start() if (clocks and ctx.rank == 0) else None
        launches0 = B.launch_count()
        if per_kernel:
            B.kernel_timing_begin()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ctx.fence()
        e0.record()
        for _ in range(steps):
            self.step(reduce)
        e1.record()
        ctx.fence()
        kt = B.kernel_timing_end() if per_kernel else None
        launches = B.launch_count() - launches0
        clk = sampler.stop() if sampler is not None else None
        ms_total = ctx.max_over_ranks(e0.elapsed_time(e1))
        assert B.check_status(self.ws) == B.OK
        return dict(ms_total=ms_total, steps=steps, warmup=warmup, launches=int(launches), kernels=kt, clocks=clk)

    def summary(self, t: dict, executed_rows_bwd=None) -> dict:
        """Throughput and tensor fractions of a timed region.  Executed flops = (2 T + 6 T_bwd) H V."""
        wl, ctx = self.wl, self.ctx
        ms = t["ms_total"] / t["steps"]
        t_bwd = wl.T if executed_rows_bwd is None else executed_rows_bwd
        tflops = (2.0 * wl.T + 6.0 * t_bwd) * wl.H * wl.V / (ms * 1e-3) / 1e12      # per GPU
        clk = t["clocks"]
        peaks = ctx.peaks
        return {"workload": wl.name, "T": wl.T, "H": wl.H, "V": wl.V, "sequences": wl.S, "dtype": wl.dtype,
                "is_mode": wl.is_mode, "mpt_mode": wl.mpt_mode,
                "value": ctx.world * wl.T / (ms * 1e-3), "unit": "tokens/s", "ms_per_step": ms,
                "mhz_ms": (ms * clk["sm_mhz"]) if clk and clk.get("sm_mhz") else None,
                "steps": t["steps"], "warmup": t["warmup"],
                "executed_tflops_per_gpu": tflops,
                "of_nominal_2250": tflops / NOMINAL_BF16_TFLOPS,
                "of_measured_burst": tflops / peaks["bf16_tflops"],
                "of_measured_sustained": tflops / peaks["bf16_tflops_sustained"],
                "clocks": clk}


def roofline_of(leg: Leg, t: dict, traffic_ok: bool) -> dict:
    wl, peaks = leg.wl, leg.ctx.peaks
    steps = t["steps"]
    ms_total = t["ms_total"]
    kt = t["kernels"]
    flops_kernel = 2.0 * wl.T * wl.H * wl.V                       # per step, each of the four kernels
    kinds = {k: {"ms_total": v[0], "launches": v[1],
                 "tflops": (flops_kernel * steps / (v[0] * 1e-3) / 1e12) if v[0] > 0 else None}
             for k, v in kt.items()}
    dom = max(kinds, key=lambda k: kinds[k]["ms_total"])
    if kinds[dom]["ms_total"] > 0:
        n_launch = max(kinds[dom]["launches"], 1)
        achieved = flops_kernel * steps / n_launch / (kinds[dom]["ms_total"] / n_launch * 1e-3) / 1e12
        peak = peaks["bf16_tflops_sustained"]
        return {"bound": "tensor", "kernel": f"umma_kernel<{dom}>", "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_kind": f"bf16 sustained, {peaks['source']}",
                "traffic": load_traffic(wl.name, dom) if traffic_ok else None,
                "flops_per_launch": flops_kernel * steps / n_launch,
                "avg_launch_ms": kinds[dom]["ms_total"] / n_launch, "per_kernel": kinds}
    # float32 workloads run on the CUDA-core kernels, which the per-kernel timer does not bracket
    achieved = 8.0 * wl.T * wl.H * wl.V * steps / (ms_total * 1e-3) / 1e12
    alu_peak = 148 * 128 * 2 * 1.965e9 / 1e12
    return {"bound": "alu", "kernel": "simt kernels (whole step)", "achieved": achieved, "peak": alu_peak,
            "unit": "TFLOP/s", "frac": achieved / alu_peak,
            "peak_kind": "fp32 FMA: 148 SMs x 128 lanes x 2 flop x 1.965 GHz", "traffic": None}


def e2e_run(leg: Leg, steps: int, dw_dtype: str) -> dict:
    """The whole step through the host-buffer entry point: pinned host inputs copied in, every result copied
    back, all inside the timed region (wall clock around synchronised steps, maximum over ranks)."""
    ctx, wl, hb_src = leg.ctx, leg.wl, leg.host_batch
    gp = dataclasses.replace(leg.gp, dw_dtype=dw_dtype, compact_rows=False)
    pin = lambda t: t.contiguous().pin_memory()
    hb = {k: pin(getattr(hb_src, k)) for k in ("hidden", "W", "targets", "old_logp", "segment_version",
                                               "advantages", "seq_offsets")}
    ho = dict(logp=torch.empty(wl.T).pin_memory(), entropy=torch.empty(wl.T).pin_memory(),
              flags=torch.empty(wl.T, dtype=torch.uint8).pin_memory(),
              seq_entropy=torch.empty(wl.S).pin_memory(), loss=torch.empty(1).pin_memory(),
              stats=torch.empty(leg.out.stats.numel(), dtype=torch.uint8).pin_memory(),
              d_hidden=torch.empty(wl.T, wl.H, dtype=leg.b.hidden.dtype).pin_memory(),
              d_W=torch.empty(wl.V, wl.H, dtype=gp.dw_torch_dtype).pin_memory())
    arena = torch.empty(B.host_step_arena_bytes(gp), dtype=torch.uint8, device=ctx.dev)
    host_step = lambda: B.token_loss_step_host(gp, arena, hb["hidden"], hb["W"], hb["targets"], hb["old_logp"],
                                               hb["segment_version"], hb["advantages"], hb["seq_offsets"], **ho)
    for _ in range(2):
        host_step()
        torch.cuda.synchronize()
    ctx.fence()
    t0 = time.perf_counter()
    for _ in range(steps):
        host_step()
        torch.cuda.synchronize()
    dt = ctx.max_over_ranks(time.perf_counter() - t0)
    ctx.fence()
    h2d = sum(t.numel() * t.element_size() for t in hb.values())
    d2h = sum(t.numel() * t.element_size() for t in ho.values())
    # outside the timed region: the host-buffer step reorders copies and launches, never results -- its
    # gradients are those of the device-resident step of this leg, bit for bit (a bf16 d_W: its rounding)
    checked = False
    if ctx.world == 1:          # (with several ranks the leg's d_W holds the sum over ranks)
        same_dh = bool(torch.equal(ho["d_hidden"].to(ctx.dev), leg.d_hidden))
        want_dw = leg.d_W if leg.d_W.dtype == ho["d_W"].dtype else leg.d_W.to(ho["d_W"].dtype)
        same_dw = bool(torch.equal(ho["d_W"].to(ctx.dev), want_dw))
        assert same_dh and same_dw, "host-buffer step and device-resident step disagree"
        checked = True
    return {"value": ctx.world * wl.T * steps / dt, "unit": "tokens/s", "ms_per_step": 1e3 * dt / steps,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": steps, "dw_dtype": dw_dtype,
            "loss": float(ho["loss"][0]), "gradients_equal_device_step": checked}


def library_gemm_reference(ctx: Context, seconds: float = 4.0) -> dict:
    """Context, not part of the path: the vendor library's bf16 GEMM (torch.matmul, 8192^3 and the LM-head shape
    with the logits written out) run for a few seconds right behind the legs above, i.e. in the thermal and
    power state they left.  Under the power cap the clock a kernel gets depends on that state, so this is the
    like-for-like denominator for the legs that ran last."""
    out = []
    for M, N, K in ((8192, 8192, 8192), (16384, 16384, 2048)):
        a = torch.randn(M, K, device=ctx.dev, dtype=torch.bfloat16)
        b = torch.randn(N, K, device=ctx.dev, dtype=torch.bfloat16)
        c = torch.empty(M, N, device=ctx.dev, dtype=torch.bfloat16)
        for _ in range(3):
            torch.matmul(a, b.t(), out=c)
        torch.cuda.synchronize()
        sampler = ClockSampler(ctx.local_rank).start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n, t0 = 0, time.perf_counter()
        e0.record()
        while time.perf_counter() - t0 < seconds / 2:
            for _ in range(20):
                torch.matmul(a, b.t(), out=c)
            n += 20
            torch.cuda.synchronize()
        e1.record()
        torch.cuda.synchronize()
        clk = sampler.stop()
        out.append({"kernel": "torch.matmul bf16 (cuBLAS)", "M": M, "N": N, "K": K,
                    "tflops": 2.0 * M * N * K * n / (e0.elapsed_time(e1) * 1e-3) / 1e12, "clocks": clk})
        del a, b, c
    return {"note": "library GEMM in the state the last legs left the GPU in; context only", "runs": out}


def run_ours(args, world, rank, local_rank):
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    ctx = Context(world, rank, local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=ctx.dev)
        ctx.dist = dist

    wl = synth.WORKLOADS[args.workload]
    reduced = args.tokens > 0
    if reduced:
        wl = wl.scaled(T=args.tokens, S=1, lengths="single", segment_len=max(1, args.tokens // wl.max_segments))
    warmup = max(args.warmup, 3) if not reduced else args.warmup
    full = args.legs == "all" and world == 1 and not reduced

    # ---- headline: dense forward + backward of the named workload
    leg = Leg(ctx, wl, panel=args.panel)
    t_main = leg.timed(args.steps, warmup, per_kernel=True)
    main = leg.summary(t_main)
    stats = leg.out.stats_host()
    roofline = roofline_of(leg, t_main, traffic_ok=(not reduced and args.panel == 0))

    # ---- what the d_W reduction costs on top of the compute (data-parallel runs)
    comm = None
    if world > 1:
        t_nc = leg.timed(max(3, args.steps // 2), 1, reduce=False, clocks=False)
        compute_ms = t_nc["ms_total"] / t_nc["steps"]
        comm = {"comm_exposed_ms": main["ms_per_step"] - compute_ms, "compute_only_ms_per_step": compute_ms,
                "dw_bytes_reduced_per_step": int(leg.d_W.numel() * leg.d_W.element_size()),
                "how": "d_W all-reduced in slabs of vocabulary rows behind the last backward panel (NCCL, own stream); "
                       "exposed = step with the reduction - step without it"}

    # ---- the same step with the backward restricted to the tokens whose coefficient is non-zero
    compacted = None
    if args.compact_steps > 0 and wl.dtype == "bf16":
        leg_c = leg.with_params(compact_rows=True)
        t_c = leg_c.timed(args.compact_steps, warmup, clocks=full)
        compacted = leg_c.summary(t_c, executed_rows_bwd=stats["n_active"])
        compacted.update(active_tokens=stats["n_active"], active_fraction=stats["n_active"] / wl.T,
                         note="backward contractions on tokens with a non-zero coefficient only; same results")
        del leg_c

    # ---- end to end through the host-buffer entry point
    e2e, e2e_bf16 = None, None
    if args.e2e_steps > 0:
        leg.ws = None
        torch.cuda.empty_cache()
        e2e = e2e_run(leg, args.e2e_steps, "f32")
        assert abs(e2e["loss"] - stats["loss"]) <= 1e-6 * max(1.0, abs(stats["loss"]))
        e2e["of_device_resident"] = e2e["value"] / main["value"]
        if full and wl.dtype == "bf16":
            e2e_bf16 = e2e_run(leg, args.e2e_steps, "bf16")
            e2e_bf16["of_device_resident"] = e2e_bf16["value"] / main["value"]
    host_batch = leg.host_batch
    del leg
    torch.cuda.empty_cache()

    # ---- the other gate state of the headline workload and the other named workloads
    gate_shut, others = None, []
    if full:
        if wl.name == "ultra":
            lg = Leg(ctx, synth.WORKLOADS["ultra_open"])
            tg = lg.timed(args.steps, warmup, per_kernel=True)
            gate_shut = lg.summary(tg)
            sg = lg.out.stats_host()
            per_kernel = roofline_of(lg, tg, False).get("per_kernel", {})
            gate_shut.update(mean_entropy=sg["mean_entropy"], n_masked=sg["n_masked"], n_active=sg["n_active"],
                             per_kernel_tflops={k: v["tflops"] for k, v in per_kernel.items()},
                             note="same shape as the headline with weaker plants: mean entropy above sigma, the gate "
                                  "of Eq. 10 stays shut and nothing is masked")
            del lg
            torch.cuda.empty_cache()
        for name in args.others.split(","):
            if not name or name == wl.name:
                continue
            lo = Leg(ctx, synth.WORKLOADS[name])
            to = lo.timed(10, warmup, min_seconds=LEG_SECONDS)
            so = lo.summary(to)
            st_o = lo.out.stats_host()
            so.update(mean_entropy=st_o["mean_entropy"], n_masked=st_o["n_masked"], n_active=st_o["n_active"])
            others.append(so)
            del lo
            torch.cuda.empty_cache()

    library_ref = library_gemm_reference(ctx) if full else None

    if rank != 0:
        if ctx.dist is not None:
            ctx.dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": main["value"], "unit": "tokens/s", "n_gpus": world, "steps": t_main["steps"],
        "warmup": warmup, "ms_per_step": main["ms_per_step"], "mhz_ms": main["mhz_ms"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
        "config": {"workload": wl.name + (" (reduced T)" if reduced else ""), "T": wl.T, "H": wl.H, "V": wl.V,
                   "sequences": wl.S, "is_mode": wl.is_mode, "mpt_mode": wl.mpt_mode,
                   "gate": "open" if stats["n_masked"] > 0 else "shut",
                   "l2": "inputs larger than L2 (hidden + W = 1.1 GB)", "parallelism": f"dp{world}"},
        "tensor_frac": {"executed_tflops_per_gpu": main["executed_tflops_per_gpu"],
                        "of_measured_burst": main["of_measured_burst"],
                        "of_measured_sustained": main["of_measured_sustained"],
                        "of_nominal_2250": main["of_nominal_2250"], "peaks": ctx.peaks["source"]},
        "loss": stats["loss"], "mean_entropy": stats["mean_entropy"], "n_masked": stats["n_masked"],
        "n_active": stats["n_active"],
        "roofline": roofline, "gate_shut": gate_shut, "other_workloads": others, "compacted": compacted,
        "e2e": e2e, "e2e_bf16_dw": e2e_bf16, "comm": comm, "library_gemm_same_state": library_ref,
        "gpu_launches": t_main["launches"], "clocks": main["clocks"],
    }
    if world == 1 and args.cpu_rows > 0:
        line["cpu_baseline"] = cpu_baseline(host_batch, args.cpu_rows)
    print(json.dumps(line))
    if ctx.dist is not None:
        ctx.dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="ultra", choices=list(synth.WORKLOADS))
    ap.add_argument("--legs", default="all", choices=["all", "main"],
                    help="all: also the gate-shut state, the other workloads and the bf16-d_W end-to-end run "
                         "(one GPU only); main: the headline workload alone")
    ap.add_argument("--others", default="small,qwen,mixed", help="workloads of the other_workloads legs")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--compact-steps", type=int, default=5, help="steps of the run with active-row compaction (0 = skip)")
    ap.add_argument("--cpu-rows", type=int, default=2048, help="rows of the CPU-baseline sample (0 = skip)")
    ap.add_argument("--ref-rows", type=int, default=256)
    ap.add_argument("--panel", type=int, default=0, help="backward panel tokens (0 = library default)")
    ap.add_argument("--tokens", type=int, default=0,
                    help="run the workload's recipe at this many tokens instead of its own T (small cases for "
                         "profiler captures; not the benchmark configuration)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    env = dp.world_from_env(args.gpus)          # raises when a launcher's world size is not --gpus
    if env is None and args.gpus > 1:
        # no launcher around this process: start one rank per GPU ourselves and hand over
        raise SystemExit(dp.launch_ranks(os.path.abspath(__file__), sys.argv[1:], args.gpus))
    world, rank, local_rank = env if env is not None else (1, 0, 0)
    run_ours(args, world, rank, local_rank)


if __name__ == "__main__":
    main()

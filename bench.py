"""Benchmark of the fused UloRL token-loss path (forward + backward) on synthetic batches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload ultra] [--impl ours|reference]

One step = one forward and one backward pass of the whole path over one batch.  The default
workload is the ultra-long single response (T=131072 tokens, H=2048, V=151936, bf16).  Rank 0
prints one JSON line.  `--impl reference` times the fp64 CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
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
from paper_2507_19766_b200 import synth  # noqa: E402

METRIC = "fused loss fwd+bwd tokens/sec at H=2048,V=151936; % of B200 bf16 tensor peak"
NOMINAL_BF16_TFLOPS = 2250.0
# DRAM bytes (read + write) per launch of each tensor-core kernel at the full ultra workload, from the ncu
# capture summarised in profiles/launch_list_ultra_full_size.md.  They describe the kernels as they were at
# that capture: set an entry to None when its kernel changes, until the counters are taken again.
NCU_TRAFFIC_BYTES = {"ultra": {"stats": 9.320e9, "dz": 8.847e9, "d_hidden": 12.524e9, "d_W": 13.737e9}}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


# ------------------------------------------------------------------ clocks during the timed region
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
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="ultra", choices=list(synth.WORKLOADS))
    ap.add_argument("--e2e-steps", type=int, default=2)
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

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    wl = synth.WORKLOADS[args.workload]
    if args.tokens > 0:
        wl = wl.scaled(T=args.tokens, S=1, lengths="single", segment_len=max(1, args.tokens // wl.max_segments))
    warmup = max(args.warmup, 3) if args.tokens == 0 else args.warmup
    host_batch = synth.make_batch(wl, seed=synth.BASE_SEED + wl.index + 1000 * rank, device=str(dev))
    b = host_batch.to(dev)
    gp = B.Params(T=wl.T, H=wl.H, V=wl.V, num_seqs=wl.S, dtype=wl.dtype, is_mode=wl.is_mode, mpt_mode=wl.mpt_mode,
                  clip_eps_low=wl.clip_eps_low, clip_eps_high=wl.clip_eps_high, mpt_tau=wl.mpt_tau,
                  entropy_target=wl.entropy_target, current_version=host_batch.current_version,
                  bwd_panel_tokens=args.panel,
                  norm_tokens=dp.global_token_count(wl.T, dev) if world > 1 else 0)
    ws = B.alloc_workspace(gp, dev)
    out = B.alloc_fwd_outputs(gp, dev)
    d_hidden = torch.empty_like(b.hidden)
    d_W = torch.empty(wl.V, wl.H, dtype=torch.float32, device=dev)

    def step():
        B.token_loss_fwd(gp, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages, b.seq_offsets,
                         out=out, workspace=ws)
        B.token_loss_bwd(gp, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_hidden=d_hidden, d_W=d_W,
                         workspace=ws)
        if dist is not None:         # data-parallel exchange: the summed head gradient and loss
            dp.reduce_step_outputs(d_W, out.loss)

    def fence():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(warmup):
        step()
    fence()
    assert B.check_status(ws) == B.OK, "device status word is set"

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = B.launch_count()
    B.kernel_timing_begin()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fence()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    fence()
    kt = B.kernel_timing_end()
    launches = B.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ms = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    ms_total = float(ms.item())
    tokens = world * wl.T * args.steps
    value = tokens / (ms_total * 1e-3)
    stats = out.stats_host()

    # ---- the same step with the backward restricted to the tokens whose coefficient is non-zero
    compacted = None
    if args.compact_steps > 0 and wl.dtype == "bf16":
        import dataclasses
        gp_c = dataclasses.replace(gp, compact_rows=True)
        ws_c = B.alloc_workspace(gp_c, dev)

        def step_c():
            B.token_loss_fwd(gp_c, b.hidden, b.W, b.targets, b.old_logp, b.segment_version, b.advantages,
                             b.seq_offsets, out=out, workspace=ws_c)
            B.token_loss_bwd(gp_c, b.hidden, b.W, b.targets, out.lse, out.grad_coef, d_hidden=d_hidden, d_W=d_W,
                             workspace=ws_c)
            if dist is not None:
                dp.reduce_step_outputs(d_W, out.loss)

        for _ in range(warmup):
            step_c()
        fence()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        for _ in range(args.compact_steps):
            step_c()
        c1.record()
        fence()
        assert B.check_status(ws_c) == B.OK
        cms = torch.tensor([c0.elapsed_time(c1)], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(cms, op=dist.ReduceOp.MAX)
        cms = float(cms.item())
        t_act = stats["n_active"]
        compacted = {"value": world * wl.T * args.compact_steps / (cms * 1e-3), "unit": "tokens/s",
                     "ms_per_step": cms / args.compact_steps, "steps": args.compact_steps,
                     "active_tokens": t_act, "active_fraction": t_act / wl.T,
                     "executed_tflops_per_gpu": (2.0 * wl.T + 6.0 * t_act) * wl.H * wl.V * args.compact_steps
                                                / (cms * 1e-3) / 1e12,
                     "note": "backward contractions on tokens with a non-zero coefficient only; same results"}
        del ws_c

    # ---- end to end through the host-buffer entry point
    e2e = None
    if args.e2e_steps > 0:
        pin = lambda t: t.contiguous().pin_memory()
        hb = {k: pin(getattr(host_batch, k)) for k in ("hidden", "W", "targets", "old_logp", "segment_version",
                                                      "advantages", "seq_offsets")}
        ho = dict(logp=torch.empty(wl.T).pin_memory(), entropy=torch.empty(wl.T).pin_memory(),
                  flags=torch.empty(wl.T, dtype=torch.uint8).pin_memory(),
                  seq_entropy=torch.empty(wl.S).pin_memory(), loss=torch.empty(1).pin_memory(),
                  stats=torch.empty(out.stats.numel(), dtype=torch.uint8).pin_memory(),
                  d_hidden=torch.empty(wl.T, wl.H, dtype=b.hidden.dtype).pin_memory(),
                  d_W=torch.empty(wl.V, wl.H).pin_memory())
        del ws
        torch.cuda.empty_cache()
        arena = torch.empty(B.host_step_arena_bytes(gp), dtype=torch.uint8, device=dev)
        host_step = lambda: B.token_loss_step_host(gp, arena, hb["hidden"], hb["W"], hb["targets"], hb["old_logp"],
                                                   hb["segment_version"], hb["advantages"], hb["seq_offsets"], **ho)
        host_step()
        fence()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            host_step()
            torch.cuda.synchronize()
        fence()
        dt = torch.tensor([time.perf_counter() - t0], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(dt, op=dist.ReduceOp.MAX)
        h2d = sum(t.numel() * t.element_size() for t in hb.values())
        d2h = sum(t.numel() * t.element_size() for t in ho.values())
        assert abs(float(ho["loss"][0]) - stats["loss"]) <= 1e-6 * max(1.0, abs(stats["loss"]))
        e2e = {"value": world * wl.T * args.e2e_steps / float(dt.item()), "unit": "tokens/s",
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": args.e2e_steps}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    flops_kernel = 2.0 * wl.T * wl.H * wl.V                       # per step, each of the four kernels
    kinds = {k: {"ms_total": v[0], "launches": v[1],
                 "tflops": (flops_kernel * args.steps / (v[0] * 1e-3) / 1e12) if v[0] > 0 else None}
             for k, v in kt.items()}
    dom = max(kinds, key=lambda k: kinds[k]["ms_total"])
    if kinds[dom]["ms_total"] > 0:
        n_launch = max(kinds[dom]["launches"], 1)
        achieved = flops_kernel * args.steps / n_launch / (kinds[dom]["ms_total"] / n_launch * 1e-3) / 1e12
        peak = peaks["bf16_tflops_sustained"]
        roofline = {"bound": "tensor", "kernel": f"umma_kernel<{dom}>", "achieved": achieved, "peak": peak,
                    "unit": "TFLOP/s", "frac": achieved / peak,
                    "peak_kind": f"bf16 sustained, {peaks['source']}",
                    "traffic": (NCU_TRAFFIC_BYTES.get(wl.name, {}).get(dom)
                                if args.tokens == 0 and args.panel == 0 else None),
                    "flops_per_launch": flops_kernel * args.steps / n_launch,
                    "avg_launch_ms": kinds[dom]["ms_total"] / n_launch, "per_kernel": kinds}
    else:   # float32 workloads run on the CUDA-core kernels, which the per-kernel timer does not bracket
        achieved = 8.0 * wl.T * wl.H * wl.V * args.steps / (ms_total * 1e-3) / 1e12
        roofline = {"bound": "alu", "kernel": "simt kernels (whole step)", "achieved": achieved,
                    "peak": 148 * 128 * 2 * 1.965e9 / 1e12, "unit": "TFLOP/s",
                    "frac": achieved / (148 * 128 * 2 * 1.965e9 / 1e12),
                    "peak_kind": "fp32 FMA: 148 SMs x 128 lanes x 2 flop x 1.965 GHz", "traffic": None}
    exec_tflops = 8.0 * wl.T * wl.H * wl.V * world * args.steps / (ms_total * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": wl.dtype, "data": "synthetic",
        "config": {"workload": wl.name + (" (reduced T)" if args.tokens > 0 else ""), "T": wl.T, "H": wl.H, "V": wl.V, "sequences": wl.S,
                   "is_mode": wl.is_mode, "mpt_mode": wl.mpt_mode, "l2": "inputs larger than L2 (hidden + W = 1.1 GB)",
                   "parallelism": f"dp{world}"},
        "tensor_frac": {"executed_tflops_per_gpu": exec_tflops / world,
                        "of_measured_burst": exec_tflops / world / peaks["bf16_tflops"],
                        "of_measured_sustained": exec_tflops / world / peaks["bf16_tflops_sustained"],
                        "of_nominal_2250": exec_tflops / world / NOMINAL_BF16_TFLOPS, "peaks": peaks["source"]},
        "loss": stats["loss"], "mean_entropy": stats["mean_entropy"], "n_masked": stats["n_masked"],
        "n_active": stats["n_active"],
        "roofline": roofline, "compacted": compacted, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
    }
    if world == 1 and args.cpu_rows > 0:
        line["cpu_baseline"] = cpu_baseline(host_batch, args.cpu_rows)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

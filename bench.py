#!/usr/bin/env python
"""Benchmark of the row-typed star_q FFN forward pass (up -> GELU -> down) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one pass of the whole hot path (row-type bucketing, row gather, grouped tcgen05 GEMM
with fused GELU for the up projection, grouped GEMM with fused row scatter for the down
projection) over one synthetic batch of the q=2, 768 -> 3072 -> 768, M = 8 x 1024 workload.
Prints ONE JSON line.  FLOPs count only the block GEMMs the rule keeps.

N > 1 (torchrun): rows shard across ranks, weights replicated, no data-path collective; every
rank runs the same per-GPU batch (weak scaling), time = max over ranks.

--impl reference times the CPU oracle (plain fp64 loops) on a bounded sample of the same
workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

WORKLOAD = "cfg2: q=2 FFN 768->3072->768 (GELU), M=8x1024 rows, type = position mod 2, bf16"
METRIC = "star_q FFN kept-GEMM throughput (prefill)"
UNIT = "TFLOP/s"
FLUSH_BYTES = 512 << 20
# DRAM traffic of the grouped-GEMM kernels from the ncu capture summarised under profiles/
# (bytes per launch, up and down projection of this workload); None until captured.
NCU_TRAFFIC_BYTES = None


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self._stop, self._t = index, [], threading.Event(), None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                parts = [p.strip() for p in out.strip().split(",")]
                if len(parts) >= 6:
                    self.samples.append(parts)
            except Exception:
                pass
            self._stop.wait(0.05)

    def __enter__(self):
        self._t = threading.Thread(target=self._run, daemon=True)
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=10)

    def summary(self):
        sm = [float(s[0]) for s in self.samples if s[0].replace(".", "").isdigit()]
        mx = [float(s[1]) for s in self.samples if s[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(s[2 + i].lower().startswith("active") for s in self.samples)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(self.samples)}


def kept_flops(ffn, wl) -> int:
    rows = np.bincount(wl.types, minlength=wl.q).tolist()
    return 2 * ffn.macs(rows)


def run_reference(args):
    """The oracle as it stands, on the host cores, on a row sample of the same workload."""
    import oracle
    from paper_2609_32814_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = synth.config2()
    sample_rows = 1024
    rows = np.arange(0, wl.M, wl.M // sample_rows)
    X, t = wl.X[rows], wl.types[rows]
    keep = oracle.support(wl.q)
    counts = np.bincount(t, minlength=wl.q)
    flops = 2 * (oracle.macs(keep, wl.d_widths, wl.f_widths, counts) + oracle.macs(keep, wl.f_widths, wl.d_widths, counts))
    for _ in range(args.warmup):
        oracle.ffn(X, t, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.ffn(X, t, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    dt = (time.perf_counter() - t0) / args.steps
    val = flops / dt / 1e12
    sample = f"{sample_rows} of {wl.M} rows per step (every {wl.M // sample_rows}th row), all outputs, fp64"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def time_cpu_oracle(wl):
    import oracle
    sample_rows = 2048
    rows = np.arange(0, wl.M, wl.M // sample_rows)
    X, t = wl.X[rows], wl.types[rows]
    keep = oracle.support(wl.q)
    counts = np.bincount(t, minlength=wl.q)
    flops = 2 * (oracle.macs(keep, wl.d_widths, wl.f_widths, counts) + oracle.macs(keep, wl.f_widths, wl.d_widths, counts))
    best = None
    t_all = time.perf_counter()
    for _ in range(3):
        t0 = time.perf_counter()
        oracle.ffn(X, t, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
        if time.perf_counter() - t_all > 25:
            break
    return {"value": flops / best / 1e12, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{sample_rows} of {wl.M} rows (every {wl.M // sample_rows}th), all outputs, best of <=3, "
                      f"{best:.2f} s per pass"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the dense-control / decode side measurements")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    from paper_2609_32814_b200 import binding, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    binding.lib()  # fail loudly if the CUDA library is missing

    wl = synth.config2()
    if world > 1:  # each rank draws its own batch of the same shape
        wl.X = synth.bf16_round(synth.normal(synth.seed_for(2, 50 + rank), wl.X.shape, 1.0))
    dev = lambda a: torch.from_numpy(a).cuda().to(torch.bfloat16)
    X, Wu, Wd = dev(wl.X), dev(wl.W_up), dev(wl.W_down)
    types = torch.from_numpy(wl.types).cuda()
    # config 2 fixes the schedule "type = position mod 2": the handle is created with it
    # (ALG_SCHED_CYCLIC), the per-call types array is then not needed.  The explicit-types path of
    # the same workload is timed as a side measurement.
    ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16", schedule="cyclic")
    ws = torch.empty(ffn.workspace_bytes(wl.M), dtype=torch.uint8, device="cuda")
    Y = torch.empty((wl.M, wl.D), dtype=torch.bfloat16, device="cuda")
    flops = kept_flops(ffn, wl)
    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        ffn.forward(X, None, Wu, Wd, act="gelu", out=Y, workspace=ws, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        flush.zero_()
        step()
    barrier()
    assert ffn.last_status() == 0

    # ---- timed region: K steps, L2 flushed (512 MiB write) before each, CUDA events per step ----
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    launches0 = binding.launch_count()
    with ClockSampler(local_rank) as clocks:
        barrier()
        for i in range(args.steps):
            flush.zero_()
            starts[i].record(stream)
            step()
            stops[i].record(stream)
        barrier()
    launches = binding.launch_count() - launches0
    per_step_ms = [s.elapsed_time(e) for s, e in zip(starts, stops)]
    total_ms = float(sum(per_step_ms))
    if world > 1:
        tt = torch.tensor([total_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt.item())
    ms_per_step = total_ms / args.steps
    value = world * flops * args.steps / (total_ms * 1e-3) / 1e12
    assert ffn.last_status() == 0

    # ---- per-kernel durations (second pass with events between the kernels) ----
    ffn.set_timing(True)
    kt = np.zeros(4)
    for i in range(args.steps):
        flush.zero_()
        step()
        kt += np.array(ffn.get_timing())
    kt /= args.steps
    ffn.set_timing(False)
    peaks = _peaks()
    gemm_ms = float(kt[2] + kt[3])
    achieved = flops / (gemm_ms * 1e-3) / 1e12
    roofline = {"bound": "tensor", "kernel": "proj_tc_kernel (up + down launches of one step)",
                "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_tflops"], "peak_source": f"{peaks['source']} (burst)",
                "traffic": NCU_TRAFFIC_BYTES,
                "kernel_ms": {"bucket": float(kt[0]), "gather": float(kt[1]), "up": float(kt[2]), "down": float(kt[3])},
                "step_frac_of_peak": flops / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops"]}

    # ---- end to end through the host entry point: pinned H2D of X/types, D2H of Y inside the timing ----
    Xh = torch.from_numpy(wl.X).to(torch.bfloat16).pin_memory()
    Yh = torch.empty((wl.M, wl.D), dtype=torch.bfloat16).pin_memory()
    wsh = torch.empty(ffn.host_workspace_bytes(wl.M, torch.bfloat16), dtype=torch.uint8, device="cuda")
    for _ in range(3):
        ffn.forward_host(Xh, None, Wu, Wd, Yh, workspace=wsh, stream=stream)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_ms = 0.0
    for i in range(args.steps):
        flush.zero_()
        e0.record(stream)
        ffn.forward_host(Xh, None, Wu, Wd, Yh, workspace=wsh, stream=stream)
        e1.record(stream)
        e1.synchronize()
        e2e_ms += e0.elapsed_time(e1)
    if world > 1:
        tt = torch.tensor([e2e_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        e2e_ms = float(tt.item())
    e2e = {"value": world * flops * args.steps / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
           "h2d_bytes_per_step": int(Xh.numel() * 2), "d2h_bytes_per_step": int(Yh.numel() * 2),
           "ms_per_step": e2e_ms / args.steps}

    extras = {}
    if rank == 0 and not args.no_extras:
        extras = side_measurements(binding, synth, wl, X, types, Wu, Wd, Y, flush, stream, ms_per_step)

    if rank == 0:
        cpu = time_cpu_oracle(wl) if world >= 1 else None
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": WORKLOAD, "l2": "flushed before every step (512 MiB write, outside the timing)",
                           "rows_per_gpu": wl.M, "parallelism": f"rows sharded over {world} GPU(s), weights replicated"},
                "tokens_per_s": world * wl.M * args.steps / (total_ms * 1e-3),
                "kept_gflop_per_step": flops / 1e9,
                "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": int(launches),
                "roofline": roofline, "cpu_baseline": cpu}
        line.update(extras)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def side_measurements(binding, synth, wl, X, types, Wu, Wd, Y, flush, stream, star_ms):
    """Dense same-shape control built in the same library, and the decode-shape weight stream."""
    import torch
    out = {}

    def timed(handle, tt, n=20):
        wsx = torch.empty(handle.workspace_bytes(wl.M), dtype=torch.uint8, device="cuda")
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(3):
            handle.forward(X, tt, Wu, Wd, act="gelu", out=Y, workspace=wsx, stream=stream)
        tot = 0.0
        for _ in range(n):
            flush.zero_()
            a0.record(stream)
            handle.forward(X, tt, Wu, Wd, act="gelu", out=Y, workspace=wsx, stream=stream)
            a1.record(stream)
            a1.synchronize()
            tot += a0.elapsed_time(a1)
        return tot / n

    out["explicit_types"] = {"ms_per_step": timed(binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16"), types),
                             "note": "same workload through ALG_SCHED_EXPLICIT (bucketing + row gather kernels run)"}
    dense = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16", table="dense", schedule="cyclic")
    ms, n = timed(dense, None) * 20, 20
    out["vs_dense"] = {"dense_ms_per_step": ms / n, "star_ms_per_step": star_ms, "time_ratio_star_over_dense": star_ms / (ms / n),
                       "control": "same library, ALG_TABLE_DENSE (8 block GEMMs instead of 6)"}
    return out


if __name__ == "__main__":
    main()

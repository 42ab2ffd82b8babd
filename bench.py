#!/usr/bin/env python
"""Benchmark of the row-typed star_q FFN forward pass (up -> GELU -> down) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

One step = one pass of the whole hot path over one synthetic batch: grouped tcgen05 GEMM with
fused GELU for the up projection, grouped GEMM with fused row scatter for the down projection;
with explicit row types also the bucketing and row-gather kernels.  Prints ONE JSON line.  FLOPs
count only the block GEMMs the rule keeps.

--config selects the workload (default 2, the q=2 768 -> 3072 -> 768 FFN at M = 8 x 1024 rows):
    2                  q=2 FFN of the ~110M model, type = position mod 2 (cyclic schedule)
    3q4 3q8            general q, groups of 128 / 512, M = 16384, i.i.d. row types
    4                  KV-cached decode step, M in {1, 8, 32, 64}: 64-layer dependent FFN chain
    5q2 5q4 5q8 5q16   scale sweep 4096 -> 16384 -> 4096, M = 32768, i.i.d. row types
    pilot              tensor-square law Q_2 (x) Q_2 at the paper's pilot shape (768 -> 1536 -> 768)
    gpilot g8b         gated (SwiGLU) FFN with merged gate/up bank: the pilot's FFN; 4096 -> 12288 at q=32
    train2 train8b     forward + both gradient maps of one projection (768 -> 3072 at q=2; 4096 -> 12288 at q=32)
    kp1p7b kp4b kp8b kp30b kpdsv3  the expansion projections of the paper's main kernel table (M = 2048)
    sq4096 .. sq32768  square product of two n x n algebra elements with 128 x 128 blocks (q = n / 128 up to 256);
                       sq<n>b256: the same with 256 x 256 blocks
    qwu<q>m<M> qwd<q>m<M>  one projection 5120 -> 25600 (u) or 25600 -> 5120 (d) cut into q in {32, 64, 128, 256} equal
                       groups (blocks 160 x 800 ... 20 x 100), M in {2048, 8192, 32768} rows, type = row block

N > 1 (torchrun): rows shard across ranks, weights replicated, no data-path collective; every
rank runs the same per-GPU batch (weak scaling), time = max over ranks.

--impl reference times the CPU oracle (plain fp64 loops) on a bounded sample of the same
workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "star_q FFN kept-GEMM throughput (prefill)"
UNIT = "TFLOP/s"
BIG_METRIC = "star_q projection kept-GEMM throughput (large algebra, fixed blocks)"
N_SETS = 6            # working sets of configuration 2
L2_BYTES = 126e6

CONFIGS = {
    "2": dict(q=2, D=768, F=3072, M=8192, law="qq", schedule="cyclic",
              label="cfg2: q=2 FFN 768->3072->768 (GELU), M=8x1024 rows, type = position mod 2, bf16"),
    "3q4": dict(q=4, D=512, F=2048, M=16384, law="qq", schedule="explicit",
                label="cfg3: q=4 FFN 512->2048->512 (groups of 128 / 512), M=16384 rows, i.i.d. row types, bf16"),
    "3q8": dict(q=8, D=1024, F=4096, M=16384, law="qq", schedule="explicit",
                label="cfg3: q=8 FFN 1024->4096->1024 (groups of 128 / 512), M=16384 rows, i.i.d. row types, bf16"),
    "5q2": dict(q=2, D=4096, F=16384, M=32768, law="qq", schedule="explicit",
                label="cfg5: q=2 FFN 4096->16384->4096, M=32768 rows, i.i.d. row types, bf16"),
    "5q4": dict(q=4, D=4096, F=16384, M=32768, law="qq", schedule="explicit",
                label="cfg5: q=4 FFN 4096->16384->4096, M=32768 rows, i.i.d. row types, bf16"),
    "5q8": dict(q=8, D=4096, F=16384, M=32768, law="qq", schedule="explicit",
                label="cfg5: q=8 FFN 4096->16384->4096, M=32768 rows, i.i.d. row types, bf16"),
    "5q16": dict(q=16, D=4096, F=16384, M=32768, law="qq", schedule="explicit",
                 label="cfg5: q=16 FFN 4096->16384->4096, M=32768 rows, i.i.d. row types, bf16"),
    "pilot": dict(q=4, D=768, F=1536, M=8 * 1536, law="q2pow", schedule="interval", period=768,
                  label="pilot: Q_2 (x) Q_2 FFN 768->1536->768 (4 x 192 / 4 x 384), M=8x1536 rows, interval schedule, bf16"),
    "gpilot": dict(q=4, D=768, F=1536, M=8 * 1536, law="q2pow", schedule="interval", period=768, gated=True,
                   label="gated pilot: bias-free SwiGLU FFN 768->1536->768 under Q_2 (x) Q_2 (4 x 192 / 4 x 384), merged gate/up "
                         "bank, M=8x1536 rows, interval schedule, bf16"),
    "g8b": dict(q=32, D=4096, F=12288, M=2048, law="qq", schedule="explicit", gated=True,
                label="gated FFN 4096->12288->4096 at q=32 (groups of 128 / 384), merged gate/up bank, M=2048 rows, "
                      "i.i.d. row types, bf16"),
    "train2": dict(q=2, D=768, F=3072, M=8192, law="qq", schedule="cyclic", train=True,
                   label="training step of one projection: forward + dX + dW of the cfg2 up projection 768->3072, q=2, M=8192 rows, "
                         "type = position mod 2, bf16"),
    "train8b": dict(q=32, D=4096, F=12288, M=2048, law="qq", schedule="explicit", train=True,
                    label="training step of one projection: forward + dX + dW of 4096->12288 at q=32 (groups of 128 / 384), "
                          "M=2048 rows, i.i.d. row types, bf16"),
    "4": dict(q=2, D=768, F=3072, M=64, law="qq", schedule="explicit",
              label="cfg4: KV-cached decode step, q=2 FFN 768->3072->768, M in {1,8,32,64}, type = position mod 2, bf16"),
}


def _large_algebra_configs():
    """Fixed-block workloads of the paper's kernel study (appendix "Large Projections and Square Products");
    paper_ms = the warm median the paper prints for its own kernel on an H200 NVL, kept for context."""
    out = {}
    for n, q, ms in ((4096, 32, 0.044), (8192, 64, 0.166), (16384, 128, 0.689), (32768, 256, 2.868)):
        out[f"sq{n}"] = dict(big=True, q=q, s=128, r=128, M=n, schedule="interval", paper_ms=ms,
                             label=f"square product of two n={n} algebra elements, 128x128 blocks (q={q}): typed projection "
                                   f"{n}->{n} with type = block row, bf16")
    for n, q, ms in ((4096, 16, 0.058), (8192, 32, 0.225), (16384, 64, 0.991), (32768, 128, 5.344)):
        out[f"sq{n}b256"] = dict(big=True, q=q, s=256, r=256, M=n, schedule="interval", paper_ms=ms,
                                 label=f"square product of two n={n} algebra elements, 256x256 blocks (q={q}): typed projection "
                                       f"{n}->{n} with type = block row, bf16")
    paper = {("u", 32, 2048): 0.168, ("u", 64, 2048): 0.232, ("u", 128, 2048): 0.248, ("u", 32, 8192): 0.583,
             ("u", 64, 8192): 0.523, ("u", 128, 8192): 0.401, ("u", 32, 32768): 2.335, ("u", 64, 32768): 2.055,
             ("u", 128, 32768): 1.558, ("d", 32, 2048): 0.181, ("d", 64, 2048): 0.147, ("d", 128, 2048): 0.174,
             ("d", 32, 8192): 0.576, ("d", 64, 8192): 0.396, ("d", 128, 8192): 0.411, ("d", 32, 32768): 2.354,
             ("d", 64, 32768): 1.519, ("d", 128, 32768): 1.684,
             ("u", 256, 2048): 0.266, ("u", 256, 8192): 0.414, ("u", 256, 32768): 1.169,
             ("d", 256, 2048): 0.243, ("d", 256, 8192): 0.552, ("d", 256, 32768): 1.958}
    # the paper's main kernel table (M = 2048 rows, the q it selects): model shape -> (K, N, q, its kernel's ms)
    # (the last figure: the paper's kernel at M = 1 with q = 32, its fixed-q table, in microseconds)
    for name, (K, N, q, ms, m1_us) in {"kp1p7b": (2048, 6144, 32, 0.0249, 3.8), "kp4b": (2560, 9728, 32, 0.0511, 4.1),
                                       "kp8b": (4096, 12288, 32, 0.0636, 4.4), "kp30b": (2048, 768, 16, 0.0084, 3.3),
                                       "kpdsv3": (7168, 2048, 16, 0.0283, 3.8)}.items():
        out[name] = dict(big=True, q=q, s=K // q, r=N // q, M=2048, schedule="interval", paper_ms=ms, paper_m1_us=m1_us,
                         label=f"projection {K}->{N} in q={q} equal groups, X as q x q blocks of {2048 // q}x{K // q}, "
                               f"W of {K // q}x{N // q}, M=2048 rows, type = row block, bf16")
    for (way, q, M), ms in paper.items():
        K, N = (5120, 25600) if way == "u" else (25600, 5120)
        out[f"qw{way}{q}m{M}"] = dict(big=True, q=q, s=K // q, r=N // q, M=M, schedule="interval", paper_ms=ms,
                                      label=f"projection {K}->{N} in q={q} equal groups, X as q x q blocks of {M // q}x{K // q}, "
                                            f"W of {K // q}x{N // q}, M={M} rows, type = row block, bf16")
    return out


CONFIGS.update(_large_algebra_configs())


def _gated_table_configs():
    """The public shapes of the paper's gated-FFN table (complete SwiGLU FFN forward, q = 32, merged gate/up; appendix
    "Kernel Benchmark Details"): M = 2048 rows is the step, the M = 1 row is measured beside it as a chain of
    layers in one CUDA graph.  paper_us = the paper's own kernel on its H200 NVL at (M = 1, M = 2048)."""
    out = {}
    for tag, D, F, m1, m2048 in (("1p7b", 2048, 6144, 8.7, 107.4), ("4b", 2560, 9728, 10.4, 193.8), ("8b", 4096, 12288, 12.6, 247.3),
                                 ("30b", 2048, 768, 6.7, 23.2), ("dsv3", 7168, 2048, 8.5, 81.3)):
        out[f"gt{tag}"] = dict(q=32, D=D, F=F, M=2048, law="qq", schedule="explicit", gated=True, paper_us=(m1, m2048),
                               label=f"gated FFN {D}->{F}->{D} at q=32 (groups of {D // 32} / {F // 32}), merged gate/up bank, "
                                     "M=2048 rows, i.i.d. row types, bf16")
    return out


CONFIGS.update(_gated_table_configs())
CONFIGS["g8b"]["paper_us"] = (12.6, 247.3)
WORKLOAD = CONFIGS["2"]["label"]


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "hbm_gbs": float(p["hbm_gbs"]), "source": "measured",
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", 0.0)) or None}
    return {"bf16_tflops": 1590.0, "hbm_gbs": 6650.0, "source": "fallback", "bf16_tflops_sustained": 1400.0}


class ClockSampler:
    """Samples SM clock and throttle reasons (NVML, read-only) while the timed region runs.
    Sampling starts with the context; only samples taken after arm() -- called once the first
    launch of the timed region is enqueued -- count."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.index, self.samples, self._stop, self._t = index, [], threading.Event(), None
        self.max_mhz = None
        self.t_arm = None

    def arm(self):
        if self.t_arm is None:
            self.t_arm = time.time()

    def _run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while not self._stop.is_set():
                mhz = pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)
                mask = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
                self.samples.append((float(mhz), int(mask), time.time()))
                self._stop.wait(0.001)
        except Exception:
            self._run_smi()

    def _run_smi(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        bits = [0x8, 0x40, 0x20, 0x4]
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-i",
                                      str(self.index)], capture_output=True, text=True, timeout=5).stdout
                parts = [p.strip() for p in out.strip().split(",")]
                if len(parts) >= 6:
                    self.max_mhz = float(parts[1])
                    mask = sum(b for b, v in zip(bits, parts[2:6]) if v.lower().startswith("active"))
                    self.samples.append((float(parts[0]), mask, time.time()))
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

    def armed_samples(self):
        return [s for s in self.samples if self.t_arm is not None and s[2] >= self.t_arm]

    def summary(self):
        live = self.armed_samples()
        sm = [s[0] for s in live]
        mask = 0
        for s in live:
            mask |= s[1]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": self.max_mhz,
                "reasons": [n for b, n in self.REASONS.items() if mask & b], "samples": len(live)}


def extend_clock_record(clocks, step, local_rank, torch):
    """When the timed region was too short for five clock samples, the same steps run on, untimed, under a
    second sampler for a quarter of a second so that the clock record covers this load.  Returns the note
    that goes beside the record."""
    if len(clocks.armed_samples()) >= 5:
        return "sampled during the timed region"
    with ClockSampler(local_rank) as clocks2:
        t_end = time.time() + 0.25
        i = 0
        while time.time() < t_end:
            for _ in range(20):
                step(i)
                i += 1
            clocks2.arm()
            torch.cuda.synchronize()
    clocks.samples = clocks.armed_samples() + clocks2.armed_samples()
    clocks.t_arm = min([s[2] for s in clocks.samples], default=None)
    clocks.max_mhz = clocks.max_mhz or clocks2.max_mhz
    return "timed region too short for five samples: extended by 0.25 s of the same steps, untimed"


def max_over_ranks(value: float, device=None) -> float:
    """Multi-rank timing rule: the job is as slow as its slowest rank (no-op without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_batch_seed(rank: int, world: int, set_index: int) -> int:
    """Seed of working set `set_index` on `rank`: every rank draws its own rows (rows shard across
    ranks, weights are replicated); rank 0 of a single-GPU run keeps the parity-test batch."""
    from paper_2609_32814_b200 import synth
    return synth.seed_for(2, 50 + rank * N_SETS + set_index)


def whole_job_value(flops_per_rank_step: int, world: int, steps: int, total_ms: float) -> float:
    """Weak scaling: every rank runs the same per-GPU batch; value = work of all ranks / slowest rank's time."""
    return world * flops_per_rank_step * steps / (total_ms * 1e-3) / 1e12


def make_workload(name: str):
    """The synthetic problem of a configuration (host arrays; the parity tests use the same generators)."""
    from paper_2609_32814_b200 import synth
    if name == "2":
        return synth.config2()
    if name in ("3q4", "3q8"):
        return synth.config3(CONFIGS[name]["q"])
    if name.startswith("5q"):
        return synth.config5(CONFIGS[name]["q"])
    if name == "pilot":
        return synth.pilot_ffn(M=CONFIGS[name]["M"])
    if name == "4":
        return synth.config4(64)
    if name in ("gpilot", "g8b") or name.startswith("gt"):
        cfg = CONFIGS[name]
        types = synth.interval_types(cfg["M"], 4, 768) if name == "gpilot" else synth.uniform_types(synth.seed_for(8, 32), cfg["M"], cfg["q"])
        wl, Wg = synth.gated_ffn(name, cfg["q"], cfg["M"], cfg["D"], cfg["F"], types, variant=7)
        wl.meta["W_gate"] = Wg
        return wl
    raise ValueError(name)


def oracle_sample(name: str, wl, budget_macs: float = 2.0e11):
    """Rows of the workload the CPU oracle is timed on: evenly spaced, about `budget_macs` of work."""
    import oracle
    cfg = CONFIGS[name]
    keep = oracle.support(wl.q, cfg["law"])
    up_factor = 2 if cfg.get("gated") else 1      # gate and up are two D x F projections
    per_row = (up_factor * oracle.macs(keep, wl.d_widths, wl.f_widths, np.ones(wl.q, dtype=np.int64)) +
               oracle.macs(keep, wl.f_widths, wl.d_widths, np.ones(wl.q, dtype=np.int64))) / wl.q
    n = int(min(wl.M, max(16, 2 ** int(math.log2(max(16.0, budget_macs / per_row))))))
    rows = np.arange(0, wl.M, max(1, wl.M // n))[:n]
    counts = np.bincount(wl.types[rows], minlength=wl.q)
    flops = 2 * (up_factor * oracle.macs(keep, wl.d_widths, wl.f_widths, counts) + oracle.macs(keep, wl.f_widths, wl.d_widths, counts))
    return rows, keep, flops


def oracle_ffn(name, wl, rows, keep):
    import oracle
    if CONFIGS[name].get("gated"):
        return oracle.ffn_swiglu(wl.X[rows], wl.types[rows], wl.meta["W_gate"], wl.W_up, wl.W_down, wl.d_widths, wl.f_widths, keep=keep)
    return oracle.ffn(wl.X[rows], wl.types[rows], wl.W_up, wl.W_down, wl.d_widths, wl.f_widths, keep=keep)


def big_oracle_sample(cfg, budget_macs: float = 6.0e10):
    """Sample of a large-algebra workload the CPU oracle can hold: the rows of the first q' types and the output
    groups of the same types.  Because B(i,j) = {i,j}, that is the Q_q' projection over the same blocks, and its
    outputs are outputs of the full problem.  Returns (callable, flops, description)."""
    import oracle
    from paper_2609_32814_b200 import synth
    q, s, r, M = cfg["q"], cfg["s"], cfg["r"], cfg["M"]
    qs = min(q, 32)
    per_row = (2 * qs - 1) * s * r
    n = int(max(qs, min(qs * (M // q), budget_macs // per_row)))
    n -= n % qs
    types = synth.cyclic_types(n, qs)
    X = synth.bf16_round(synth.normal(synth.seed_for(9, 1), (n, qs * s), 1.0))
    W = synth.bf16_round(synth.normal(synth.seed_for(9, 2), (qs * s, qs * r), 0.02))
    flops = 2 * n * per_row
    desc = f"{n} rows of {qs} of the {q} types, output groups of the same types (the Q_{qs} projection over the same {s}x{r} blocks), fp64"
    return (lambda: oracle.proj(X, types, W, [s] * qs, [r] * qs)), flops, desc


def run_reference(args):
    """The oracle as it stands, on the host cores, on a row sample of the same workload."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    if CONFIGS[args.config].get("big"):
        fn, flops, sample = big_oracle_sample(CONFIGS[args.config], 3.0e10)
        for _ in range(args.warmup):
            fn()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            fn()
        dt = (time.perf_counter() - t0) / args.steps
        val = flops / dt / 1e12
        print(json.dumps({"impl": "reference", "metric": BIG_METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                          "config": {"workload": CONFIGS[args.config]["label"], "sample": sample},
                          "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
                          "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                          "gpu_launches": 0}), flush=True)
        return
    wl = make_workload(args.config)
    rows, keep, flops = oracle_sample(args.config, wl, 1.0e11)
    for _ in range(args.warmup):
        oracle_ffn(args.config, wl, rows, keep)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_ffn(args.config, wl, rows, keep)
    dt = (time.perf_counter() - t0) / args.steps
    val = flops / dt / 1e12
    sample = f"{len(rows)} of {wl.M} rows per step (evenly spaced), all outputs, fp64"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": CONFIGS[args.config]["label"], "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def time_cpu_oracle(name, wl):
    import oracle
    rows, keep, flops = oracle_sample(name, wl)
    best = None
    t_all = time.perf_counter()
    for _ in range(3):
        t0 = time.perf_counter()
        oracle_ffn(name, wl, rows, keep)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
        if time.perf_counter() - t_all > 25:
            break
    return {"value": flops / best / 1e12, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{len(rows)} of {wl.M} rows (evenly spaced), all outputs, best of <=3, {best:.2f} s per pass"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=12)
    ap.add_argument("--config", default="2", choices=sorted(CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the dense-control / explicit-types / decode side measurements")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = {"2": 600, "3q4": 300, "3q8": 200, "pilot": 300, "gpilot": 300, "g8b": 100, "4": 20, "train2": 200,
                      "train8b": 100}.get(args.config, 100 if args.config.startswith("gt") else 20) if args.impl == "ours" else 3
        if args.impl == "ours" and CONFIGS[args.config].get("big"):
            args.steps = 200 if CONFIGS[args.config]["M"] <= 8192 else 50
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else min(args.warmup, 1)
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    from paper_2609_32814_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    binding.lib()  # fail loudly if the CUDA library is missing
    ctx = {"world": world, "rank": rank, "local_rank": local_rank, "dist": dist, "torch": torch, "binding": binding}
    cfg = CONFIGS[args.config]
    line = (run_decode(args, ctx) if args.config == "4" else run_train(args, ctx) if cfg.get("train") else
            run_big(args, ctx) if cfg.get("big") else run_prefill(args, ctx))
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_prefill(args, ctx):
    torch, binding, dist = ctx["torch"], ctx["binding"], ctx["dist"]
    world, rank, local_rank = ctx["world"], ctx["rank"], ctx["local_rank"]
    from paper_2609_32814_b200 import synth
    name, cfg = args.config, CONFIGS[args.config]
    wl = make_workload(name)
    dev = lambda a: torch.from_numpy(a).cuda().to(torch.bfloat16)
    # configuration 2 fixes the schedule "type = position mod 2" and the pilot shapes the interval typing
    # of period 768: their handles are created with that schedule (the per-call types array is then not
    # needed, rows are read and written in place); the explicit-types path of the same
    # workload is timed as a side measurement.  The other configurations draw i.i.d. row types.
    gated = bool(cfg.get("gated"))
    Handle = binding.GatedFFN if gated else binding.FFN
    def make_handle(table):
        h = Handle(wl.d_widths, wl.f_widths, dtype="bf16", table=table, schedule=cfg["schedule"])
        if cfg.get("period"):       # interval typing that repeats: type = floor((position mod period) / (period / q))
            h.set_option("interval_period", cfg["period"])
        return h

    ffn = make_handle(cfg["law"])
    w_up_host = np.concatenate([wl.meta["W_gate"], wl.W_up], axis=1) if gated else wl.W_up   # merged bank [W_gate | W_up]
    counts = np.bincount(wl.types, minlength=wl.q).tolist()
    flops = 2 * ffn.macs(counts)
    stream = torch.cuda.current_stream()
    types = torch.from_numpy(wl.types).cuda()
    call_types = types if cfg["schedule"] == "explicit" else None
    M, D, F = wl.M, wl.D, wl.F

    # ---- working sets: independent copies of (X, W_up, W_down, Y, workspace) used round-robin, so
    # every step reads inputs and weights that have left the 126 MB L2 since their last use (no
    # explicit flush: a write-flush would leave L2 full of dirty lines whose write-back the next
    # step then pays for).  A set larger than twice the L2 needs no second one.
    ws_bytes = ffn.workspace_bytes(M)
    set_bytes = 2 * M * D * 2 + (3 if gated else 2) * D * F * 2 + ws_bytes
    n_sets = N_SETS if name == "2" else (1 if set_bytes > 2 * L2_BYTES else int(min(6, max(2, math.ceil(4 * L2_BYTES / set_bytes)))))
    sets = []
    for r in range(n_sets):
        if r == 0 and world == 1:
            Xr = dev(wl.X)
        elif name == "2":
            Xr = dev(synth.bf16_round(synth.normal(rank_batch_seed(rank, world, r), wl.X.shape, 1.0)))
        else:
            g = torch.Generator(device="cuda").manual_seed(synth.seed_for(9, rank * 16 + r))
            Xr = torch.randn((M, D), device="cuda", generator=g).to(torch.bfloat16)
        sets.append({"X": Xr, "Wu": dev(w_up_host).clone(), "Wd": dev(wl.W_down).clone(),
                     "Y": torch.empty((M, D), dtype=torch.bfloat16, device="cuda"),
                     "ws": torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")})
    footprint_mb = n_sets * set_bytes / 1e6

    def step(i, handle=None, tt=call_types):
        s_ = sets[i % n_sets]
        if gated:
            (handle or ffn).forward(s_["X"], tt, s_["Wu"], s_["Wd"], out=s_["Y"], workspace=s_["ws"], stream=stream)
        else:
            (handle or ffn).forward(s_["X"], tt, s_["Wu"], s_["Wd"], act="gelu", out=s_["Y"], workspace=s_["ws"], stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def time_steps(n, handle=None, tt=call_types, first=0, clocks=None):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for i in range(n):
            step(first + i, handle, tt)
            if clocks is not None and i == 0:
                clocks.arm()      # samples count from the moment the first launch is enqueued
        e1.record(stream)
        barrier()
        return e0.elapsed_time(e1)

    for i in range(args.warmup):
        step(i)
    barrier()
    assert ffn.last_status() == 0

    # ---- timed region: exactly K steps between two events, barrier + synchronize on both sides ----
    launches0 = binding.launch_count()
    with ClockSampler(local_rank) as clocks:
        total_ms = time_steps(args.steps, first=args.warmup, clocks=clocks)
    launches = binding.launch_count() - launches0
    clock_note = extend_clock_record(clocks, step, local_rank, torch)
    total_ms = max_over_ranks(total_ms, "cuda")
    ms_per_step = total_ms / args.steps
    value = whole_job_value(flops, world, args.steps, total_ms)
    assert ffn.last_status() == 0

    # ---- per-kernel durations (second pass with events between the kernels) ----
    ffn.set_timing(True)
    kt = np.zeros(4)
    n_kt = min(args.steps, 100)
    for i in range(n_kt):
        step(i)
        kt += np.array(ffn.get_timing())
    kt /= n_kt
    ffn.set_timing(False)

    # ---- roofline: the slower of (kept FLOPs at the bf16 peak) and (algorithmic bytes at the HBM rate) ----
    peaks = _peaks()
    region_s = total_ms * 1e-3
    burst = region_s < 0.1       # a region this short runs at burst clocks, like the burst measurement of the peak
    peak_tf = peaks["bf16_tflops"] if burst or not peaks["bf16_tflops_sustained"] else peaks["bf16_tflops_sustained"]
    bytes_proj = (M * D + D * F + M * F) * 2          # one projection: activations in, weights, activations out
    bytes_step = 2 * bytes_proj + (D * F * 2 if gated else 0)   # H is written by the up kernel and read by the down kernel
    t_tensor, t_hbm = flops / (peak_tf * 1e12), bytes_step / (peaks["hbm_gbs"] * 1e9)
    gemm_launches = 2 * args.steps                    # the dominant kernel runs twice per step
    avg_launch_ms = total_ms / gemm_launches
    kernel = ("proj_tc_kernel (two launches per step: merged gate/up with silu(gate) * up, down with row scatter)" if gated
              else "proj_tc_kernel (two launches per step: up with GELU, down with row scatter)")
    if cfg["law"] == "qq" and cfg["schedule"] == "explicit" and M <= 256 * cfg["q"] and len(set(wl.d_widths)) == 1 and len(set(wl.f_widths)) == 1:
        kernel = kernel.replace("proj_tc_kernel", "proj_big_kernel")      # small buckets run on the large-algebra kernel
    if t_tensor >= t_hbm:
        achieved = flops * args.steps / region_s / 1e12
        roofline = {"bound": "tensor", "kernel": kernel, "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": achieved / peak_tf,
                    "peak_source": f"{peaks['source']} ({'burst' if peak_tf == peaks['bf16_tflops'] else 'sustained'})",
                    "peak_note": f"timed region of {args.steps} steps = {region_s * 1e3:.1f} ms: "
                                 + ("shorter than 0.1 s, runs at burst clocks like the burst measurement of the peak"
                                    if burst else "long enough for the power cap, compared with the sustained peak"),
                    "algorithmic_gflop_per_launch": flops / 2 / 1e9}
    else:
        achieved = bytes_step * args.steps / region_s / 1e9
        roofline = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                    "tensor_time_us": t_tensor * 1e6, "hbm_time_us": t_hbm * 1e6}
    roofline.update({"traffic": None, "traffic_note": "no ncu capture of this kernel version is tied to this line",
                     "avg_launch_ms": avg_launch_ms, "algorithmic_mb_per_launch": bytes_proj / 1e6,
                     "isolated_kernel_ms": {"bucketing": float(kt[0]), "gather": float(kt[1]), "up": float(kt[2]),
                                            "down": float(kt[3]), "note": "events between the kernels (no launch overlap)"}})

    # ---- end to end through the host entry point: pinned H2D of X (and types), D2H of Y inside the timing ----
    # Three slots (pinned X / Y, device workspace, stream) are used round-robin, the way a serving
    # loop would: the upload of step i+1 and the download of step i-1 overlap the kernels of step i.
    # Every step still uploads its own X and downloads its own Y inside the timed region.
    n_slots = 3
    e2e_steps = args.steps if name == "2" else min(args.steps, 12)
    slots = []
    for k in range(n_slots):
        slots.append({"X": torch.from_numpy(wl.X).to(torch.bfloat16).pin_memory(),
                      "t": None if call_types is None else torch.from_numpy(wl.types).pin_memory(),
                      "Y": torch.empty((M, D), dtype=torch.bfloat16).pin_memory(),
                      "ws": None if gated else torch.empty(ffn.host_workspace_bytes(M, torch.bfloat16), dtype=torch.uint8, device="cuda"),
                      "stream": torch.cuda.Stream()})

    if gated:   # no host entry point: the same copies are made around the device entry point
        for sl in slots:
            sl["Xd"] = torch.empty((M, D), dtype=torch.bfloat16, device="cuda")
            sl["td"] = torch.empty(M, dtype=torch.int32, device="cuda")
            sl["Yd"] = torch.empty((M, D), dtype=torch.bfloat16, device="cuda")
            sl["wsd"] = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")

    def host_step(i):
        sl = slots[i % n_slots]
        if gated:
            with torch.cuda.stream(sl["stream"]):
                sl["Xd"].copy_(sl["X"], non_blocking=True)
                if sl["t"] is not None:
                    sl["td"].copy_(sl["t"], non_blocking=True)
                ffn.forward(sl["Xd"], None if sl["t"] is None else sl["td"], sets[i % n_sets]["Wu"], sets[i % n_sets]["Wd"], out=sl["Yd"], workspace=sl["wsd"],
                            stream=sl["stream"])
                sl["Y"].copy_(sl["Yd"], non_blocking=True)
            return
        ffn.forward_host(sl["X"], sl["t"], sets[i % n_sets]["Wu"], sets[i % n_sets]["Wd"], sl["Y"], workspace=sl["ws"],
                         stream=sl["stream"])

    for i in range(2 * n_slots):
        host_step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for sl in slots:
        sl["stream"].wait_event(e0)
    for i in range(e2e_steps):
        host_step(i)
    for sl in slots:
        done = torch.cuda.Event()
        done.record(sl["stream"])
        stream.wait_event(done)
    e1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), "cuda")
    h2d = int(M * D * 2 + (0 if call_types is None else M * 4))
    e2e = {"value": whole_job_value(flops, world, e2e_steps, e2e_ms), "unit": UNIT,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": int(M * D * 2), "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps,
           "note": f"{n_slots} host-buffer slots on {n_slots} streams: copies of neighbouring steps overlap the kernels"}
    del slots

    extras = {}
    if rank == 0 and not args.no_extras:
        n = min(24, args.steps)
        try:
            dense = make_handle("dense")
        except binding.AlgError:
            dense = None      # group widths only the large-algebra kernel takes: it has no dense table
            extras["vs_dense"] = None
        if dense is not None:
            time_steps(min(6, n), dense)
            dense_ms = time_steps(n, dense) / n
            star_ms = time_steps(n) / n
            extras["vs_dense"] = {"dense_ms_per_step": dense_ms, "star_ms_per_step": star_ms,
                                  "time_ratio_star_over_dense": star_ms / dense_ms,
                                  "control": "same library, ALG_TABLE_DENSE, same schedule, measured back to back with the star_q run",
                                  "ideal_ratio": flops / (2.0 * (3 if gated else 2) * M * D * F)}
            del dense
        if cfg["schedule"] != "explicit":
            explicit = Handle(wl.d_widths, wl.f_widths, dtype="bf16", table=cfg["law"])
            time_steps(6, explicit, types)
            ex_ms = time_steps(n, explicit, types) / n
            extras["explicit_types"] = {"ms_per_step": ex_ms, "frac_of_roofline": (flops / (ex_ms * 1e-3) / 1e12) / peak_tf,
                                        "note": "same workload through ALG_SCHED_EXPLICIT (bucketing + row gather kernels run)"}
            del explicit
        if name == "2":
            extras["decode"] = decode_measurements(binding)
        if cfg.get("paper_us"):
            extras["paper_h200_us"] = {"M=1": cfg["paper_us"][0], "M=2048": cfg["paper_us"][1],
                                       "note": "the paper's own kernel on its H200 NVL (another machine: context)"}
            extras["decode_m1"] = gated_decode_chain(binding, cfg["q"], D, F)
            cyc = Handle(wl.d_widths, wl.f_widths, dtype="bf16", table=cfg["law"], schedule="cyclic")
            time_steps(6, cyc, None)
            l0 = binding.launch_count()
            cyc_ms = time_steps(n, cyc, None) / n
            extras["cyclic_schedule"] = {"ms_per_step": cyc_ms, "launches_per_step": (binding.launch_count() - l0) // n,
                                         "note": "same shapes and weights with type = position mod q as the handle's schedule: equal "
                                                 "buckets, rows read and written in place (no bucketing, no gather)"}
            del cyc

    cpu = time_cpu_oracle(name, wl) if rank == 0 else None
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg["label"],
                       "l2": (f"{n_sets} working sets of inputs, weights, outputs and workspace used round-robin "
                              f"({footprint_mb:.0f} MB in total, L2 is 126 MB)" if n_sets > 1 else
                              f"one working set of {footprint_mb:.0f} MB, several times the 126 MB L2"),
                       "rows_per_gpu": M, "rows_per_type": counts, "schedule": cfg["schedule"], "law": cfg["law"],
                       "parallelism": f"rows sharded over {world} GPU(s), weights replicated"},
            "tokens_per_s": world * M * args.steps / region_s,
            "kept_gflop_per_step": flops / 1e9,
            "clocks": dict(clocks.summary(), note=clock_note), "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "cpu_baseline": cpu}
    line.update(extras)
    return line


def run_train(args, ctx):
    """--config train*: a step = forward, input gradient and weight gradient of ONE projection (the
    matrix products of a training step, three times the forward MACs)."""
    torch, binding = ctx["torch"], ctx["binding"]
    world, rank, local_rank = ctx["world"], ctx["rank"], ctx["local_rank"]
    from paper_2609_32814_b200 import synth
    import oracle
    name, cfg = args.config, CONFIGS[args.config]
    q, M, D, F = cfg["q"], cfg["M"], cfg["D"], cfg["F"]
    dw_, fw_ = [D // q] * q, [F // q] * q
    types_h = synth.cyclic_types(M, q, period=1024) if cfg["schedule"] == "cyclic" else synth.uniform_types(synth.seed_for(8, 41), M, q)
    counts = np.bincount(types_h, minlength=q).tolist()
    Xh = synth.bf16_round(synth.normal(synth.seed_for(8, 42), (M, D), 1.0))
    Wh = synth.bf16_round(synth.normal(synth.seed_for(8, 43), (D, F), 0.02))
    Gh = synth.bf16_round(synth.normal(synth.seed_for(8, 44), (M, F), 1.0))
    dev = lambda a_: torch.from_numpy(a_).cuda().to(torch.bfloat16)
    stream = torch.cuda.current_stream()
    tt = None if cfg["schedule"] == "cyclic" else torch.from_numpy(types_h).cuda()

    def handles(table):
        return (binding.Proj(dw_, fw_, dtype="bf16", table=table, schedule=cfg["schedule"]),
                binding.ProjGrad(dw_, fw_, table=table, schedule=cfg["schedule"]))
    fwd, grad = handles(cfg["law"])
    flops = 3 * 2 * fwd.macs(counts)
    set_bytes = (2 * M * D + 2 * D * F + 2 * M * F) * 2 + D * F * 4
    n_sets = 1 if set_bytes > 2 * L2_BYTES else int(min(6, max(2, math.ceil(4 * L2_BYTES / set_bytes))))
    sets = []
    for r in range(n_sets):
        sets.append({"X": dev(Xh).clone(), "W": dev(Wh).clone(), "G": dev(Gh).clone(),
                     "Y": torch.empty((M, F), dtype=torch.bfloat16, device="cuda"),
                     "dX": torch.empty((M, D), dtype=torch.bfloat16, device="cuda"),
                     "dW": torch.empty((D, F), dtype=torch.float32, device="cuda"),
                     "ws": torch.empty(max(fwd.workspace_bytes(M), grad.workspace_bytes(M)), dtype=torch.uint8, device="cuda")})

    def step(i, f=fwd, g=grad):
        s_ = sets[i % n_sets]
        f.forward(s_["X"], tt, s_["W"], out=s_["Y"], workspace=s_["ws"], stream=stream)
        g.grad_input(s_["G"], tt, s_["W"], out=s_["dX"], workspace=s_["ws"], stream=stream)
        g.grad_weight(s_["X"], s_["G"], tt, out=s_["dW"], workspace=s_["ws"], stream=stream)

    def time_steps(n, f=fwd, g=grad, clocks=None):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for i in range(n):
            step(i, f, g)
            if clocks is not None and i == 0:
                clocks.arm()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    assert fwd.last_status() == 0 and grad.last_status() == 0
    launches0 = binding.launch_count()
    with ClockSampler(local_rank) as clocks:
        total_ms = time_steps(args.steps, clocks=clocks)
    launches = binding.launch_count() - launches0
    total_ms = max_over_ranks(total_ms, "cuda")
    # the three parts on their own
    parts = {}
    for key, fn in (("forward", lambda s_: fwd.forward(s_["X"], tt, s_["W"], out=s_["Y"], workspace=s_["ws"], stream=stream)),
                    ("grad_input", lambda s_: grad.grad_input(s_["G"], tt, s_["W"], out=s_["dX"], workspace=s_["ws"], stream=stream)),
                    ("grad_weight", lambda s_: grad.grad_weight(s_["X"], s_["G"], tt, out=s_["dW"], workspace=s_["ws"], stream=stream))):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for i in range(min(args.steps, 50)):
            fn(sets[i % n_sets])
        e1.record(stream)
        torch.cuda.synchronize()
        parts[key + "_ms"] = e0.elapsed_time(e1) / min(args.steps, 50)
    peaks = _peaks()
    region_s = total_ms * 1e-3
    peak_tf = peaks["bf16_tflops"] if region_s < 0.1 or not peaks["bf16_tflops_sustained"] else peaks["bf16_tflops_sustained"]
    bytes_step = (3 * M * D + 2 * D * F + 3 * M * F) * 2 + D * F * 4    # X, W, Y | G, W, dX | X, G, dW (fp32)
    t_tensor, t_hbm = flops / (peak_tf * 1e12), bytes_step / (peaks["hbm_gbs"] * 1e9)
    value = whole_job_value(flops, world, args.steps, total_ms)
    if t_tensor >= t_hbm:
        roofline = {"bound": "tensor", "achieved": value / world, "peak": peak_tf, "unit": "TFLOP/s", "frac": value / world / peak_tf,
                    "peak_source": f"{peaks['source']} ({'burst' if peak_tf == peaks['bf16_tflops'] else 'sustained'})"}
    else:
        gbs = bytes_step * args.steps / region_s / 1e9
        roofline = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                    "peak_source": peaks["source"], "tensor_time_us": t_tensor * 1e6, "hbm_time_us": t_hbm * 1e6}
    roofline.update({"kernel": "proj_tc_kernel (forward, dX with W used transposed, dW over the row buckets: in place with the cyclic schedule, padded copies otherwise)", "traffic": None,
                     "parts": parts})
    extras = {}
    if rank == 0 and not args.no_extras:
        fd, gd = handles("dense")
        time_steps(3, fd, gd)
        n = min(24, args.steps)
        dense_ms = time_steps(n, fd, gd) / n
        star_ms = time_steps(n) / n
        extras["vs_dense"] = {"dense_ms_per_step": dense_ms, "star_ms_per_step": star_ms, "time_ratio_star_over_dense": star_ms / dense_ms,
                              "control": "same library, ALG_TABLE_DENSE", "ideal_ratio": flops / (3.0 * 2 * M * D * F)}
    # CPU baseline: the oracle's forward and both gradient maps on evenly spaced rows
    cpu = None
    if rank == 0:
        keep = oracle.support(q, cfg["law"])
        n = int(min(M, max(16, 2 ** int(math.log2(max(16.0, 6e10 / (3.0 * D * F)))))))
        rows = np.arange(0, M, max(1, M // n))[:n]
        t0 = time.perf_counter()
        oracle.proj(Xh[rows], types_h[rows], Wh, dw_, fw_, keep=keep)
        oracle.proj_vjp_x(Gh[rows], types_h[rows], Wh, dw_, fw_, keep=keep)
        oracle.proj_vjp_w(Xh[rows], Gh[rows], types_h[rows], dw_, fw_, keep=keep)
        dt = time.perf_counter() - t0
        c = np.bincount(types_h[rows], minlength=q)
        cpu = {"value": 3 * 2 * oracle.macs(keep, dw_, fw_, c) / dt / 1e12, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
               "sample": f"{len(rows)} of {M} rows (evenly spaced), forward + dX + dW, {dt:.2f} s"}
    return {"metric": "star_q projection training step (forward + dX + dW), kept-GEMM throughput", "value": value, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg["label"], "rows_per_type": counts,
                       "l2": f"{n_sets} working set(s) of {set_bytes / 1e6:.0f} MB used round-robin, L2 is 126 MB"},
            "clocks": dict(clocks.summary(), note="sampled during the timed region"),
            "e2e": {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                    "note": "gradients stay on the device in a training step; no host entry point is timed"},
            "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu, **extras}


def run_big(args, ctx):
    """--config sq* / qw*: a step = ONE projection of the large-algebra path (no pre-kernel: the schedules are
    cyclic or interval with q | M)."""
    torch, binding = ctx["torch"], ctx["binding"]
    world, rank, local_rank = ctx["world"], ctx["rank"], ctx["local_rank"]
    cfg = CONFIGS[args.config]
    q, s, r, M = cfg["q"], cfg["s"], cfg["r"], cfg["M"]
    K, N = q * s, q * r
    stream = torch.cuda.current_stream()
    proj = binding.Proj([s] * q, [r] * q, dtype="bf16", schedule=cfg["schedule"])
    assert proj.kernel_path(M) == binding.ALG_PATH_TCGEN05
    counts = [M // q] * q
    flops = 2 * proj.macs(counts)
    set_bytes = (M * K + K * N + M * N) * 2
    n_sets = 1 if set_bytes > 2 * L2_BYTES else int(min(6, max(2, math.ceil(4 * L2_BYTES / set_bytes))))
    gen = torch.Generator(device="cuda")
    sets = []
    for i in range(n_sets):
        gen.manual_seed(20260932 + 900 + 16 * rank + i)
        sets.append({"X": torch.randn((M, K), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16),
                     "W": (torch.randn((K, N), generator=gen, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16),
                     "Y": torch.empty((M, N), dtype=torch.bfloat16, device="cuda")})
    ws = torch.empty(max(256, proj.workspace_bytes(M)), dtype=torch.uint8, device="cuda")
    # group widths that are multiples of 4 only: the bank is padded to multiples of 8 ONCE, outside the timed region
    # (weights are laid out when they are loaded); X is still padded inside every step
    packed = proj.packed_weight_bytes() > 0
    if packed:
        for s_ in sets:
            s_["Wp"] = proj.pack_weight(s_["W"])
        proj.set_option("weight_packed", 1)
    use_packed = [packed]

    def step(i, h=proj):
        s_ = sets[i % n_sets]
        h.forward(s_["X"], None, s_["Wp"] if use_packed[0] and h is proj else s_["W"], out=s_["Y"], workspace=ws, stream=stream)

    def time_steps(n, h=proj, clocks=None):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for i in range(n):
            step(i, h)
            if clocks is not None and i == 0:
                clocks.arm()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    assert proj.last_status() == 0
    launches0 = binding.launch_count()
    with ClockSampler(local_rank) as clocks:
        total_ms = time_steps(args.steps, clocks=clocks)
    launches = binding.launch_count() - launches0
    clock_note = extend_clock_record(clocks, step, local_rank, torch)
    total_ms = max_over_ranks(total_ms, "cuda")
    peaks = _peaks()
    region_s = total_ms * 1e-3
    peak_tf = peaks["bf16_tflops"] if region_s < 0.1 or not peaks["bf16_tflops_sustained"] else peaks["bf16_tflops_sustained"]
    t_tensor, t_hbm = flops / (peak_tf * 1e12), set_bytes / (peaks["hbm_gbs"] * 1e9)
    value = whole_job_value(flops, world, args.steps, total_ms)
    if t_tensor >= t_hbm:
        roofline = {"bound": "tensor", "achieved": value / world, "peak": peak_tf, "unit": "TFLOP/s", "frac": value / world / peak_tf,
                    "peak_source": f"{peaks['source']} ({'burst' if peak_tf == peaks['bf16_tflops'] else 'sustained'})"}
    else:
        gbs = set_bytes * args.steps / region_s / 1e9
        roofline = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                    "peak_source": peaks["source"]}
    roofline.update({"kernel": "proj_big_kernel", "traffic": None, "tensor_time_us": t_tensor * 1e6, "hbm_time_us": t_hbm * 1e6,
                     "algorithmic_bytes": set_bytes, "algorithmic_flops": flops})
    ms_step = total_ms / args.steps
    extras = {"paper": {"ms_per_step": cfg["paper_ms"], "hardware": "H200 NVL, the paper's own kernel, warm median",
                        "time_ratio_paper_over_ours": cfg["paper_ms"] / ms_step}}
    e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": M * K * 2, "d2h_bytes_per_step": M * N * 2}
    if rank == 0 and not args.no_extras:
        if packed:
            proj.set_option("weight_packed", 0)
            use_packed[0] = False
            time_steps(2)
            n_un = min(args.steps, 20)
            extras["per_call_weight_padding"] = {"ms_per_step": time_steps(n_un) / n_un,
                                                 "note": "the same step with the caller's unpadded bank: X and W are both padded inside every call"}
            proj.set_option("weight_packed", 1)
            use_packed[0] = True
        if K % 64 == 0 and N % 128 == 0:
            dense = binding.Proj([K], [N], dtype="bf16", schedule="cyclic")    # q = 1: the ordinary product X W
            wsd = torch.empty(max(256, dense.workspace_bytes(M)), dtype=torch.uint8, device="cuda")
            def dstep(i):
                s_ = sets[i % n_sets]
                dense.forward(s_["X"], None, s_["W"], out=s_["Y"], workspace=wsd, stream=stream)
            def dtime(n):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record(stream)
                for i in range(n):
                    dstep(i)
                e1.record(stream)
                torch.cuda.synchronize()
                return e0.elapsed_time(e1) / n
            dtime(2)
            est = dtime(1)
            dense_ms = dtime(int(max(2, min(20, 300.0 / max(est, 1e-3)))))
            extras["vs_dense"] = {"dense_ms_per_step": dense_ms, "star_ms_per_step": ms_step, "time_ratio_star_over_dense": ms_step / dense_ms,
                                  "control": "same library, q = 1 (ordinary X W on the table-driven tcgen05 kernel)",
                                  "ideal_ratio": flops / (2.0 * M * K * N)}
        if cfg.get("paper_m1_us"):
            extras["decode_m1"] = dict(proj_decode_calls(binding, 32, K, N), paper_h200_us=cfg["paper_m1_us"])
        # end to end through the C ABI's host entry point: pinned X in, Y out, copies inside the timing
        Xh = sets[0]["X"].cpu().pin_memory()
        Yh = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
        wsh = torch.empty(proj.host_workspace_bytes(M, torch.bfloat16), dtype=torch.uint8, device="cuda")
        n_e2e = int(max(2, min(20, 2000.0 / max(1.0, (M * K + M * N) * 2 / 25e6))))
        for _ in range(2):
            proj.forward_host(Xh, None, sets[0]["Wp"] if packed else sets[0]["W"], Yh, workspace=wsh, stream=stream)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(n_e2e):
            proj.forward_host(Xh, None, sets[0]["Wp"] if packed else sets[0]["W"], Yh, workspace=wsh, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        e2e["value"] = flops * n_e2e / (e0.elapsed_time(e1) * 1e-3) / 1e12
        e2e["steps"] = n_e2e
    cpu = None
    if rank == 0:
        fn, cflops, sample = big_oracle_sample(cfg)
        t0 = time.perf_counter()
        fn()
        dt = time.perf_counter() - t0
        cpu = {"value": cflops / dt / 1e12, "unit": UNIT, "cores": __import__("oracle").threads(), "kind": "oracle",
               "sample": f"{sample}, {dt:.2f} s"}
    return {"metric": BIG_METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic (generated on the device, seeded)",
            "config": {"workload": cfg["label"] + (", bank padded to groups of multiples of 8 once (alg_proj_pack_weight)" if packed else ""),
                       "rows_per_type": M // q, "tile": "128 rows x ceil16(r / ceil(r / 256)) columns",
                       "l2": f"{n_sets} working set(s) of {set_bytes / 1e6:.0f} MB used round-robin, L2 is 126 MB"},
            "clocks": dict(clocks.summary(), note=clock_note), "e2e": e2e,
            "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu, **extras}


def decode_measurements(binding, layers=64, replays=20):
    """KV-cached decode shapes (configuration 4): M new tokens, type = absolute position mod 2.
    streaming: a CUDA graph of `layers` consecutive FFN layers with distinct weight banks
    (604 MB, far beyond L2), layer l+1 consuming layer l's output -- GB/s counts the weight
    blocks some row needs plus X and Y of every projection.  isolated: one FFN per replay."""
    import torch
    from paper_2609_32814_b200 import synth
    peaks = _peaks()
    cfg = CONFIGS["4"]
    D, F, q = cfg["D"], cfg["F"], cfg["q"]
    g = torch.Generator(device="cuda").manual_seed(1234)
    Wu = [(torch.randn((D, F), device="cuda", generator=g) * 0.02).to(torch.bfloat16) for _ in range(layers)]
    Wd = [(torch.randn((F, D), device="cuda", generator=g) * 0.02).to(torch.bfloat16) for _ in range(layers)]
    ffn = binding.FFN([D // q] * q, [F // q] * q, dtype="bf16")
    ws = torch.empty(ffn.workspace_bytes(64), dtype=torch.uint8, device="cuda")
    res = []
    stream = torch.cuda.Stream()
    launches0 = binding.launch_count()
    for M in (1, 8, 32, 64):
        w4 = synth.config4(M)
        types = torch.from_numpy(w4.types).cuda()
        present = len(set(w4.types.tolist()))
        # weight bytes some row needs: diagonal blocks always, off-diagonal block (k,j) iff type k present
        frac = 1.0 if present == 2 else 0.75
        bytes_layer = frac * 2 * D * F * 2 + 2 * M * (D + F) * 2
        acts = [torch.from_numpy(w4.X).cuda().to(torch.bfloat16)] + \
               [torch.empty((M, D), dtype=torch.bfloat16, device="cuda") for _ in range(layers)]

        def chain(n):
            for l in range(n):
                ffn.forward(acts[l], types, Wu[l], Wd[l], act="gelu", out=acts[l + 1], workspace=ws, stream=stream)

        def graph_time(n, reps):
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.stream(stream):
                chain(n)                      # warm-up outside capture
                torch.cuda.synchronize()
                with torch.cuda.graph(gr, stream=stream):
                    chain(n)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ts = []
            for _ in range(reps):
                e0.record()
                gr.replay()
                e1.record()
                e1.synchronize()
                ts.append(e0.elapsed_time(e1))
            return float(np.median(ts))

        l0 = binding.launch_count()
        chain(1)
        per_layer_launches = binding.launch_count() - l0
        t_stream = graph_time(layers, replays)
        t_iso = graph_time(1, replays)
        gbs = layers * bytes_layer / (t_stream * 1e-3) / 1e9
        res.append({"M": M, "types_present": present, "needed_mb_per_layer": bytes_layer / 1e6,
                    "launches_per_layer": per_layer_launches,
                    "stream_us_per_layer": t_stream * 1e3 / layers, "stream_gbs": gbs,
                    "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                 "frac": gbs / peaks["hbm_gbs"]},
                    "isolated_warm_us": t_iso * 1e3})
    assert ffn.last_status() == 0
    return {"protocol": f"{layers}-layer dependent FFN chain with distinct weights in one CUDA graph, median of {replays} replays",
            "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"], "results": res,
            "launches": binding.launch_count() - launches0}


def proj_decode_calls(binding, q, K, N, calls=32, replays=20):
    """One row (M = 1) through `calls` projections K -> N with distinct weight banks in one CUDA graph (independent
    calls on one stream).  GB/s counts the 2/q of the bank the row's type needs plus x and y."""
    import torch
    peaks = _peaks()
    g = torch.Generator(device="cuda").manual_seed(987)
    Ws = [(torch.randn((K, N), device="cuda", generator=g) * 0.02).to(torch.bfloat16) for _ in range(calls)]
    X = torch.randn((1, K), device="cuda", generator=g).to(torch.bfloat16)
    Ys = [torch.empty((1, N), dtype=torch.bfloat16, device="cuda") for _ in range(calls)]
    types = torch.full((1,), 5 % q, dtype=torch.int32, device="cuda")
    proj = binding.Proj([K // q] * q, [N // q] * q, dtype="bf16")
    ws = torch.empty(max(256, proj.workspace_bytes(1)), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()

    def chain():
        for l in range(calls):
            proj.forward(X, types, Ws[l], out=Ys[l], workspace=ws, stream=stream)

    l0 = binding.launch_count()
    gr = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        chain()
        torch.cuda.synchronize()
        per_call = (binding.launch_count() - l0) // calls
        with torch.cuda.graph(gr, stream=stream):
            chain()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ts = []
    for _ in range(replays):
        e0.record()
        gr.replay()
        e1.record()
        e1.synchronize()
        ts.append(e0.elapsed_time(e1))
    assert proj.last_status() == 0
    us = float(np.median(ts)) * 1e3 / calls
    bytes_call = 2 * (K // q) * N * 2 + (K + N) * 2
    gbs = bytes_call / (us * 1e-6) / 1e9
    return {"protocol": f"{calls} projections {K}->{N} at q = {q}, M = 1, distinct weights, one CUDA graph, median of {replays} replays",
            "us_per_call": us, "launches_per_call": per_call, "needed_mb_per_call": bytes_call / 1e6,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"]}}


def gated_decode_chain(binding, q, D, F, layers=32, replays=20):
    """One row (M = 1) through `layers` consecutive gated FFN layers with distinct weight banks in one CUDA graph, layer
    l+1 consuming layer l's output.  GB/s counts the weight blocks the row needs (2/q of both banks) plus x, h, y."""
    import torch
    peaks = _peaks()
    g = torch.Generator(device="cuda").manual_seed(4321)
    Wgu = [(torch.randn((D, 2 * F), device="cuda", generator=g) * 0.02).to(torch.bfloat16) for _ in range(layers)]
    Wd = [(torch.randn((F, D), device="cuda", generator=g) * 0.02).to(torch.bfloat16) for _ in range(layers)]
    ffn = binding.GatedFFN([D // q] * q, [F // q] * q, dtype="bf16")
    ws = torch.empty(ffn.workspace_bytes(1), dtype=torch.uint8, device="cuda")
    types = torch.full((1,), 5 % q, dtype=torch.int32, device="cuda")
    acts = [torch.randn((1, D), device="cuda", generator=g).to(torch.bfloat16)] + \
           [torch.empty((1, D), dtype=torch.bfloat16, device="cuda") for _ in range(layers)]
    stream = torch.cuda.Stream()

    def chain():
        for l in range(layers):
            ffn.forward(acts[l], types, Wgu[l], Wd[l], out=acts[l + 1], workspace=ws, stream=stream)

    l0 = binding.launch_count()
    gr = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        chain()
        torch.cuda.synchronize()
        per_layer = (binding.launch_count() - l0) // layers
        with torch.cuda.graph(gr, stream=stream):
            chain()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ts = []
    for _ in range(replays):
        e0.record()
        gr.replay()
        e1.record()
        e1.synchronize()
        ts.append(e0.elapsed_time(e1))
    assert ffn.last_status() == 0
    us = float(np.median(ts)) * 1e3 / layers
    bytes_layer = 2 * (D // q) * 3 * F * 2 + 2 * (D + F) * 2
    gbs = bytes_layer / (us * 1e-6) / 1e9
    return {"protocol": f"{layers}-layer dependent chain of gated FFNs with distinct weights in one CUDA graph, M = 1, median of "
                        f"{replays} replays; {layers * bytes_layer / 1e6:.0f} MB of weights needed per replay (L2 is 126 MB)",
            "us_per_layer": us, "launches_per_layer": per_layer, "needed_mb_per_layer": bytes_layer / 1e6,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"]}}


def run_decode(args, ctx):
    """--config 4: the decode chain is the step; value = needed bytes per second at M = 8."""
    torch, binding = ctx["torch"], ctx["binding"]
    world, rank, local_rank = ctx["world"], ctx["rank"], ctx["local_rank"]
    with ClockSampler(local_rank) as clocks:
        clocks.arm()
        dec = decode_measurements(binding, replays=max(3, args.steps))
    head = [r for r in dec["results"] if r["M"] == 8][0]
    wl = make_workload("4")
    cpu = time_cpu_oracle("4", wl) if rank == 0 else None
    return {"metric": "star_q FFN decode: needed weight and activation bytes per second (64-layer dependent chain)",
            "value": world * head["stream_gbs"], "unit": "GB/s", "n_gpus": world, "steps": max(3, args.steps), "warmup": args.warmup,
            "ms_per_step": head["stream_us_per_layer"] * 64 / 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": CONFIGS["4"]["label"], "step": "one replay of the 64-layer chain at M = 8; the other M are in `decode`",
                       "l2": "64 distinct weight banks, 604 MB in total, L2 is 126 MB"},
            "clocks": dict(clocks.summary(), note="sampled over the whole decode measurement"),
            "e2e": {"value": None, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                    "note": "a decode step keeps its activations on the device; no host entry point is timed"},
            "gpu_launches": int(dec["launches"]), "roofline": dict(head["roofline"], kernel="ffn_decode_kernel", traffic=None),
            "cpu_baseline": cpu, "decode": dec}


if __name__ == "__main__":
    main()

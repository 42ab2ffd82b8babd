"""Timing sweep over the benchmark configurations 3 and 5 (and their dense same-shape controls).

    python -m paper_2609_32814_b200.sweep [--configs 3,5,pilot] [--reps 10]

Prints one JSON line per measured object: the square d->d projection, the up and down projections
and the whole FFN, each next to the same call with ALG_TABLE_DENSE.  FLOPs count only the block
GEMMs the rule keeps; the roofline time is the slower of (kept FLOPs / measured bf16 peak) and
(algorithmic bytes / measured HBM rate), bytes = every operand read or written once.
Inputs are synthetic (random bf16, types i.i.d. uniform); working sets rotate so nothing is served
from L2 across repetitions when a single set is smaller than L2.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
L2_BYTES = 126e6


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["bf16_tflops"]), float(p["hbm_gbs"]), "measured"
    return 1590.0, 6650.0, "fallback"


def _time(fn, n_sets, reps):
    for i in range(max(3, n_sets)):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(reps):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def measure(name, q, M, D, F, seed, reps, want=("up", "down", "ffn"), law="qq", types=None):
    peak_tf, hbm_gbs, src = _peaks()
    g = torch.Generator(device="cuda").manual_seed(seed)
    if types is None:
        types = torch.randint(0, q, (M,), device="cuda", generator=g, dtype=torch.int32)
    counts = torch.bincount(types.long(), minlength=q).tolist()
    dw, fw = [D // q] * q, [F // q] * q
    set_bytes = 2 * (2 * M * D + 2 * D * F + M * F)
    n_sets = 1 if set_bytes > 2 * L2_BYTES else int(np.ceil(4 * L2_BYTES / set_bytes))
    X = [torch.randn((M, D), device="cuda", generator=g).to(torch.bfloat16) for _ in range(n_sets)]
    Hh = [torch.randn((M, F), device="cuda", generator=g).to(torch.bfloat16) for _ in range(n_sets)]
    Wu = [(torch.randn((D, F), device="cuda", generator=g) * 0.02).to(torch.bfloat16) for _ in range(n_sets)]
    Wd = [(torch.randn((F, D), device="cuda", generator=g) * 0.02).to(torch.bfloat16) for _ in range(n_sets)]
    Wsq = [(torch.randn((D, D), device="cuda", generator=g) * 0.02).to(torch.bfloat16) for _ in range(n_sets)]
    Yd = [torch.empty((M, D), device="cuda", dtype=torch.bfloat16) for _ in range(n_sets)]
    Yf = [torch.empty((M, F), device="cuda", dtype=torch.bfloat16) for _ in range(n_sets)]
    out = []
    for table in (law, "dense"):
        objs = {}
        if "square" in want:
            p = binding.Proj(dw, dw, dtype="bf16", table=table)
            ws = torch.empty(p.workspace_bytes(M), dtype=torch.uint8, device="cuda")
            objs["square"] = (lambda i, p=p, ws=ws: p.forward(X[i % n_sets], types, Wsq[i % n_sets], out=Yd[i % n_sets], workspace=ws),
                              2 * p.macs(counts), 2 * (2 * M * D + D * D), p)
        if "up" in want:
            p = binding.Proj(dw, fw, dtype="bf16", table=table)
            ws = torch.empty(p.workspace_bytes(M), dtype=torch.uint8, device="cuda")
            objs["up"] = (lambda i, p=p, ws=ws: p.forward(X[i % n_sets], types, Wu[i % n_sets], act="gelu", out=Yf[i % n_sets], workspace=ws),
                          2 * p.macs(counts), 2 * (M * D + D * F + M * F), p)
        if "down" in want:
            p = binding.Proj(fw, dw, dtype="bf16", table=table)
            ws = torch.empty(p.workspace_bytes(M), dtype=torch.uint8, device="cuda")
            objs["down"] = (lambda i, p=p, ws=ws: p.forward(Hh[i % n_sets], types, Wd[i % n_sets], out=Yd[i % n_sets], workspace=ws),
                            2 * p.macs(counts), 2 * (M * F + D * F + M * D), p)
        if "ffn" in want:
            f = binding.FFN(dw, fw, dtype="bf16", table=table)
            ws = torch.empty(f.workspace_bytes(M), dtype=torch.uint8, device="cuda")
            objs["ffn"] = (lambda i, f=f, ws=ws: f.forward(X[i % n_sets], types, Wu[i % n_sets], Wd[i % n_sets], act="gelu", out=Yd[i % n_sets], workspace=ws),
                           2 * f.macs(counts), 2 * (2 * M * D + 2 * D * F + 2 * M * F), f)
        for obj, (fn, flops, nbytes, handle) in objs.items():
            ms = _time(fn, n_sets, reps)
            assert handle.last_status() == 0
            t_roof = max(flops / (peak_tf * 1e12), nbytes / (hbm_gbs * 1e9))
            out.append({"config": name, "object": obj, "table": table, "q": q, "M": M, "D": D, "F": F, "ms": ms,
                        "kept_gflop": flops / 1e9, "tflops": flops / (ms * 1e-3) / 1e12, "algorithmic_mb": nbytes / 1e6,
                        "roofline_us": t_roof * 1e6, "bound": "tensor" if flops / (peak_tf * 1e12) >= nbytes / (hbm_gbs * 1e9) else "hbm",
                        "frac_of_roofline": t_roof / (ms * 1e-3), "peaks": src, "working_sets": n_sets})
    by = {(r["object"], r["table"]): r for r in out}
    for r in out:
        if r["table"] != "dense":
            r["time_vs_dense"] = r["ms"] / by[(r["object"], "dense")]["ms"]
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="3,5")
    ap.add_argument("--reps", type=int, default=10)
    args = ap.parse_args()
    cfgs = [int(c) for c in args.configs.split(",") if c.isdigit()]
    if 3 in cfgs:
        for q in (4, 8):
            for r in measure(f"cfg3-q{q}", q, 16384, q * 128, 4 * q * 128, 300 + q, args.reps, want=("square", "up", "down", "ffn")):
                print(json.dumps(r), flush=True)
    if "pilot" in args.configs:
        # the paper's pilot FFN projections: tensor-square law, D = 768 = 4 x 192, F = 1536 = 4 x 384,
        # interval schedule floor((p mod 768) / 192), 8 sequences of 1536 tokens
        from . import synth
        M = 8 * 1536
        t = torch.from_numpy(synth.interval_types(M, 4, 768)).cuda()
        for r in measure("pilot-q2pow", 4, M, 768, 1536, 600, args.reps, law="q2pow", types=t):
            print(json.dumps(r), flush=True)
    if 5 in cfgs:
        for q in (2, 4, 8, 16):
            for r in measure(f"cfg5-q{q}", q, 32768, 4096, 16384, 500 + q, max(3, args.reps // 2)):
                print(json.dumps(r), flush=True)
            torch.cuda.empty_cache()


if __name__ == "__main__":
    main()

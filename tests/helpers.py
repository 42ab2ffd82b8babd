"""Shared helpers of the GPU parity tests: upload a synthetic workload, run the oracle, compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2609_32814_b200 import synth

# spec tolerances for bf16 operands with fp32 accumulation against the fp64 oracle
BF16_REL_FRO = 5e-3
BF16_MAX_ABS = 2e-2
# fp32 path (true fp32 FMAs): derived from K <= 256 sequential fp32 additions of N(0,1) products
F32_REL_FRO = 1e-5
F32_MAX_ABS = 1e-3


def to_dev(x: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def dev_types(types: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(types, dtype=np.int32)).cuda()


def to_np(y: torch.Tensor) -> np.ndarray:
    return y.float().cpu().numpy().astype(np.float64)


def rel_fro(got: np.ndarray, ref: np.ndarray) -> float:
    den = float(np.linalg.norm(ref))
    return float(np.linalg.norm(got - ref)) / (den if den > 0 else 1.0)


def max_abs(got: np.ndarray, ref: np.ndarray) -> float:
    return float(np.max(np.abs(got - ref))) if got.size else 0.0


def assert_bf16_close(got: np.ndarray, ref: np.ndarray, out_is_bf16: bool, what: str = ""):
    """rel-Frobenius <= 5e-3 always; max-abs <= 2e-2 on fp32 outputs; with bf16 outputs the
    final rounding adds up to half an ulp (2^-9 relative), so the bound is 2e-2 + 2^-8 |ref|."""
    rf = rel_fro(got, ref)
    assert rf <= BF16_REL_FRO, f"{what}: rel-Frobenius {rf:.3e}"
    err = np.abs(got - ref)
    bound = BF16_MAX_ABS + (2.0 ** -8) * np.abs(ref) if out_is_bf16 else BF16_MAX_ABS
    worst = float(np.max(err - bound)) if err.size else -1.0
    assert worst <= 0, f"{what}: max-abs {float(err.max()):.3e} exceeds the bound by {worst:.3e}"


def bf16_rne(x64: np.ndarray) -> np.ndarray:
    """Round exact fp64 values to bf16 (via fp32; exact for the integer tests)."""
    return synth.bf16_round(x64.astype(np.float32)).astype(np.float64)


def oracle_proj_rows(wl: synth.Workload, rows=None, keep=None, bias=None, which="up"):
    X, types = wl.X, wl.types
    if rows is not None:
        X, types = X[rows], types[rows]
    if which == "up":
        return oracle.proj(X, types, wl.W_up, wl.d_widths, wl.f_widths, keep=keep, bias=bias)
    return oracle.proj(X, types, wl.W_down, wl.f_widths, wl.d_widths, keep=keep, bias=bias)

"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds no arithmetic of the method: it only draws numbers, rounds them to bf16 and
describes the five benchmark workloads (shapes, group widths, row-type schedules).  Both the
CUDA binding and the CPU oracle are fed from here, so they see identical bit patterns.

Generator: numpy's counter-based Philox stream, seed = 20260932 + 100*config + variant.
Values are drawn in fp32; bf16 workloads round them once (round-to-nearest-even) and both
sides consume the rounded values, so input quantisation is not part of any error budget.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 20260932


def seed_for(config: int, variant: int = 0) -> int:
    return BASE_SEED + 100 * config + variant


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(seed))


def normal(seed: int, shape, std: float = 1.0) -> np.ndarray:
    return (_rng(seed).standard_normal(shape, dtype=np.float32) * np.float32(std)).astype(np.float32)


def small_ints(seed: int, shape, lo: int = -3, hi: int = 3) -> np.ndarray:
    return _rng(seed).integers(lo, hi + 1, size=shape).astype(np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round-to-nearest-even; inputs must be finite."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> the exact fp32 values they denote."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_round(x: np.ndarray) -> np.ndarray:
    return from_bf16_bits(to_bf16_bits(x))


def equal_widths(total: int, q: int) -> list[int]:
    if total % q:
        raise ValueError("total not divisible by q")
    return [total // q] * q


def cyclic_types(M: int, q: int, period: int | None = None, start: int = 0) -> np.ndarray:
    """type = (position mod q); positions restart every `period` rows (sequence length)."""
    pos = np.arange(M, dtype=np.int64)
    if period:
        pos = pos % period
    return ((pos + start) % q).astype(np.int32)


def uniform_types(seed: int, M: int, q: int) -> np.ndarray:
    return _rng(seed).integers(0, q, size=M).astype(np.int32)


def decode_types(seed: int, M: int, q: int, max_pos: int = 2048) -> np.ndarray:
    """Each new token sits at an absolute position drawn uniformly from [0, max_pos)."""
    pos = _rng(seed).integers(0, max_pos, size=M)
    return (pos % q).astype(np.int32)


@dataclass
class Workload:
    """One projection or FFN problem. Arrays are fp32 holding values exactly representable in
    `dtype` ("f32" or "bf16")."""
    name: str
    dtype: str
    q: int
    M: int
    d_widths: list[int]
    f_widths: list[int]
    types: np.ndarray
    X: np.ndarray
    W_up: np.ndarray
    W_down: np.ndarray | None = None
    meta: dict = field(default_factory=dict)

    @property
    def D(self) -> int:
        return int(sum(self.d_widths))

    @property
    def F(self) -> int:
        return int(sum(self.f_widths))


def _maybe_bf16(x: np.ndarray, dtype: str) -> np.ndarray:
    return bf16_round(x) if dtype == "bf16" else x


def make_workload(name: str, *, config: int, variant: int, dtype: str, q: int, M: int, D: int, F: int,
                  types: np.ndarray, x_std: float = 1.0, w_std: float = 0.02, integer: bool = False,
                  with_down: bool = True, d_widths=None, f_widths=None) -> Workload:
    s0 = seed_for(config, variant)
    if integer:
        X = small_ints(s0 + 1, (M, D))
        Wu = small_ints(s0 + 2, (D, F))
        Wd = small_ints(s0 + 3, (F, D)) if with_down else None
    else:
        X = _maybe_bf16(normal(s0 + 1, (M, D), x_std), dtype)
        Wu = _maybe_bf16(normal(s0 + 2, (D, F), w_std), dtype)
        Wd = _maybe_bf16(normal(s0 + 3, (F, D), w_std), dtype) if with_down else None
    return Workload(name=name, dtype=dtype, q=q, M=M,
                    d_widths=list(d_widths) if d_widths else equal_widths(D, q),
                    f_widths=list(f_widths) if f_widths else equal_widths(F, q),
                    types=np.ascontiguousarray(types, dtype=np.int32), X=X, W_up=Wu, W_down=Wd,
                    meta={"config": config, "variant": variant, "integer": integer})


# ---- the five benchmark workloads -------------------------------------------------------------

def config1(integer: bool = False) -> Workload:
    """q=2 single projection, fp32: X 512x256, W 256x1024, type = row mod 2."""
    return make_workload("cfg1-int" if integer else "cfg1", config=1, variant=int(integer), dtype="f32",
                         q=2, M=512, D=256, F=1024, types=cyclic_types(512, 2), x_std=1.0, w_std=1.0,
                         integer=integer, with_down=False)


def config2(M: int = 8192, seq: int = 1024, integer: bool = False) -> Workload:
    """q=2 FFN of a ~110M decoder LM, bf16: 768 -> 3072 -> 768, type = position mod 2."""
    return make_workload("cfg2", config=2, variant=int(integer), dtype="bf16", q=2, M=M, D=768, F=3072,
                         types=cyclic_types(M, 2, period=seq), integer=integer)


def config3(q: int, M: int = 16384, integer: bool = False) -> Workload:
    """general q, groups of 128 on the model side, 512 on the hidden side, uniform row types."""
    d = q * 128
    return make_workload(f"cfg3-q{q}", config=3, variant=q * 2 + int(integer), dtype="bf16", q=q, M=M,
                         D=d, F=4 * d, types=uniform_types(seed_for(3, q) + 7, M, q), integer=integer)


def config4(M: int, integer: bool = False) -> Workload:
    """KV-cached decode step: M new tokens typed by absolute position mod 2."""
    return make_workload(f"cfg4-M{M}", config=4, variant=M * 2 + int(integer), dtype="bf16", q=2, M=M,
                         D=768, F=3072, types=decode_types(seed_for(4, M) + 7, M, 2), integer=integer)


def config5(q: int, M: int = 32768, D: int = 4096, F: int = 16384, integer: bool = False) -> Workload:
    """scale sweep: 4096 -> 16384, uniform row types."""
    return make_workload(f"cfg5-q{q}", config=5, variant=q * 2 + int(integer), dtype="bf16", q=q, M=M,
                         D=D, F=F, types=uniform_types(seed_for(5, q) + 7, M, q), integer=integer)


def interval_types(M: int, q: int, period: int, start: int = 0) -> np.ndarray:
    """The pilot's schedule: type = floor((position mod period) / (period / q)) -- consecutive
    intervals of period/q positions share a type."""
    pos = (np.arange(M, dtype=np.int64) + start) % period
    return (pos // (period // q)).astype(np.int32)


def pilot_ffn(M: int = 4 * 1536, integer: bool = False) -> Workload:
    """Shape of the paper's ~110M pilot FFN projections: D = 768 split 4 x 192, F = 1536 split
    4 x 384 (tensor-square law, q = 4), interval schedule with period 768."""
    return make_workload("pilot", config=6, variant=int(integer), dtype="bf16", q=4, M=M, D=768, F=1536,
                         types=interval_types(M, 4, 768), integer=integer)


def gated_ffn(name: str, q: int, M: int, D: int, F: int, types: np.ndarray, variant: int = 0, integer: bool = False):
    """A gated (SwiGLU) FFN problem: the Workload of the two-map FFN plus the gate bank.  Returns
    (workload, W_gate); the merged bank the library takes is [W_gate | workload.W_up]."""
    wl = make_workload(name, config=7, variant=300 + variant, dtype="bf16", q=q, M=M, D=D, F=F, types=types, integer=integer)
    s0 = seed_for(7, 300 + variant)
    Wg = small_ints(s0 + 4, (D, F)) if integer else bf16_round(normal(s0 + 4, (D, F), 0.02))
    return wl, Wg

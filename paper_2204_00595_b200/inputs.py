"""Seeded synthetic inputs for the Monarch multiply, shared by tests and bench.

This module holds no arithmetic of the method: it only draws Gaussian tensors
of the benchmark shapes and rounds them to the storage dtype, so that the CUDA
library and the CPU oracle see bit-identical values.

Recipe: ``numpy.random.default_rng(595000 + config)``; tensors are drawn in the
fixed order x, L, R, dy, L2, R2, b1, b2 as float32 ``standard_normal * std``
(only those the config uses), then rounded to nearest-even to the storage
dtype.  ``N(0, v)`` in the workload descriptions is read as variance v.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Config:
    index: int          # 1-based, as the workloads are numbered
    name: str
    dtype: str          # "f32" or "bf16" storage / operand type
    m: int
    tokens: int
    ops: tuple          # subset of ("fwd", "bwd_dx", "bwd_dw", "mlp_fwd")
    std_x: float
    std_w: float
    std_b: float = 0.0

    @property
    def n(self) -> int:
        return self.m * self.m


CONFIGS = {
    1: Config(1, "fwd f32 n=256 m=16 T=64", "f32", 16, 64, ("fwd",), 0.25, 0.25),
    2: Config(2, "fwd bf16 n=1024 m=32 T=16384", "bf16", 32, 16384, ("fwd",),
              1.0, 1.0 / math.sqrt(32)),
    3: Config(3, "fwd+bwd bf16 n=4096 m=64 T=8192", "bf16", 64, 8192,
              ("fwd", "bwd_dx", "bwd_dw"), 1.0, 1.0 / 8.0),
    4: Config(4, "fwd+bwd bf16 n=16384 m=128 T=4096", "bf16", 128, 4096,
              ("fwd", "bwd_dx", "bwd_dw"), 1.0, 1.0 / math.sqrt(128)),
    5: Config(5, "mlp fwd bf16 n=4096 m=64 T=32768", "bf16", 64, 32768,
              ("mlp_fwd",), 1.0, 1.0 / 8.0, math.sqrt(0.02)),
}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact promotion of bfloat16 bit patterns to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    """float32 array whose values are exactly representable in ``dtype``."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f32":
        return a
    if dtype == "bf16":
        return bf16_bits_to_f32(f32_to_bf16_bits(a)).reshape(a.shape)
    raise ValueError(dtype)


def make_inputs(config: int, tokens: int | None = None, m: int | None = None,
                dtype: str | None = None, seed: int | None = None, with_dy: bool = False) -> dict:
    """Draw the tensors of workload ``config`` (1..5).

    ``tokens``, ``m`` and ``dtype`` override the workload's values (for small
    parity cases of the same distribution).  Returns float32 arrays already
    rounded to the storage dtype, plus the scalars ``m``, ``n``, ``tokens``,
    ``dtype``.  ``with_dy`` adds an output gradient ``dy`` to workloads that
    do not list a backward call (for the backward of the feed-forward block).
    """
    c = CONFIGS[config]
    T = c.tokens if tokens is None else int(tokens)
    mm = c.m if m is None else int(m)
    dt = c.dtype if dtype is None else dtype
    std_w = c.std_w if m is None else 1.0 / math.sqrt(mm)
    n = mm * mm
    rng = np.random.default_rng(595000 + config if seed is None else seed)

    def draw(shape, std):
        a = rng.standard_normal(shape, dtype=np.float32) * np.float32(std)
        return round_to_storage(a, dt)

    out = {"m": mm, "n": n, "tokens": T, "dtype": dt, "config": config}
    out["x"] = draw((T, n), c.std_x)
    out["L"] = draw((mm, mm, mm), std_w)
    out["R"] = draw((mm, mm, mm), std_w)
    if "bwd_dx" in c.ops or "bwd_dw" in c.ops:
        out["dy"] = draw((T, n), 1.0)
    if "mlp_fwd" in c.ops:
        out["L2"] = draw((mm, mm, mm), std_w)
        out["R2"] = draw((mm, mm, mm), std_w)
        out["b1"] = draw((n,), c.std_b)
        out["b2"] = draw((n,), c.std_b)
    if with_dy and "dy" not in out:
        out["dy"] = draw((T, n), 1.0)      # drawn last: the tensors above do not depend on the flag
    return out


# General (rectangular) Monarch class of the paper's appendix: R has q blocks of b x b1, L has b blocks of
# r x q.  One measured case with the block count the paper's experiments use (four blocks).
RECT_WORKLOAD = {"q": 4, "b1": 1024, "b": 1024, "r": 4, "tokens": 8192, "dtype": "bf16"}


def make_rect_inputs(tokens: int | None = None, seed: int = 595006, **sizes) -> dict:
    """Seeded tensors x [T, q*b1], R [q, b, b1], L [b, r, q] of the general class (unit-variance
    activations, weights scaled so that u and y keep unit variance), rounded to the storage dtype."""
    cfg = dict(RECT_WORKLOAD)
    cfg.update(sizes)
    if tokens is not None:
        cfg["tokens"] = int(tokens)
    q, b1, b, r, T, dt = cfg["q"], cfg["b1"], cfg["b"], cfg["r"], cfg["tokens"], cfg["dtype"]
    rng = np.random.default_rng(seed)

    def draw(shape, std):
        return round_to_storage(rng.standard_normal(shape, dtype=np.float32) * np.float32(std), dt)

    out = dict(cfg)
    out["x"] = draw((T, q * b1), 1.0)
    out["R"] = draw((q, b, b1), 1.0 / math.sqrt(b1))
    out["L"] = draw((b, r, q), 1.0 / math.sqrt(q))
    return out


# The same class with wrapped-diagonal blocks (b2 != b3): R has q blocks of b2 x b1, L an r x q grid of b3 x b2 blocks
# with max(b2, b3) stored entries each.  One measured case beside the diagonal one: the same 4096 x 4096 product with
# blocks of L twice as tall as wide.
RECTW_WORKLOAD = {"q": 4, "b1": 1024, "b2": 1024, "b3": 2048, "r": 2, "tokens": 8192, "dtype": "bf16"}


def make_rectw_inputs(tokens: int | None = None, seed: int = 595009, **sizes) -> dict:
    """Seeded tensors x [T, q*b1], R [q, b2, b1], L [r, q, max(b2, b3)] of the wrapped-diagonal class (weights scaled
    so that u and y keep unit variance), rounded to the storage dtype."""
    cfg = dict(RECTW_WORKLOAD)
    cfg.update(sizes)
    if tokens is not None:
        cfg["tokens"] = int(tokens)
    q, b1, b2, b3, r, T, dt = cfg["q"], cfg["b1"], cfg["b2"], cfg["b3"], cfg["r"], cfg["tokens"], cfg["dtype"]
    rng = np.random.default_rng(seed)

    def draw(shape, std):
        return round_to_storage(rng.standard_normal(shape, dtype=np.float32) * np.float32(std), dt)

    out = dict(cfg)
    out["x"] = draw((T, q * b1), 1.0)
    out["R"] = draw((q, b2, b1), 1.0 / math.sqrt(b1))
    out["L"] = draw((r, q, max(b2, b3)), 1.0 / math.sqrt(q * max(1, b2 // b3)))
    return out


def to_device(a: np.ndarray, dtype: str):
    """float32 numpy array (already rounded to the storage dtype) -> torch CUDA tensor, exactly."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def to_host64(t) -> np.ndarray:
    """torch tensor (any float dtype, any device) -> float64 numpy array, exactly."""
    import torch
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)

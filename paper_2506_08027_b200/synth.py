"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module only draws numbers; it holds none of the MXFP8 arithmetic and imports
neither the CUDA binding nor the CPU oracle.  The tensors stand in for the activations,
weights and output gradients of the paper's GPT-style models (Sec. 3.1, Table 2): the
paper's training data and model checkpoints are not available, so shapes follow the
benchmark configurations and values follow the distributions named there.

Host tensors come from ``numpy.random.default_rng(seed)`` (PCG64) as float32 and are
rounded to bfloat16 (ties to even) where a bfloat16 source is asked for.  Large
benchmark tensors are drawn on the device with a seeded ``torch.Generator``; whoever
needs them on the host copies the bytes back, so both sides always see the same bits.
"""
from __future__ import annotations

import numpy as np

SEED_BASE = 250608027 * 1000


def seed_for(config: int, tensor_index: int) -> int:
    return SEED_BASE + 100 * config + tensor_index


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 bit patterns (uint16), ties to even, NaN kept quiet."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    nan = (u & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    out = np.where(nan, (u >> np.uint32(16)) | np.uint32(0x40), rounded)
    return out.astype(np.uint16)


def bf16_bits_as_f32(bits: np.ndarray) -> np.ndarray:
    """The float32 array holding exactly the values of these bfloat16 bit patterns."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def pr1_tensor(tensor_index: int = 0, rows: int = 256, cols: int = 512) -> np.ndarray:
    """The small reference tensor: FP32 [256, 512].

    z ~ N(0,1) times a per-row scale 2^u, u ~ U(-20, 10); 1 % of the elements times 100;
    four aligned 32x32 sub-tiles zeroed (all-zero blocks in both orientations); one row
    block and one column block whose amax is exactly 448.
    """
    rng = np.random.default_rng(seed_for(1, tensor_index))
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    u = rng.uniform(-20.0, 10.0, size=(rows, 1))
    x = (x * np.exp2(u)).astype(np.float32)
    outliers = rng.random((rows, cols)) < 0.01
    x = np.where(outliers, x * np.float32(100.0), x).astype(np.float32)
    for (tr, tc) in ((0, 0), (3, 7), (5, 2), (7, 15)):
        if (tr + 1) * 32 <= rows and (tc + 1) * 32 <= cols:
            x[tr * 32:(tr + 1) * 32, tc * 32:(tc + 1) * 32] = 0.0
    if rows >= 128 and cols >= 256:
        # row block: row 70, columns 128..159 ; column block: rows 96..127, column 200
        blk = x[70, 128:160]
        blk *= np.float32(2.0 ** -np.ceil(np.log2(max(np.abs(blk).max(), 1e-30) / 256.0)))
        np.clip(blk, -400.0, 400.0, out=blk)
        blk[5] = 448.0
        blk = x[96:128, 200]
        blk *= np.float32(2.0 ** -np.ceil(np.log2(max(np.abs(blk).max(), 1e-30) / 256.0)))
        np.clip(blk, -400.0, 400.0, out=blk)
        blk[11] = -448.0
    return x


def gaussian(shape, seed: int, std: float = 1.0) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return (rng.standard_normal(shape) * std).astype(np.float32)


def student_t(shape, seed: int, nu: float = 3.0) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.standard_t(nu, size=shape).astype(np.float32)


def gradient_like(shape, seed: int) -> np.ndarray:
    """z * 2^s with a per-row exponent s ~ N(log2 1e-8, 4.5) clipped to [-40, 0]."""
    rng = np.random.default_rng(seed)
    rows = shape[0]
    s = np.clip(rng.normal(np.log2(1e-8), 4.5, size=(rows, 1)), -40.0, 0.0)
    return (rng.standard_normal(shape) * np.exp2(s)).astype(np.float32)


def with_nonfinite(x: np.ndarray, seed: int, frac: float = 1e-4) -> np.ndarray:
    """Replace a fraction of the elements by NaN, +Inf, -Inf in equal thirds."""
    rng = np.random.default_rng(seed)
    x = x.copy()
    n = max(3, int(round(x.size * frac)))
    idx = rng.choice(x.size, size=n, replace=False)
    flat = x.reshape(-1)
    flat[idx[0::3]] = np.nan
    flat[idx[1::3]] = np.inf
    flat[idx[2::3]] = -np.inf
    return x


def output_gradient(shape, seed: int) -> np.ndarray:
    """dY = 1e-6 * exp(2 g_t) * z with g_t ~ N(0,1) per row (log-normal row spread)."""
    rng = np.random.default_rng(seed)
    g = rng.standard_normal((shape[0], 1))
    return (1e-6 * np.exp(2.0 * g) * rng.standard_normal(shape)).astype(np.float32)


DISTRIBUTIONS = ("gaussian", "student_t", "gradient_like", "nonfinite")


def draw(dist: str, shape, seed: int) -> np.ndarray:
    if dist == "gaussian":
        return gaussian(shape, seed)
    if dist == "student_t":
        return student_t(shape, seed)
    if dist == "gradient_like":
        return gradient_like(shape, seed)
    if dist == "nonfinite":
        return with_nonfinite(gaussian(shape, seed), seed + 1)
    raise ValueError(dist)


# ---------------------------------------------------------------------------------
# Device-side draws for tensors too large to generate on the host in reasonable time.
# ---------------------------------------------------------------------------------

def device_tensor(kind: str, shape, seed: int, dtype="bf16", device="cuda"):
    """A seeded tensor drawn on ``device``; kind in {activation, weight, output_gradient,
    gaussian, student_t, gradient_like, nonfinite (Gaussian with 0.01 % of the elements replaced by NaN, +Inf, -Inf
    in equal thirds)}."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(seed)
    rows = shape[0]

    def randn(*s):
        return torch.randn(*s, generator=g, device=device, dtype=torch.float32)

    if kind in ("activation", "gaussian"):
        x = randn(*shape)
    elif kind == "nonfinite":
        x = randn(*shape)
        u = torch.rand(*shape, generator=g, device=device, dtype=torch.float32)
        x = torch.where(u < 1e-4 / 3, torch.full_like(x, float("nan")), x)
        x = torch.where((u >= 1e-4 / 3) & (u < 2e-4 / 3), torch.full_like(x, float("inf")), x)
        x = torch.where((u >= 2e-4 / 3) & (u < 1e-4), torch.full_like(x, float("-inf")), x)
    elif kind == "weight":
        x = randn(*shape) * 0.02
    elif kind == "output_gradient":
        x = randn(*shape) * (1e-6 * torch.exp(2.0 * randn(rows, 1)))
    elif kind == "student_t":
        z = randn(*shape)
        w = (randn(*shape) ** 2 + randn(*shape) ** 2 + randn(*shape) ** 2) / 3.0
        x = z / torch.sqrt(w)
    elif kind == "gradient_like":
        s = torch.clamp(randn(rows, 1) * 4.5 + float(np.log2(1e-8)), -40.0, 0.0)
        x = randn(*shape) * torch.exp2(s)
    else:
        raise ValueError(kind)
    return x.to(torch.bfloat16) if dtype == "bf16" else x.contiguous()

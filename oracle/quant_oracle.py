"""The exit layers' weight quantiser, stated plainly on the CPU (numpy, fp32 arithmetic).

TEST INFRASTRUCTURE ONLY: only tests/ may import this module; the CUDA library shares no code with it.

What it follows.  River-LLM builds an exit layer by copying a backbone block and applying a training-free 4-bit
weight-only quantisation (HQQ) to its Attention and FFN matrices (paper Section 4.1, "within one minute").  HQQ is
a half-quadratic solver for the zero-point of an affine grid: with the scale fixed by the group's range it alternates
  W_q = clamp(round(W / s + z), 0, 15)                    (quantise)
  W_e = shrink_p(W - (W_q - z) s; beta)                   (generalised soft threshold of the residual, l_p norm, p < 1)
  z   = mean over the group of (W_q - (W - W_e) / s)      (closed-form zero-point update)
with beta growing by kappa per iteration.  Groups of `group` inputs along a row; codes u4 in [0, 15]; scale and zero
stored as bf16; w ~ (q - z) s.  With zero iterations this is the plain min/max round-to-nearest grid.

Precision: the codes are integers decided by floating point, so every operation below is a single fp32 operation in a
fixed order (sums over a group run sequentially over its inputs) - the precision and order the CUDA kernel uses.
Constants: p = 0.7, beta0 = 10, kappa = 1.01 (the defaults HQQ publishes).

Pins (tests/test_quant_oracle.py): zero iterations against the closed min/max formula and against the independent
torch generator of the workloads; grid bounds; exact round trip of on-grid and of constant groups; a one-iteration
example worked by hand in float64; refinement lowers the l_p residual of heavy-tailed groups.
"""
from __future__ import annotations

import numpy as np

P_NORM = np.float32(0.7)
BETA0 = np.float32(10.0)
KAPPA = np.float32(1.01)
F = np.float32


def _bf16_round(x: np.ndarray) -> np.ndarray:
    """fp32 -> nearest bf16 (ties to even), returned as fp32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def _seq_sum(a: np.ndarray) -> np.ndarray:
    """Sum over the last axis, sequentially in fp32 (the order a thread that owns the group uses)."""
    acc = np.zeros(a.shape[:-1], np.float32)
    for k in range(a.shape[-1]):
        acc = (acc + a[..., k]).astype(np.float32)
    return acc


def quantize_w4(w: np.ndarray, group: int = 64, refine_iters: int = 20, return_float_zero: bool = False):
    """w fp32 [out, in] (bf16-representable values) -> (codes u8 [out, in/2], scale fp32 [out, in/g], zero fp32 [out, in/g]);
    scale and zero hold bf16-representable values.  Low nibble = even input."""
    out, inn = w.shape
    assert inn % group == 0 and group % 2 == 0
    g = np.ascontiguousarray(w, dtype=np.float32).reshape(out, inn // group, group)
    mn = g.min(axis=2)
    mx = g.max(axis=2)
    const = mx == mn
    s = _bf16_round(((mx - mn).astype(F) / F(15.0)).astype(F))
    s = np.where(const | (s == 0), F(1.0), s).astype(F)
    z = ((-mn).astype(F) / s).astype(F)
    s3 = s[..., None]
    beta = BETA0
    for _ in range(refine_iters):
        q = np.clip(np.rint((g / s3).astype(F) + z[..., None]).astype(F), F(0), F(15))
        r = ((q - z[..., None]).astype(F) * s3).astype(F)
        e = (g - r).astype(F)
        ae = np.abs(e)
        with np.errstate(divide="ignore", invalid="ignore"):
            t = (ae - ((F(1.0) / beta) * np.power(ae, P_NORM - F(1.0), dtype=F)).astype(F)).astype(F)
        we = np.where(ae > 0, np.sign(e) * np.maximum(t, F(0)), F(0)).astype(F)
        term = (q - ((g - we).astype(F) / s3).astype(F)).astype(F)
        z = (_seq_sum(term) / F(group)).astype(F)
        beta = F(beta * KAPPA)
    z_float = z.copy()
    zb = _bf16_round(z)
    zb = np.where(const, _bf16_round((-mn).astype(F)), zb).astype(F)
    q = np.clip(np.rint((g / s3).astype(F) + zb[..., None]).astype(F), F(0), F(15))
    q = np.where(const[..., None], F(0), q).astype(np.uint8).reshape(out, inn)
    codes = (q[:, 0::2] | (q[:, 1::2] << 4)).astype(np.uint8)
    if return_float_zero:
        return codes, s, zb, z_float
    return codes, s, zb


def dequantize(codes: np.ndarray, scale: np.ndarray, zero: np.ndarray, group: int = 64) -> np.ndarray:
    out, half = codes.shape
    q = np.empty((out, half * 2), np.float64)
    q[:, 0::2] = codes & 15
    q[:, 1::2] = codes >> 4
    return (q - np.repeat(zero.astype(np.float64), group, axis=1)) * np.repeat(scale.astype(np.float64), group, axis=1)

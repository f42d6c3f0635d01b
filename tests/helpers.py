"""Shared test helpers: draw a model once, hand the same buffers to whoever needs them."""
from __future__ import annotations

import functools

import numpy as np
import torch

from workloads import rtn_w4, synth


@functools.lru_cache(maxsize=4)
def cpu_model(name: str, n_layers=None, first_river_layer0: int = 0):
    """(shape, backbone, river) on the CPU for a named shape."""
    shape = synth.SHAPES[name]
    bb = synth.make_backbone(shape, "cpu", n_layers)
    rv = rtn_w4.make_river(bb, shape.group, first_river_layer0)
    return shape, bb, rv


def f64(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).numpy()


def dequant_np(codes: torch.Tensor, scale: torch.Tensor, zero: torch.Tensor, group: int) -> np.ndarray:
    c = codes.numpy()
    out, half = c.shape
    q = np.empty((out, half * 2), np.float64)
    q[:, 0::2] = c & 15
    q[:, 1::2] = c >> 4
    s = np.repeat(f64(scale), group, axis=1)
    z = np.repeat(f64(zero), group, axis=1)
    return (q - z) * s


def cosine(a: np.ndarray, b: np.ndarray) -> float:
    a = a.astype(np.float64).ravel()
    b = b.astype(np.float64).ravel()
    return float(a @ b / (np.linalg.norm(a) * np.linalg.norm(b)))

"""Seeded synthetic inputs for the early-exit decode path.

This module only *draws inputs*: weights, token ids, prompt lengths, exit schedules.  It
holds none of the method's arithmetic (no norm, projection, attention, score or
dequantisation) and is the one piece of code both the CPU oracle's tests and the CUDA
path's tests / benchmark use, so that both consume byte-identical buffers.

Random numbers come from a counter-based generator (a splitmix64-style integer hash of
(seed, stream, index) followed by Box-Muller in fp64) written with plain torch tensor ops,
so a tensor can be drawn directly on the device that needs it.  A model is always drawn
once and the very same buffers are handed to both sides (copied across devices, never
re-drawn), so parity never depends on two devices agreeing on a transcendental's last bit.

Recipe (stands in for the paper's real checkpoints, which are not available): weights
N(0, 0.02) in bf16; the residual-writing matrices (attention output and FFN down
projection) of 0-based layer l are scaled by resid_decay**l so that the block input/output
cosine similarity rises with depth, as the paper's Fig. 6(b) reports for trained models;
norm gains 1; token ids uniform in [0, V).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import torch

_M1 = -4658895280553007687  # 0xBF58476D1CE4E5B9 as int64
_M2 = -7723592293110705685  # 0x94D049BB133111EB as int64
_GOLD = -7046029254386353131  # 0x9E3779B97F4A7C15 as int64


def _lshr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lshr(x, 30)) * _M1
    x = (x ^ _lshr(x, 27)) * _M2
    return x ^ _lshr(x, 31)


def _key(seed: int, stream: int) -> int:
    """Scalar 64-bit key for (seed, stream), computed with python ints."""
    mask = (1 << 64) - 1
    x = (seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & mask
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & mask
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & mask
    x = x ^ (x >> 31)
    return x - (1 << 64) if x >= (1 << 63) else x


def hash_u64(seed: int, stream: int, n: int, device="cpu", start: int = 0) -> torch.Tensor:
    """n hashed 64-bit words (as int64) for counters start..start+n-1."""
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    return _mix64(idx * _GOLD + _key(seed, stream))


def uniform_int(seed: int, stream: int, n: int, lo: int, hi: int, device="cpu") -> torch.Tensor:
    """n integers uniform in [lo, hi) (int64)."""
    u = _lshr(hash_u64(seed, stream, n, device), 11)  # 53 bits
    return lo + (u % (hi - lo))


def normal(seed: int, stream: int, shape, std: float, device="cpu", dtype=torch.bfloat16,
           chunk: int = 1 << 25) -> torch.Tensor:
    """Tensor of N(0, std^2) samples, drawn chunk by chunk to bound temporaries."""
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        hw = hash_u64(seed, stream, m, device, start=s)
        u1 = (_lshr(hw, 32).to(torch.float64) + 0.5) * (1.0 / 4294967296.0)
        u2 = ((hw & 0xFFFFFFFF).to(torch.float64) + 0.5) * (1.0 / 4294967296.0)
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        out[s:s + m] = (z * std).to(torch.float32).to(dtype)
    return out.view(*shape)


@dataclasses.dataclass
class ModelShape:
    name: str
    L: int
    d: int
    Hq: int
    Hkv: int
    dh: int
    F: int
    V: int
    seed: int
    resid_decay: float
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    entry_layer: int = 1
    group: int = 64

    def layer_params(self) -> int:
        return self.d * self.Hq * self.dh + 2 * self.d * self.Hkv * self.dh + self.Hq * self.dh * self.d \
            + 3 * self.d * self.F


def _rel_decay(L: int) -> float:
    # same total decay over the depth as 0.5**3 over the tiny model's 4 layers
    return 0.125 ** (1.0 / (L - 1))


SHAPES: Dict[str, ModelShape] = {
    "tiny": ModelShape("tiny", 4, 256, 4, 2, 64, 1024, 1024, seed=0, resid_decay=0.5),
    "1b": ModelShape("1b", 16, 2048, 32, 8, 64, 8192, 128256, seed=1, resid_decay=_rel_decay(16)),
    "8b": ModelShape("8b", 32, 4096, 32, 8, 128, 14336, 128256, seed=2, resid_decay=_rel_decay(32)),
    # a mid-size shape with the 8B head geometry (dh 128, group 4) for fast multi-tile tests
    "mini8": ModelShape("mini8", 6, 512, 8, 2, 128, 1536, 4096, seed=5, resid_decay=_rel_decay(6)),
}

MATS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")


def mat_dims(s: ModelShape) -> Dict[str, tuple]:
    return {
        "wq": (s.Hq * s.dh, s.d), "wk": (s.Hkv * s.dh, s.d), "wv": (s.Hkv * s.dh, s.d),
        "wo": (s.d, s.Hq * s.dh), "wg": (s.F, s.d), "wu": (s.F, s.d), "wd": (s.d, s.F),
    }


def make_backbone(s: ModelShape, device="cpu", n_layers: Optional[int] = None) -> dict:
    """Draw the bf16 backbone.  Returns {'embed','lm_head','final_norm','layers':[{...}]}."""
    L = s.L if n_layers is None else n_layers
    dims = mat_dims(s)
    w = {
        "embed": normal(s.seed, 1, (s.V, s.d), 0.02, device),
        "lm_head": normal(s.seed, 2, (s.V, s.d), 0.02, device),
        "final_norm": torch.ones(s.d, dtype=torch.bfloat16, device=device),
        "layers": [],
    }
    for l in range(L):
        lay = {
            "attn_norm": torch.ones(s.d, dtype=torch.bfloat16, device=device),
            "ffn_norm": torch.ones(s.d, dtype=torch.bfloat16, device=device),
        }
        for j, name in enumerate(MATS):
            std = 0.02 * (s.resid_decay ** l if name in ("wo", "wd") else 1.0)
            lay[name] = normal(s.seed, 16 + l * 8 + j, dims[name], std, device)
        w["layers"].append(lay)
    return w


def tokens(seed: int, stream: int, n: int, V: int) -> torch.Tensor:
    return uniform_int(seed, 1000 + stream, n, 0, V).to(torch.int32)


def prompt_lengths(seed: int, n: int, lo: int, hi: int) -> List[int]:
    return [int(v) for v in uniform_int(seed, 2000, n, lo, hi + 1)]


def forced_exit_schedule(seed: int, stream: int, n: int, L: int, entry_layer: int, kind: str = "uniform",
                         mean: float = 3.0) -> torch.Tensor:
    """Seeded target exit layers in [max(entry_layer,1), L] (L = runs the whole backbone)."""
    lo = max(entry_layer, 1)
    if kind == "uniform":
        return uniform_int(seed, 3000 + stream, n, lo, L + 1).to(torch.int32)
    if kind == "geometric":
        u = (_lshr(hash_u64(seed, 3000 + stream, n), 11).to(torch.float64) + 0.5) / float(1 << 53)
        p = 1.0 / max(mean - lo + 1.0, 1.0)
        k = torch.floor(torch.log(u) / math.log(1.0 - p)).to(torch.int64)
        return torch.clamp(lo + k, max=L).to(torch.int32)
    raise ValueError(kind)


def shuffled(seed: int, stream: int, n: int) -> List[int]:
    """A seeded permutation of range(n) (sort by hashed key)."""
    return [int(v) for v in torch.argsort(_lshr(hash_u64(seed, 4000 + stream, n), 1))]

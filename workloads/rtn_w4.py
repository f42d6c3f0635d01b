"""Round-to-nearest 4-bit weight-only quantiser that prepares the Exit River's weights.

Input preparation, not part of the decode path: the paper builds each exit layer by
copying a backbone block and applying a training-free 4-bit weight-only PTQ to its
Attention and FFN matrices (Section 4.1).  Its HQQ zero-point refinement is an offline
step outside this build; a plain min/max affine grid per group of `group` input columns
stands in.  Both the CPU oracle and the CUDA path consume the codes / scales / zeros this
module emits (w = (q - z) * s), so the choice of quantiser cannot affect parity.

Layout: codes u8 [out, in/2], low nibble = even input index; scale, zero bf16 [out, in/group].
"""
from __future__ import annotations

import torch


def quantize_w4(w: torch.Tensor, group: int = 64):
    """w bf16/fp32 [out, in] -> (codes u8 [out,in/2], scale bf16 [out,in/g], zero bf16 [out,in/g])."""
    out, inn = w.shape
    assert inn % group == 0 and group % 2 == 0
    g = w.to(torch.float32).view(out, inn // group, group)
    mn = g.amin(dim=2, keepdim=True)
    mx = g.amax(dim=2, keepdim=True)
    const = mx == mn
    s = ((mx - mn) / 15.0).to(torch.bfloat16).to(torch.float32)
    s = torch.where(const | (s == 0), torch.ones_like(s), s)
    z = (-mn / s).to(torch.bfloat16).to(torch.float32)
    z = torch.where(const, (-mn).to(torch.bfloat16).to(torch.float32), z)  # constant group: q = 0, (0 - z) * 1 = w
    q = torch.clamp(torch.round(g / s + z), 0, 15)  # torch.round: half to even
    q = torch.where(const, torch.zeros_like(q), q).to(torch.uint8).view(out, inn)
    codes = (q[:, 0::2] | (q[:, 1::2] << 4)).contiguous()
    return codes, s.view(out, inn // group).to(torch.bfloat16), z.view(out, inn // group).to(torch.bfloat16)


def snap_to_grid(w: torch.Tensor, group: int = 64):
    """Snap weights onto a 4-bit grid that bf16 holds exactly (for the identity-river invariant).

    Returns (w_snapped bf16, codes, scale, zero) with (codes - zero) * scale == w_snapped exactly:
    integer steps in [-7, 7] around a zero of 8 with a power-of-two scale per group."""
    out, inn = w.shape
    g = w.to(torch.float32).view(out, inn // group, group)
    amax = g.abs().amax(dim=2, keepdim=True).clamp_min(1e-30)
    s = torch.exp2(torch.ceil(torch.log2(amax / 7.0)))
    q = torch.clamp(torch.round(g / s), -7, 7)
    snapped = (q * s).view(out, inn).to(torch.bfloat16)
    qq = (q + 8).to(torch.uint8).view(out, inn)
    codes = (qq[:, 0::2] | (qq[:, 1::2] << 4)).contiguous()
    scale = s.view(out, inn // group).to(torch.bfloat16)
    zero = torch.full_like(scale, 8.0)
    return snapped, codes, scale, zero


def make_river(backbone: dict, group: int = 64, first_layer0: int = 0) -> list:
    """River copy of every 0-based layer >= first_layer0: {name: (codes, scale, zero)} or None."""
    river = []
    for l, lay in enumerate(backbone["layers"]):
        if l < first_layer0:
            river.append(None)
            continue
        river.append({n: quantize_w4(lay[n], group) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd")})
    return river

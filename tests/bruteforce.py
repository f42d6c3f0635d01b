"""A no-cache, whole-sequence recompute of decode-with-exit in numpy fp64.

Independent of the oracle's C code: no KV cache and no step loop.  Given the token
history and the number of backbone blocks each token ran (its exit layer), every block is
evaluated for all positions at once with a dense causal softmax; token i uses the
backbone weights in blocks 1..e_i and the dequantised river weights afterwards
(paper, Section 4.2).  Used to pin the oracle's cache slots, positions, causal range and
per-token path choice on tiny inputs.
"""
from __future__ import annotations

import numpy as np

from tests.helpers import dequant_np, f64


def _rms(H, g, eps):
    return H / np.sqrt((H * H).mean(axis=1, keepdims=True) + eps) * g


def _rope(X, n_heads, dh, theta):
    T = X.shape[0]
    X = X.reshape(T, n_heads, dh).copy()
    half = dh // 2
    inv = theta ** (-2.0 * np.arange(half) / dh)
    ang = np.arange(T)[:, None] * inv[None, :]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = X[..., :half].copy(), X[..., half:].copy()
    X[..., :half] = a * c - b * s
    X[..., half:] = b * c + a * s
    return X.reshape(T, n_heads * dh)


def _bf16(x):
    import torch
    return torch.from_numpy(x).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def recompute(shape, bb, rv, tokens, exit_layers, kv_bf16=False, strategy=0):
    """-> logits [T,V], K [L,T,Hkv*dh] (after RoPE), V [L,T,Hkv*dh], scores [T,L].
    kv_bf16: keys and values are rounded to bf16 (through torch's cast) before they are used or returned.
    strategy (what a skipped block does, Section 3): 0 = the quantised copy of the block runs (Section 4.1); 1 = State
    Propagation: K/V of the block from the hidden state at the exit through the BACKBONE's K / V projections, the
    hidden state itself unchanged; 2 = Mono-Decreasing Exit: nothing (the block's K/V rows of that token come back as
    NaN; no later token may need them, which holds when the exit layers never increase); 3 = KV Mask: nothing either,
    and a token's attention in a block sees only the earlier positions whose token ran that block, and itself."""
    tokens = np.asarray(tokens)
    e = np.asarray(exit_layers)
    T = len(tokens)
    L = len(bb["layers"])
    Hq, Hkv, dh = shape.Hq, shape.Hkv, shape.dh
    H = f64(bb["embed"])[tokens]
    Ks, Vs = [], []
    scores = np.full((T, L), np.nan)
    causal = np.tril(np.ones((T, T), bool))
    for l in range(1, L + 1):
        lay = bb["layers"][l - 1]
        in_river = e < l

        def proj(name, X):
            Y = X @ f64(lay[name]).T
            if in_river.any() and strategy == 0:
                Wr = dequant_np(*rv[l - 1][name], shape.group)
                Y = np.where(in_river[:, None], X @ Wr.T, Y)
            return Y

        x = _rms(H, f64(lay["attn_norm"]), shape.rms_eps)
        q = _rope(proj("wq", x), Hq, dh, shape.rope_theta).reshape(T, Hq, dh)
        k = _rope(proj("wk", x), Hkv, dh, shape.rope_theta)
        v = proj("wv", x)
        if kv_bf16:
            k, v = _bf16(k), _bf16(v)
        if strategy == 2:
            assert all(e[j] <= e[i] for i in range(T) for j in range(i + 1, T)), "exit layers must not increase"
        if strategy in (2, 3):
            k = np.where(in_river[:, None], np.nan, k)
            v = np.where(in_river[:, None], np.nan, v)
        visible = causal if strategy != 3 else causal & (~in_river[None, :] | np.eye(T, dtype=bool))
        Ks.append(k)
        Vs.append(v)
        k3, v3 = np.nan_to_num(k).reshape(T, Hkv, dh), np.nan_to_num(v).reshape(T, Hkv, dh)
        att = np.empty((T, Hq, dh))
        for i in range(Hq):
            j = i // (Hq // Hkv)
            sc = q[:, i, :] @ k3[:, j, :].T / np.sqrt(dh)
            sc = np.where(visible, sc, -np.inf)
            p = np.exp(sc - sc.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            att[:, i, :] = p @ v3[:, j, :]
        Hm = H + proj("wo", att.reshape(T, Hq * dh))
        y = _rms(Hm, f64(lay["ffn_norm"]), shape.rms_eps)
        g = proj("wg", y)
        u = proj("wu", y)
        Hn = Hm + proj("wd", g / (1.0 + np.exp(-g)) * u)
        s = (H * Hn).sum(1) / (np.linalg.norm(H, axis=1) * np.linalg.norm(Hn, axis=1))
        scores[:, l - 1] = np.where(in_river, np.nan, s)
        H = Hn if strategy == 0 else np.where(in_river[:, None], H, Hn)
    logits = _rms(H, f64(bb["final_norm"]), shape.rms_eps) @ f64(bb["lm_head"]).T
    return logits, np.stack(Ks), np.stack(Vs), scores

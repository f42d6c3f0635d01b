"""Single stages of the path through the C ABI against the oracle's pieces (needs a B200).

river_attention (step a3) against the oracle's attention over the same cache, and river_project_kv (step a2, on the
bf16 block and on its 4-bit exit-layer copy) against a numpy fp64 evaluation of norm -> projection -> rotary embedding.
"""
import numpy as np
import pytest
import torch

from tests.gpu_harness import KV_RTOL, Pair, draw_model
from tests.helpers import dequant_np, f64
from workloads import synth

pytestmark = pytest.mark.gpu

_m = {}


def model(name, n_layers=None):
    if (name, n_layers) not in _m:
        _m[(name, n_layers)] = draw_model(name, n_layers)
    return _m[(name, n_layers)]


@pytest.mark.parametrize("lens", [[700], [33, 1, 250], [1500, 16, 640, 5, 2047, 90, 300]])
def test_attention_stage_matches_oracle_attention(lens):
    # one row and three rows: the small-step kernel; seven rows: the TMA-fed split-KV kernel
    m = model("mini8")
    shape = m[0]
    B = len(lens)
    p = Pair(m, B, max(lens) + 1, 8, page_shuffle_seed=13, kv_store=1)
    p.fill_history(lens)
    w = shape.Hq * shape.dh
    for layer in (1, p.L):
        q = synth.normal(77, layer, (B, w), 1.0, "cuda", torch.float32)
        out = torch.full((B, w), float("nan"), dtype=torch.float32, device="cuda")
        order = synth.shuffled(5, layer, B)
        p.gpu.attention(layer, [int(i) for i in order], q, out)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        qn = q.cpu().numpy()
        for i, s in enumerate(order):
            want = p.oracle.attention(layer - 1, int(s), lens[s] - 1, qn[i])
            err = np.abs(got[i] - want).max()
            assert np.isfinite(got[i]).all() and err < 2e-3 * max(1.0, np.abs(want).max()), (layer, s, err)
    assert p.gpu.stats().device_error == 0
    p.close()


def _rope_at(x, n_heads, dh, theta, pos):
    x = x.reshape(n_heads, dh).copy()
    half = dh // 2
    ang = pos * theta ** (-2.0 * np.arange(half) / dh)
    a, b = x[:, :half].copy(), x[:, half:].copy()
    x[:, :half] = a * np.cos(ang) - b * np.sin(ang)
    x[:, half:] = b * np.cos(ang) + a * np.sin(ang)
    return x.reshape(-1)


@pytest.mark.parametrize("name,rows,exit_layer", [("mini8", 1, 1), ("mini8", 3, 0), ("mini8", 3, 1), ("mini8", 7, 0),
                                                  ("mini8", 7, 1), ("8b", 7, 0), ("8b", 7, 1), ("8b", 2, 1)])
def test_project_kv_stage_matches_numpy(name, rows, exit_layer):
    # K/V generation for the newest position on the backbone block and on its exit-layer copy: the same cache slot
    # either way (Section 4.1).  One to three rows: streaming kernel; seven rows: the tcgen05 GEMMs.  On the 8B layer
    # shape too: with the block's input given, the plain K/V tolerance holds there as well (no amplification through
    # earlier layers).
    m = model(name, 4 if name == "8b" else None)
    shape, (bb, rv), _ = m
    lens = [40, 9, 75, 18, 31, 6, 17][:rows]
    p = Pair(m, rows, 80, 8, page_shuffle_seed=21)
    p.fill_history(lens)
    layer = min(4, len(bb["layers"]))
    lay, riv = bb["layers"][layer - 1], rv[layer - 1]
    h = synth.normal(88, 0, (rows, shape.d), 1.0, "cuda", torch.float32)
    qo = torch.empty((rows, shape.Hq * shape.dh), dtype=torch.float32, device="cuda")
    slots = list(range(rows))
    before = [p.gpu.read_kv(s, layer, 0, lens[s]) for s in slots]
    p.gpu.project_kv(layer, bool(exit_layer), slots, h, qo)
    torch.cuda.synchronize()
    hn = h.cpu().numpy().astype(np.float64)
    x = hn / np.sqrt((hn * hn).mean(axis=1, keepdims=True) + shape.rms_eps) * f64(lay["attn_norm"])
    W = {n: (dequant_np(*riv[n], shape.group) if exit_layer else f64(lay[n])) for n in ("wq", "wk", "wv")}
    for s in slots:
        pos = lens[s] - 1
        q = _rope_at(W["wq"] @ x[s], shape.Hq, shape.dh, shape.rope_theta, pos)
        k = _rope_at(W["wk"] @ x[s], shape.Hkv, shape.dh, shape.rope_theta, pos)
        v = W["wv"] @ x[s]
        kg, vg = p.gpu.read_kv(s, layer, 0, lens[s])
        assert np.abs(qo[s].cpu().numpy() - q).max() < 1e-3 * max(1.0, np.abs(q).max())
        for got, want in ((kg[pos], k), (vg[pos], v)):
            got = got.float().cpu().numpy()
            bound = KV_RTOL * np.abs(want) + KV_RTOL * np.sqrt((want ** 2).mean())
            assert (np.abs(got - want) <= bound).all()
        # every other cached position is untouched
        assert torch.equal(kg[:pos], before[s][0][:pos]) and torch.equal(vg[:pos], before[s][1][:pos])
    assert p.gpu.stats().device_error == 0
    p.close()

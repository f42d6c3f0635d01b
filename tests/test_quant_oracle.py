"""Pins of the quantiser oracle (CPU only): the zero-point refinement of the exit layers' 4-bit grid."""
import numpy as np
import torch

from oracle import quant_oracle as qo
from workloads import rtn_w4, synth


def _bf16(x):
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def _weights(out=24, inn=256, seed=3, heavy=False):
    w = synth.normal(seed, 11, (out, inn), 0.02, "cpu", torch.float32).numpy()
    if heavy:  # a few large entries per group, as trained weight matrices have
        idx = synth.uniform_int(seed, 12, out * (inn // 64), 0, 64).numpy().reshape(out, inn // 64)
        for o in range(out):
            for g in range(inn // 64):
                w[o, g * 64 + idx[o, g]] *= 8.0
    return _bf16(w)


def test_zero_iterations_is_the_minmax_grid_and_matches_the_workload_generator():
    w = _weights()
    codes, s, z = qo.quantize_w4(w, 64, 0)
    g = w.reshape(24, 4, 64)
    mn, mx = g.min(axis=2), g.max(axis=2)
    s_want = _bf16((mx - mn) / np.float32(15.0))
    z_want = _bf16(-mn / s_want)
    assert np.array_equal(s, s_want) and np.array_equal(z, z_want)
    q = np.clip(np.rint(g / s_want[..., None] + z_want[..., None]), 0, 15).reshape(24, 256)
    assert np.array_equal(codes & 15, q[:, 0::2].astype(np.uint8)) and np.array_equal(codes >> 4, q[:, 1::2].astype(np.uint8))
    c2, s2, z2 = rtn_w4.quantize_w4(torch.from_numpy(w), 64)  # independent torch implementation
    assert np.array_equal(codes, c2.numpy()) and np.array_equal(s, s2.float().numpy()) and np.array_equal(z, z2.float().numpy())


def test_grid_bounds_and_exact_round_trips():
    w = _weights(heavy=True)
    for iters in (0, 20):
        codes, s, z = qo.quantize_w4(w, 64, iters)
        assert codes.max() <= 255 and (codes & 15).max() <= 15
        d = qo.dequantize(codes, s, z, 64)
        q = np.empty(w.shape)
        q[:, 0::2], q[:, 1::2] = codes & 15, codes >> 4
        interior = (q > 0) & (q < 15)  # codes not clamped: within half a step
        assert (np.abs(d - w)[interior] <= 0.5 * np.repeat(s, 64, axis=1)[interior] * (1 + 1e-6)).all()
    # a matrix that already sits on a 16-level grid spanning each group's range (power-of-two step, integer zero, both
    # end codes present) is reproduced exactly, with or without refinement
    qs = synth.uniform_int(5, 1, 8 * 256, 0, 16).numpy().reshape(8, 256).astype(np.float32)
    qs[:, 0::64] = 0
    qs[:, 1::64] = 15
    ws = ((qs - 6.0) * np.float32(2.0 ** -6)).astype(np.float32)
    for iters in (0, 20):
        codes, s, z = qo.quantize_w4(ws, 64, iters)
        assert np.array_equal(qo.dequantize(codes, s, z, 64), ws.astype(np.float64))
        assert np.array_equal(codes & 15, qs[:, 0::2].astype(np.uint8)) and (z == 6.0).all()
    const = np.full((2, 64), np.float32(0.0123), np.float32)
    const = _bf16(const)
    codes, s, z = qo.quantize_w4(const, 64, 20)
    assert np.array_equal(qo.dequantize(codes, s, z, 64), const.astype(np.float64))


def test_one_refinement_step_worked_by_hand():
    # one group of four inputs, one iteration, every step in float64 by hand
    w = _bf16(np.array([[-0.5, 0.0, 0.25, 1.0]], np.float32))
    codes, s, zb, zf = qo.quantize_w4(w, 4, 1, return_float_zero=True)
    s0 = float(_bf16(np.float32(1.5 / 15.0)))  # range 1.5 over 15 steps
    z0 = 0.5 / s0
    q = np.clip(np.rint(w[0].astype(np.float64) / s0 + z0), 0, 15)
    e = w[0] - (q - z0) * s0
    ae = np.abs(e)
    shr = np.where(ae > 0, np.sign(e) * np.maximum(ae - (1 / 10.0) * np.power(ae, 0.7 - 1.0, where=ae > 0, out=np.ones_like(ae)), 0), 0)
    z1 = np.mean(q - (w[0] - shr) / s0)
    assert abs(float(s[0, 0]) - s0) == 0 and abs(float(zf[0, 0]) - z1) < 1e-5 * abs(z1)
    assert float(zb[0, 0]) == float(_bf16(np.float32(zf[0, 0])))


def test_refinement_lowers_the_lp_residual_of_heavy_tailed_groups():
    w = _weights(out=64, inn=512, seed=9, heavy=True)
    lp = []
    for iters in (0, 20):
        codes, s, z = qo.quantize_w4(w, 64, iters)
        lp.append((np.abs(qo.dequantize(codes, s, z, 64) - w) ** 0.7).sum())
    assert lp[1] <= lp[0]
    print(f"l_0.7 residual: round-to-nearest {lp[0]:.3f}, refined {lp[1]:.3f}")

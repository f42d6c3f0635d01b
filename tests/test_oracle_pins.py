"""Pins of the CPU oracle against things other than itself (CPU only).

Each test fixes one piece of the oracle to what the paper or the mathematics fixes:
a brute-force recompute, closed forms of Eq. 1, textbook attention / RoPE / matmul
special cases, invariants of the method (cache completeness, identity river, full-depth
and full-quantisation limits), the cache-size figure of the paper's memory table.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import river_oracle as orc
from tests import bruteforce
from tests.helpers import cosine, cpu_model, dequant_np, f64
from workloads import rtn_w4, synth

INF = float("inf")


def _tokens(shape, n, stream=0):
    return synth.tokens(shape.seed, stream, n, shape.V).numpy()


def _run(oracle, slot, prompt, steps_tok, tau, forced=None, prefill_exit=None):
    """prefill + teacher-forced decode of one sequence; returns per-step outputs."""
    oracle.prefill(slot, prompt, prefill_exit)
    outs = []
    for t, tk in enumerate(steps_tok):
        fe = None if forced is None else [forced[t]]
        outs.append(oracle.decode_step([slot], [tk], tau, fe))
    return outs


@pytest.fixture(scope="module")
def tiny():
    return cpu_model("tiny")


def _median_tau(tiny, prompt, steps):
    shape, bb, rv = tiny
    o = orc.Oracle(shape, bb, rv, 1, 64)
    outs = _run(o, 0, prompt, steps, INF)
    sc = np.stack([r["scores"][0] for r in outs])  # [T, L]
    return float(np.median(sc[:, shape.entry_layer - 1:shape.L - 1].max(axis=1))), sc


# ------------------------------------------------------------------ P1: full-depth limit
def test_tau_inf_equals_plain_decoder(tiny):
    shape, bb, rv = tiny
    prompt, steps = _tokens(shape, 12), _tokens(shape, 6, 1)
    a = orc.Oracle(shape, bb, rv, 2, 32)
    b = orc.Oracle(shape, bb, rv, 2, 32)
    for tk in prompt:
        a.decode_step([1], [tk], INF)
        b.plain_step([1], [tk])
    for tk in steps:
        ra = a.decode_step([1], [tk], INF)
        lb, nb = b.plain_step([1], [tk])
        assert np.array_equal(ra["logits"][0], lb[0])
        assert ra["next_tok"][0] == nb[0] and ra["exit_layer"][0] == shape.L
    for l in range(shape.L):
        ka, va = a.read_kv(1, l, 0, 18)
        kb, vb = b.read_kv(1, l, 0, 18)
        assert np.array_equal(ka, kb) and np.array_equal(va, vb)


# ------------------------------------------------------------------ P2: brute force, no cache
@pytest.mark.parametrize("mode", ["natural", "scheduled"])
def test_matches_bruteforce_recompute(tiny, mode):
    shape, bb, rv = tiny
    prompt, steps = _tokens(shape, 10), _tokens(shape, 12, 1)
    if mode == "natural":
        tau, _ = _median_tau(tiny, prompt, steps)
        forced = None
    else:
        tau = INF
        forced = synth.forced_exit_schedule(7, 0, len(steps), shape.L, shape.entry_layer).numpy()
    o = orc.Oracle(shape, bb, rv, 1, 64)
    outs = _run(o, 0, prompt, steps, tau, forced, prefill_exit=2)
    e = np.array([2] * len(prompt) + [int(r["exit_layer"][0]) for r in outs])
    if mode == "natural":
        assert 0 < (e[len(prompt):] < shape.L).sum() < len(steps), "tau should split the tokens"
    toks = np.concatenate([prompt, steps])
    logits, K, V, sc = bruteforce.recompute(shape, bb, rv, toks, e)
    for t, r in enumerate(outs):
        i = len(prompt) + t
        np.testing.assert_allclose(r["logits"][0], logits[i], rtol=0, atol=2e-6)
        ran = ~np.isnan(sc[i])
        np.testing.assert_allclose(r["scores"][0][ran], sc[i][ran], rtol=0, atol=1e-6)
        assert np.isnan(r["scores"][0][~ran]).all()
    for l in range(shape.L):
        k, v = o.read_kv(0, l, 0, len(toks))
        np.testing.assert_allclose(k, K[l], rtol=0, atol=1e-6)
        np.testing.assert_allclose(v, V[l], rtol=0, atol=1e-6)


def test_bf16_cache_storage_matches_bruteforce(tiny):
    # the optional 16-bit cache storage: every key / value is rounded to bf16 (ties to even) before any use
    shape, bb, rv = tiny
    prompt, steps = _tokens(shape, 9), _tokens(shape, 7, 1)
    forced = synth.forced_exit_schedule(5, 0, len(steps), shape.L, shape.entry_layer).numpy()
    o = orc.Oracle(shape, bb, rv, 1, 32, kv_store=1)
    outs = _run(o, 0, prompt, steps, INF, forced, prefill_exit=3)
    e = np.array([3] * len(prompt) + [int(r["exit_layer"][0]) for r in outs])
    toks = np.concatenate([prompt, steps])
    logits, K, V, _ = bruteforce.recompute(shape, bb, rv, toks, e, kv_bf16=True)
    for t, r in enumerate(outs):
        np.testing.assert_allclose(r["logits"][0], logits[len(prompt) + t], rtol=0, atol=1e-4)
    mism = 0
    for l in range(shape.L):
        k, v = o.read_kv(0, l, 0, len(toks))
        for got, want in ((k, K[l]), (v, V[l])):
            assert np.array_equal(got, torch.from_numpy(got).to(torch.bfloat16).float().numpy())  # bf16 values
            mism += int((got != want).sum())
            assert np.abs(got - want).max() <= 2.0 ** -7 * np.abs(want).max()  # at most one bf16 step apart
    assert mism <= 0.001 * 2 * shape.L * K[0].size  # rounding ties may fall either way, rarely
    plain = orc.Oracle(shape, bb, rv, 1, 32)
    ref = _run(plain, 0, prompt, steps, INF, forced, prefill_exit=3)
    assert not np.array_equal(ref[-1]["logits"], outs[-1]["logits"])


# ------------------------------------------------------------------ P3: identity river
def test_identity_river_makes_exits_invisible():
    shape = synth.SHAPES["tiny"]
    bb = synth.make_backbone(shape, "cpu")
    rv = []
    for lay in bb["layers"]:
        r = {}
        for n in synth.MATS:
            snapped, codes, scale, zero = rtn_w4.snap_to_grid(lay[n], shape.group)
            assert np.array_equal(dequant_np(codes, scale, zero, shape.group), f64(snapped))
            lay[n] = snapped
            r[n] = (codes, scale, zero)
        rv.append(r)
    prompt, steps = _tokens(shape, 8), _tokens(shape, 8, 1)
    ref = _run(orc.Oracle(shape, bb, rv, 1, 32), 0, prompt, steps, INF)
    forced = synth.forced_exit_schedule(11, 0, len(steps), shape.L, shape.entry_layer).numpy()
    assert (forced < shape.L).any()
    got = _run(orc.Oracle(shape, bb, rv, 1, 32), 0, prompt, steps, INF, forced, prefill_exit=1)
    for a, b in zip(ref, got):
        np.testing.assert_allclose(a["logits"], b["logits"], rtol=0, atol=2e-6)


# ------------------------------------------------------------------ P4: cache completeness
def test_cache_complete_after_any_exit_pattern(tiny):
    shape, bb, rv = tiny
    o = orc.Oracle(shape, bb, rv, 3, 40)
    lens = {0: 5, 2: 9}
    for slot, n in lens.items():
        o.prefill(slot, _tokens(shape, n, slot), exit_layer=1 + slot)
    for t in range(7):
        fe = synth.forced_exit_schedule(3, t, 2, shape.L, shape.entry_layer).numpy()
        o.decode_step([0, 2], _tokens(shape, 2, 50 + t), INF, fe)
    for slot in range(3):
        n = o.seq_len(slot)
        assert n == (lens.get(slot, 0) + (7 if slot in lens else 0))
        for l in range(shape.L):
            cnt = [o.write_count(slot, l, p) for p in range(40)]
            assert cnt == [1] * n + [0] * (40 - n)


# ------------------------------------------------------------------ P5: monotone in tau
def test_exit_layer_monotone_in_tau(tiny):
    shape, bb, rv = tiny
    prompt = _tokens(shape, 16)
    tk = _tokens(shape, 1, 9)
    taus = [0.0, 0.3, 0.6, 0.8, 0.9, 0.95, 0.98, 0.995, 1.0]
    els = []
    for tau in taus:
        o = orc.Oracle(shape, bb, rv, 1, 32)
        o.prefill(0, prompt)
        els.append(int(o.decode_step([0], tk, tau)["exit_layer"][0]))
    assert els == sorted(els)
    assert els[0] == shape.entry_layer and els[-1] == shape.L


# ------------------------------------------------------------------ P6: Eq. 1 closed forms
def test_similarity_closed_forms():
    lib = orc.lib()
    rng = np.random.default_rng(0)
    d = 256
    h = rng.standard_normal(d).astype(np.float32)
    delta = rng.standard_normal(d).astype(np.float32)
    delta -= (delta @ h) / (h @ h) * h  # orthogonal to h
    h2 = (h + delta).astype(np.float32)
    sim = lambda a, b: lib.orc_similarity(a.ctypes.data, b.ctypes.data, d)
    want = np.linalg.norm(h.astype(np.float64)) / math.sqrt(
        np.linalg.norm(h.astype(np.float64)) ** 2 + np.linalg.norm(delta.astype(np.float64)) ** 2)
    assert abs(sim(h, h2) - want) < 1e-6
    assert sim(h, h) == 1.0
    assert abs(sim(h, (-h).astype(np.float32)) + 1.0) < 1e-7
    assert abs(sim((3.0 * h).astype(np.float32), (0.25 * h2).astype(np.float32)) - sim(h, h2)) < 1e-6
    assert sim(h, h2) == sim(h2, h)
    e0 = np.zeros(d, np.float32); e0[0] = 1
    e1 = np.zeros(d, np.float32); e1[1] = 2
    assert sim(e0, e1) == 0.0
    assert sim(np.zeros(d, np.float32), h) == 0.0  # zero norm -> 0, never NaN


def test_dead_block_scores_one_and_exits_at_entry_layer():
    shape = synth.SHAPES["tiny"]
    bb = synth.make_backbone(shape, "cpu")
    for l in (1, 2):  # blocks 2 and 3 write nothing to the residual stream
        bb["layers"][l]["wo"] = torch.zeros_like(bb["layers"][l]["wo"])
        bb["layers"][l]["wd"] = torch.zeros_like(bb["layers"][l]["wd"])
    rv = rtn_w4.make_river(bb, shape.group)
    for entry, want in ((1, 2), (2, 2), (3, 3)):
        o = orc.Oracle(shape, bb, rv, 1, 16, entry_layer=entry)
        o.prefill(0, _tokens(shape, 4))
        r = o.decode_step([0], _tokens(shape, 1, 3), 0.9999)
        assert r["scores"][0][1] == 1.0
        assert r["exit_layer"][0] == want
    # strict '>' : tau = 1 never exits even when s == 1
    o = orc.Oracle(shape, bb, rv, 1, 16)
    o.prefill(0, _tokens(shape, 4))
    assert o.decode_step([0], _tokens(shape, 1, 3), 1.0)["exit_layer"][0] == shape.L


# ------------------------------------------------------------------ P7: attention special cases
def test_attention_special_cases(tiny):
    shape, bb, rv = tiny
    Hq, Hkv, dh = shape.Hq, shape.Hkv, shape.dh
    o = orc.Oracle(shape, bb, rv, 2, 16)
    rng = np.random.default_rng(1)
    q = rng.standard_normal((Hq, dh)).astype(np.float32)
    k = rng.standard_normal((9, Hkv * dh)).astype(np.float32)
    v = rng.standard_normal((9, Hkv * dh)).astype(np.float32)
    o.write_kv(1, 2, 0, k, v)
    grp = Hq // Hkv
    # one cached position -> the value itself
    out = o.attention(2, 1, 0, q)
    for i in range(Hq):
        j = i // grp
        np.testing.assert_allclose(out[i], v[0, j * dh:(j + 1) * dh], atol=1e-7)
    # textbook dense softmax over positions 0..pos, GQA mapping i -> i // grp, causal cut at pos
    for pos in (3, 8):
        out = o.attention(2, 1, pos, q)
        for i in range(Hq):
            j = i // grp
            kk = k[:pos + 1, j * dh:(j + 1) * dh].astype(np.float64)
            vv = v[:pos + 1, j * dh:(j + 1) * dh].astype(np.float64)
            s = kk @ q[i].astype(np.float64) / math.sqrt(dh)
            p = np.exp(s - s.max()); p /= p.sum()
            np.testing.assert_allclose(out[i], p @ vv, atol=1e-6)
    # all keys equal -> plain mean of the values
    o.write_kv(0, 1, 0, np.repeat(k[:1], 6, axis=0), v[:6])
    out = o.attention(1, 0, 5, q)
    for i in range(Hq):
        j = i // grp
        np.testing.assert_allclose(out[i], v[:6, j * dh:(j + 1) * dh].mean(axis=0), atol=1e-6)


# ------------------------------------------------------------------ P8: RoPE
def test_rope_properties():
    lib = orc.lib()
    rng = np.random.default_rng(2)
    dh, theta = 64, 10000.0

    def rot(v, pos):
        w = v.astype(np.float32).copy()
        lib.orc_rope(w.ctypes.data, dh, pos, theta)
        return w

    q = rng.standard_normal(dh).astype(np.float32)
    k = rng.standard_normal(dh).astype(np.float32)
    assert np.array_equal(rot(q, 0), q)
    assert abs(np.linalg.norm(rot(q, 37)) - np.linalg.norm(q)) < 1e-5
    a = rot(q, 40).astype(np.float64) @ rot(k, 33).astype(np.float64)
    b = rot(q, 107).astype(np.float64) @ rot(k, 100).astype(np.float64)
    c = rot(q, 7).astype(np.float64) @ rot(k, 0).astype(np.float64)
    assert abs(a - b) < 1e-4 and abs(a - c) < 1e-4
    # pair (i, i + dh/2) turns by pos * theta^(-2i/dh): check one pair against the 2-D rotation
    i, pos = 5, 11
    ang = pos * theta ** (-2.0 * i / dh)
    w = rot(q, pos)
    assert abs(w[i] - (q[i] * math.cos(ang) - q[i + 32] * math.sin(ang))) < 1e-6
    assert abs(w[i + 32] - (q[i + 32] * math.cos(ang) + q[i] * math.sin(ang))) < 1e-6
    # the last pair turns slowest; pair 0 turns by exactly pos radians
    w1 = rot(np.eye(dh, dtype=np.float32)[0], 1)
    assert abs(w1[0] - math.cos(1.0)) < 1e-7 and abs(w1[32] - math.sin(1.0)) < 1e-7


# ------------------------------------------------------------------ P9: cache size (memory table, KV column)
def test_kv_cache_size_matches_paper_table():
    golden = os.path.join(os.path.dirname(__file__), "golden", "kv_cache_mb_llama31_8b.txt")
    rows = [ln.split() for ln in open(golden) if ln.strip() and not ln.startswith("#")]
    cfg = orc.make_config(synth.SHAPES["8b"], 1, 1)
    for ctx, mb in rows:
        assert orc.lib().orc_kv_bytes_16bit(cfg, int(ctx)) == int(mb) * 2 ** 20


# ------------------------------------------------------------------ P10: the 4-bit grid
def test_quant_grid_bounds_and_roundtrip():
    w = synth.normal(9, 1, (48, 256), 0.02)
    codes, s, z = rtn_w4.quantize_w4(w, 64)
    assert codes.dtype == torch.uint8 and tuple(codes.shape) == (48, 128)
    out = np.empty((48, 256), np.float32)
    orc.lib().orc_dequant_w4(codes.data_ptr(), s.data_ptr(), z.data_ptr(), 64, 48, 256, out.ctypes.data)
    np.testing.assert_array_equal(out.astype(np.float64), dequant_np(codes, s, z, 64).astype(np.float32))
    step = np.repeat(f64(s), 64, axis=1)
    # in-range weights sit within half a step (+ the bf16 rounding of scale and zero) of the grid
    assert (np.abs(out - f64(w)) <= 0.5 * step * 1.1 + 1e-9).mean() > 0.999
    assert np.abs(out - f64(w)).max() <= 1.01 * step.max()
    # a constant group comes back exactly
    c = torch.full((2, 64), 0.0123, dtype=torch.bfloat16)
    cc, cs, cz = rtn_w4.quantize_w4(c, 64)
    np.testing.assert_array_equal(dequant_np(cc, cs, cz, 64), f64(c))
    # nibble order: low nibble = even input index
    one = torch.zeros((1, 64), dtype=torch.bfloat16); one[0, 1] = 1.0
    oc, os_, oz = rtn_w4.quantize_w4(one, 64)
    assert oc[0, 0].item() >> 4 == 15 and oc[0, 0].item() & 15 == 0


def test_matvec_matches_library_matmul():
    lib = orc.lib()
    w = synth.normal(4, 1, (40, 192), 0.05)
    x = np.random.default_rng(3).standard_normal(192).astype(np.float32)
    y = np.empty(40, np.float32)
    lib.orc_matvec_bf16(w.data_ptr(), 40, 192, x.ctypes.data, y.ctypes.data)
    np.testing.assert_allclose(y, f64(w) @ x.astype(np.float64), atol=1e-6)
    codes, s, z = rtn_w4.quantize_w4(w, 64)
    lib.orc_matvec_w4(codes.data_ptr(), s.data_ptr(), z.data_ptr(), 64, 40, 192, x.ctypes.data, y.ctypes.data)
    np.testing.assert_allclose(y, dequant_np(codes, s, z, 64) @ x.astype(np.float64), atol=1e-6)


def test_rmsnorm_closed_form():
    lib = orc.lib()
    d = 128
    g = torch.full((d,), 0.5, dtype=torch.bfloat16)
    h = np.full(d, 3.0, np.float32)
    x = np.empty(d, np.float32)
    lib.orc_rmsnorm(h.ctypes.data, g.data_ptr(), d, 0.0, x.ctypes.data)
    np.testing.assert_allclose(x, 0.5, atol=1e-7)  # constant vector -> gain
    h = np.zeros(d, np.float32); h[3] = 4.0
    lib.orc_rmsnorm(h.ctypes.data, g.data_ptr(), d, 1e-5, x.ctypes.data)
    assert abs(x[3] - 0.5 * 4.0 / math.sqrt(16.0 / d + 1e-5)) < 1e-6 and x[0] == 0.0


# ------------------------------------------------------------------ P11: compaction lists
def test_row_lists_are_a_stable_partition(tiny):
    shape, bb, rv = tiny
    B = 6
    o = orc.Oracle(shape, bb, rv, B, 24)
    for b in range(B):
        o.prefill(b, _tokens(shape, 3 + b, b))
    fe = np.array([4, 1, 3, 1, 2, 4], np.int32)
    r = o.decode_step(list(range(B)), _tokens(shape, B, 77), INF, fe)
    assert np.array_equal(r["exit_layer"], fe)
    act, na, riv, nr = o.last_lists(B)
    for l in range(1, shape.L + 2):  # lists entering block l; l = L+1: at the LM head (L = never left)
        want_a = [b for b in range(B) if fe[b] >= min(l, shape.L)]
        want_r = [b for b in range(B) if fe[b] < min(l, shape.L)]
        assert list(act[l - 1][:na[l - 1]]) == want_a and list(riv[l - 1][:nr[l - 1]]) == want_r
        assert na[l - 1] + nr[l - 1] == B


# ------------------------------------------------------------------ P12: full-quantisation limit
def test_full_quant_limit_equals_plain_river_decoder(tiny):
    shape, bb, rv = tiny
    a = orc.Oracle(shape, bb, rv, 1, 16, entry_layer=0)
    b = orc.Oracle(shape, bb, rv, 1, 16, entry_layer=0)
    for tk in _tokens(shape, 6):
        ra = a.decode_step([0], [tk], INF, [0])
        lb, nb = b.plain_step([0], [tk], use_river=True)
        assert np.array_equal(ra["logits"][0], lb[0]) and ra["exit_layer"][0] == 0
    # and it differs from the backbone (the river is a real approximation), yet stays close
    c = orc.Oracle(shape, bb, rv, 1, 16)
    for tk in _tokens(shape, 6):
        lc, _ = c.plain_step([0], [tk])
    assert not np.array_equal(lc, lb) and cosine(lc, lb) > 0.9


# ------------------------------------------------------------------ batching and modes
def test_rows_are_independent_and_batch_min_mode(tiny):
    shape, bb, rv = tiny
    prompts = [_tokens(shape, 5 + 2 * b, b) for b in range(3)]
    tk = _tokens(shape, 3, 20)
    tau, _ = _median_tau(tiny, _tokens(shape, 10), _tokens(shape, 12, 1))
    together = orc.Oracle(shape, bb, rv, 3, 32)
    for b in range(3):
        together.prefill(b, prompts[b])
    rt = together.decode_step([2, 0, 1], tk, tau)
    for i, b in enumerate([2, 0, 1]):
        solo = orc.Oracle(shape, bb, rv, 3, 32)
        solo.prefill(b, prompts[b])
        rs = solo.decode_step([b], [tk[i]], tau)
        assert np.array_equal(rs["logits"][0], rt["logits"][i]) and rs["exit_layer"][0] == rt["exit_layer"][i]
    # Eq. 1 literal: the batch switches together at the first layer where every row passes
    sc = rt["scores"]
    bm = orc.Oracle(shape, bb, rv, 3, 32, exit_mode=1)
    for b in range(3):
        bm.prefill(b, prompts[b])
    full = orc.Oracle(shape, bb, rv, 3, 32)
    for b in range(3):
        full.prefill(b, prompts[b])
    sc_full = full.decode_step([2, 0, 1], tk, INF)["scores"]
    rb = bm.decode_step([2, 0, 1], tk, tau)
    want = shape.L
    for l in range(shape.entry_layer, shape.L):
        if (sc_full[:, l - 1] > tau).all():
            want = l
            break
    assert (rb["exit_layer"] == want).all()


def test_argmax_ties_and_bad_arguments(tiny):
    shape, bb, rv = tiny
    o = orc.Oracle(shape, bb, rv, 2, 4)
    with pytest.raises(ValueError):
        o.decode_step([0, 0], [1, 2], INF)  # a sequence twice in one step
    with pytest.raises(ValueError):
        o.decode_step([0], [shape.V], INF)
    with pytest.raises(ValueError):
        o.decode_step([0], [1], INF, [0])  # river from block 1 needs entry_layer 0
    for tk in (1, 2, 3, 4):
        o.decode_step([0], [tk], INF)
    with pytest.raises(ValueError):
        o.decode_step([0], [5], INF)  # sequence full
    r = o.decode_step([1], [7], INF)
    assert r["next_tok"][0] == int(np.argmax(r["logits"][0]))


# ------------------------------------------------------------------ prefill at the depth the exit rule picks
def test_prefill_auto_depth_matches_bruteforce_rule(tiny):
    # Section 4.2, "Prefill Phase": one depth for the whole prompt.  The depth the oracle picks is checked against the
    # rule applied to an independent no-cache recompute of the full-depth scores (every position of the prompt must
    # pass s > tau at that block and at least one position must fail at every earlier eligible block), and the cache
    # and logits it leaves behind against a recompute with every token leaving at that depth.
    shape, bb, rv = tiny
    prompt = _tokens(shape, 14, 7)
    _, _, _, sc_full = bruteforce.recompute(shape, bb, rv, prompt, [shape.L] * len(prompt))
    lo = max(shape.entry_layer, 1)
    col_min = sc_full[:, lo - 1:shape.L - 1].min(axis=0)  # min over positions, per eligible block
    seen = set()
    taus = [-1.0] + [float(m) - 1e-4 for m in col_min] + [float(m) + 1e-4 for m in col_min] + [2.0]
    for tau in taus:
        if np.abs(col_min - tau).min() < 5e-5:
            continue
        want = shape.L
        for l in range(lo, shape.L):
            if col_min[l - lo] > tau:
                want = l
                break
        o = orc.Oracle(shape, bb, rv, 1, 32)
        logits, nxt, depth = o.prefill_auto(0, prompt, tau)
        assert depth == want, (tau, depth, want, col_min)
        seen.add(depth)
        lg, K, V, _ = bruteforce.recompute(shape, bb, rv, prompt, [depth] * len(prompt))
        assert np.abs(logits - lg[-1]).max() < 2e-4
        for l in range(shape.L):
            k, v = o.read_kv(0, l, 0, len(prompt))
            assert np.abs(k - K[l]).max() < 1e-4 and np.abs(v - V[l]).max() < 1e-4
            for pos in range(len(prompt)):
                assert o.write_count(0, l, pos) == 1  # the second pass leaves every slot written exactly once
        assert o.seq_len(0) == len(prompt)
        o.close()
    assert lo in seen and shape.L in seen and len(seen) >= 3


def test_prefill_auto_limits(tiny):
    shape, bb, rv = tiny
    prompt = _tokens(shape, 9, 3)
    a = orc.Oracle(shape, bb, rv, 1, 16)
    b = orc.Oracle(shape, bb, rv, 1, 16)
    la, na, depth = a.prefill_auto(0, prompt, INF)       # nothing passes: the whole backbone
    lb, nb = b.prefill(0, prompt, shape.L)
    assert depth == shape.L and np.array_equal(la, lb) and na == nb
    a.release(0), b.release(0)
    la, na, depth = a.prefill_auto(0, prompt, -2.0)      # everything passes: the entry layer
    lb, nb = b.prefill(0, prompt, max(shape.entry_layer, 1))
    assert depth == max(shape.entry_layer, 1) and np.array_equal(la, lb) and na == nb


# ------------------------------------------------------------------ the other KV strategies (Section 3)
def test_state_propagation_matches_whole_sequence_recompute(tiny):
    # kv_strategy = 1: a skipped block's K/V come from the hidden state at the exit through the backbone's K / V
    # projections; checked against the cache-free numpy recompute (logits, every K / V entry, scores)
    shape, bb, rv = tiny
    toks = _tokens(shape, 11, 7)
    rng = np.random.default_rng(3)
    e = rng.integers(max(shape.entry_layer, 1), shape.L + 1, len(toks))
    o = orc.Oracle(shape, bb, rv, 1, 16, kv_strategy=1)
    lg = []
    for t, tk in enumerate(toks):
        r = o.decode_step([0], [tk], INF, [int(e[t])])
        assert r["exit_layer"][0] == e[t]
        lg.append(r["logits"][0])
    logits, K, V, sc = bruteforce.recompute(shape, bb, rv, toks, e, strategy=1)
    assert np.abs(np.stack(lg) - logits).max() < 2e-4
    for l in range(shape.L):
        k, v = o.read_kv(0, l, 0, len(toks))
        assert np.abs(k - K[l]).max() < 2e-4 and np.abs(v - V[l]).max() < 2e-4
        assert all(o.write_count(0, l, p) == 1 for p in range(len(toks)))  # every (token, layer) slot written once
    # and it is NOT the river: with some early exits the logits differ from strategy 0 on the same path
    o0 = orc.Oracle(shape, bb, rv, 1, 16)
    d = max(np.abs(o0.decode_step([0], [tk], INF, [int(e[t])])["logits"][0] - lg[t]).max() for t, tk in enumerate(toks))
    assert (e < shape.L).any() and d > 1e-3
    o.close(); o0.close()


def test_mono_decreasing_exit_caps_depth_and_writes_no_skipped_slot(tiny):
    # kv_strategy = 2: a token leaves no later than the previous token of its sequence did (whatever its score or
    # the forced schedule says), skipped blocks write nothing, and the result equals the cache-free recompute
    shape, bb, rv = tiny
    L = shape.L
    toks = _tokens(shape, 9, 8)
    wish = [L, L, 3, L, 2, 3, 2, 1, L]  # requested exit layers; the cap makes them non-increasing
    want, cap = [], L
    for w in wish:
        cap = min(cap, w)
        want.append(cap)
    o = orc.Oracle(shape, bb, rv, 2, 16, entry_layer=1, kv_strategy=2)
    lg, got = [], []
    for t, tk in enumerate(toks):
        r = o.decode_step([1], [tk], INF, [wish[t]])
        got.append(int(r["exit_layer"][0]))
        lg.append(r["logits"][0])
    assert got == want
    logits, K, V, _ = bruteforce.recompute(shape, bb, rv, toks, want, strategy=2)
    assert np.abs(np.stack(lg) - logits).max() < 2e-4
    for l in range(L):
        k, v = o.read_kv(1, l, 0, len(toks))
        for p in range(len(toks)):
            ran = want[p] >= l + 1
            assert o.write_count(1, l, p) == (1 if ran else 0)
            if ran:
                assert np.abs(k[p] - K[l][p]).max() < 2e-4 and np.abs(v[p] - V[l][p]).max() < 2e-4
    # a second sequence starts with a fresh cap; releasing a slot resets it
    r = o.decode_step([0], [toks[0]], INF)
    assert r["exit_layer"][0] == L
    o.release(1)
    assert o.decode_step([1], [toks[0]], INF)["exit_layer"][0] == L
    o.close()


def test_kv_mask_hides_positions_without_cache_entries(tiny):
    # kv_strategy = 3: exit layers vary freely, skipped blocks write nothing, and attention in block l runs over the
    # positions whose token ran block l (plus the row itself): equal to the cache-free recompute with that mask
    shape, bb, rv = tiny
    L = shape.L
    toks = _tokens(shape, 12, 9)
    rng = np.random.default_rng(5)
    e = rng.integers(1, L + 1, len(toks))
    e[0], e[3] = 1, L  # an early position that most later blocks cannot see, and one that every block sees
    o = orc.Oracle(shape, bb, rv, 1, 16, entry_layer=1, kv_strategy=3)
    lg = []
    for t, tk in enumerate(toks):
        r = o.decode_step([0], [tk], INF, [int(e[t])])
        assert r["exit_layer"][0] == e[t]
        lg.append(r["logits"][0])
    logits, K, V, _ = bruteforce.recompute(shape, bb, rv, toks, e, strategy=3)
    assert np.abs(np.stack(lg) - logits).max() < 2e-4
    for l in range(L):
        k, v = o.read_kv(0, l, 0, len(toks))
        for p in range(len(toks)):
            if e[p] >= l + 1:
                assert np.abs(k[p] - K[l][p]).max() < 2e-4 and np.abs(v[p] - V[l][p]).max() < 2e-4
    # the mask matters: the same path with every position visible (river weights aside, strategy 2 semantics are
    # undefined here) gives other logits - compare with a recompute that ignores the mask
    unmasked, _, _, _ = bruteforce.recompute(shape, bb, rv, toks, np.full(len(toks), L))
    assert np.abs(logits[-1] - unmasked[-1]).max() > 1e-3
    o.close()

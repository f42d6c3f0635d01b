"""Parity of the CUDA decode path with the CPU oracle, element by element, through the C ABI (needs a B200).

Passes:
  * scheduled: per-row, per-step thresholds placed by the oracle so that no evaluated score is within 1.25e-3 of
    its threshold; the GPU decides freely and exit layers, row lists and cache contents must match exactly /
    within tolerance at every step.
  * natural: one threshold for the run (about half of the tokens leave early); GPU decisions are compared with
    the oracle's, a mismatch is allowed only when an oracle score lies within 1e-3 of the threshold (counted).
  * forced: the oracle's exit layers are imposed on the GPU; logits and K/V are compared with no decision flips.
Tolerances: logits max-abs 2e-2 and cosine >= 0.999 against the fp32 oracle; cached K/V |a-b| <= 1e-2|b| + 1e-2 rms(b).
"""
import numpy as np
import pytest
import torch

from tests.gpu_harness import INF, NEAR, Pair, draw_model, natural_tau
from workloads import synth

pytestmark = pytest.mark.gpu

_models = {}


def model(name, n_layers=None, identity=False):
    key = (name, n_layers, identity)
    if key not in _models:
        if name in ("1b", "8b"):
            _models.clear()  # one big model at a time
            torch.cuda.empty_cache()
        _models[key] = draw_model(name, n_layers, identity)
    return _models[key]


@pytest.fixture(autouse=True, params=[0, 8], ids=["stage-kernels", "chain-kernel"])
def launch_plan(request):
    """Every test runs twice: steps of 1-4 rows as one kernel per stage (default), and through the persistent chain
    kernel (flag 8).  Steps of five or more rows take the same tensor-core kernels either way."""
    import tests.gpu_harness as gh
    gh.EXTRA_FLAGS = request.param
    yield
    gh.EXTRA_FLAGS = 0


def toks(shape, n, stream):
    return synth.tokens(shape.seed, stream, n, shape.V).numpy()


def run_scheduled(m, prompt_lens, n_steps, kind="uniform", prefill_exit=None, page_seed=0, max_batch=None,
                  seed=21, kv_store=0, flags=0):
    shape = m[0]
    B = len(prompt_lens)
    L = len(m[1][0]["layers"])
    p = Pair(m, B, max(prompt_lens) + n_steps + 1, max_batch or max(B, 8), page_shuffle_seed=page_seed,
             kv_store=kv_store, flags=flags)
    prompts = [toks(shape, n, 100 + b) for b, n in enumerate(prompt_lens)]
    slots = list(range(B))
    p.prefill(slots, prompts, prefill_exit)
    worst_logit, n_early = 0.0, 0
    for t in range(n_steps):
        tk = toks(shape, B, 200 + t)
        order = synth.shuffled(seed, t, B)  # rows in a different slot order every step
        sl = [slots[i] for i in order]
        targets = synth.forced_exit_schedule(seed, t, B, L, shape.entry_layer, kind).numpy()
        tau, o = p.oracle_scheduled_step(sl, tk, targets)
        g = p.gpu_step(sl, tk, tau)
        assert np.array_equal(g.exit_layer, o.exit_layer), f"step {t}: exit layers {g.exit_layer} vs {o.exit_layer}"
        p.compare_lists(B)
        worst_logit = max(worst_logit, p.compare_logits(g.logits, o.logits, f"step {t}"))
        ran = ~np.isnan(o.scores)
        assert np.array_equal(ran, ~np.isnan(g.scores))
        assert np.abs(g.scores[ran] - o.scores[ran]).max() < NEAR
        top2 = np.sort(o.logits, axis=1)[:, -2:]
        clear = (top2[:, 1] - top2[:, 0]) > 2 * 2e-2
        assert np.array_equal(g.next_tok[clear], o.next_tok[clear])
        n_early += int((o.exit_layer < L).sum())
    worst_kv = max(p.compare_kv(s, p.oracle.seq_len(s)) for s in slots)
    for s in slots:
        assert p.gpu.seq_len(s) == p.oracle.seq_len(s)
    st = p.gpu.stats()
    assert st.device_error == 0
    p.close()
    return dict(worst_logit=worst_logit, worst_kv=worst_kv, n_early=n_early, total=B * n_steps)


# ------------------------------------------------------------------ config 1: tiny decoder, B=1, 32 + 16
def test_tiny_config1_natural_and_forced():
    m = model("tiny")
    shape = m[0]
    prompt, steps = toks(shape, 32, 0), toks(shape, 16, 1)
    tau = natural_tau(m, [prompt], steps[:, None], 0.5)
    # free pass
    p = Pair(m, 1, 64, 4)
    p.prefill([0], [prompt])
    exits, n_near, n_cmp = [], 0, 0
    for t in range(16):
        o = p.oracle_step([0], [steps[t]], tau)
        g = p.gpu_step([0], [steps[t]], tau)
        exits.append(int(o.exit_layer[0]))
        n_cmp += 1
        if g.exit_layer[0] != o.exit_layer[0]:
            assert p.near_threshold(o.scores[0], tau, max(g.exit_layer[0], o.exit_layer[0])), \
                f"step {t}: exit {g.exit_layer[0]} vs {o.exit_layer[0]} with no score near tau"
            n_near += 1
            break  # histories differ from here on
        p.compare_logits(g.logits, o.logits, f"free step {t}")
    frac = np.mean(np.array(exits) < shape.L)
    print(f"config1: tau={tau:.4f} early-exit fraction {frac:.2f}, near-threshold flips {n_near}/{n_cmp}")
    p.close()
    # forced pass: the oracle decides, the GPU follows
    p = Pair(m, 1, 64, 4)
    p.prefill([0], [prompt])
    early = 0
    for t in range(16):
        o = p.oracle_step([0], [steps[t]], tau)
        g = p.gpu_step([0], [steps[t]], INF, o.exit_layer)
        assert np.array_equal(g.exit_layer, o.exit_layer)
        p.compare_logits(g.logits, o.logits, f"forced step {t}")
        early += int(o.exit_layer[0] < shape.L)
    assert 4 <= early <= 12, "threshold should make about half of the tokens leave early"
    p.compare_kv(0, 48)
    p.close()


def test_tiny_scheduled_ragged_batch_shuffled_pages():
    r = run_scheduled(model("tiny"), [3, 17, 40, 16, 1, 33], 20, "uniform", prefill_exit=2, page_seed=1234)
    assert r["n_early"] > r["total"] // 3
    print(r)


def test_tiny_geometric_exits_and_wide_batch():
    # more rows than one projection pass takes (8), mostly early exits (mean exit layer about 2 of 4)
    r = run_scheduled(model("tiny"), [5 + (7 * b) % 23 for b in range(19)], 6, "geometric", max_batch=32)
    assert r["n_early"] > r["total"] // 2


@pytest.mark.parametrize("flags", [0, 1, 2, 4, 5, 8, 9, 12, 32, 33, 64, 97])
def test_launch_modes_agree_with_oracle(flags):
    # 1: CUDA-graph replay; 2: no tensor-core projections; 4: plain attention kernel; 8: the persistent chain kernel
    # (three rows per step: the chain kernel takes them when 8 is set, by the parameter or by the fixture);
    # 32: the TMA-fed attention kernel for small steps too (default there: the kernel that fetches the cache early);
    # 64: exit score / decision / compaction by the last CTA of the down projection instead of a kernel of its own
    r = run_scheduled(model("mini8"), [37, 16, 3], 6, "uniform", page_seed=11, flags=flags, max_batch=4)
    assert r["n_early"] > 0


@pytest.mark.parametrize("flags", [0, 16, 2])
def test_mini8_head_dim_128_gqa4(flags):
    # five rows: backbone rows on the tcgen05 GEMM; exit-layer rows on the dequantising tcgen05 GEMM (0), on the
    # CUDA-core kernel (16), everything on CUDA cores (2)
    r = run_scheduled(model("mini8"), [70, 16, 31, 48, 5], 18, "uniform", prefill_exit=3, page_seed=7, flags=flags)
    assert r["n_early"] > 0
    print(r)


@pytest.mark.parametrize("rows", [70, 150])
def test_mini8_wide_batches_other_gemm_geometries(rows):
    # 70 rows: operand tiles of 80 rows, three CTAs per SM; 150 rows: 160-row operand tiles, one CTA per SM with deep
    # stages; both weight sets live in most layers, lengths mixed so that the attention splits differ per row.  The
    # oracle stores its cache in bf16 here as the large-shape tests do: over millions of cache entries the tail of the
    # fp32-cache deviation (Section 4.1's shared slots hold bf16) reaches the K/V tolerance without any kernel error.
    r = run_scheduled(model("mini8"), [3 + (11 * b) % 29 for b in range(rows)], 3, "uniform", page_seed=rows, max_batch=rows,
                      kv_store=1)
    assert r["n_early"] > 0


@pytest.mark.parametrize("lens,flags", [([2200, 130, 700, 1, 1500, 300], 0), ([2500, 40], 32), ([1900], 0)])
def test_mini8_long_ragged_contexts_split_kv(lens, flags):
    # contexts of hundreds to thousands of positions, mixed in one batch: the KV range of a (row, KV head) is cut into
    # several splits that meet through the partial buffers and the ticket (six rows: the TMA-fed kernel with the split
    # count of the host's cost model; flag 32: the same kernel for a two-row step; one row: the small-step kernel with
    # 30 splits), next to rows with a single, partly filled tile.  Stands in for the exit-aware attention microbenchmark:
    # scheduled exits differ per row, exit-layer K/V go to the same slots, and the whole cache is compared.
    r = run_scheduled(model("mini8"), lens, 3, "uniform", page_seed=len(lens), flags=flags, max_batch=8, kv_store=1)
    assert r["n_early"] > 0


# ------------------------------------------------------------------ invariants on the GPU
def test_identity_river_makes_exits_invisible_on_gpu():
    m = model("tiny", identity=True)
    shape = m[0]
    prompt, steps = toks(shape, 9, 0), toks(shape, 8, 1)
    outs = []
    for forced in (None, synth.forced_exit_schedule(11, 0, 8, shape.L, shape.entry_layer).numpy()):
        p = Pair(m, 1, 32, 2)
        p.prefill([0], [prompt], None if forced is None else 1)
        lg = []
        for t in range(8):
            g = p.gpu_step([0], [steps[t]], INF, None if forced is None else [forced[t]])
            lg.append(g.logits[0])
        outs.append(np.stack(lg))
        p.close()
    # same weights either way: only fp32 summation order differs between the two projection kernels
    assert np.abs(outs[0] - outs[1]).max() < 2e-4


def test_full_quant_limit_and_entry_layer_zero():
    m = model("tiny")
    shape = m[0]
    p = Pair(m, 2, 32, 2, entry_layer=0)
    p.prefill([0, 1], [toks(shape, 7, 0), toks(shape, 4, 1)], 0)
    for t in range(5):
        tk = toks(shape, 2, 30 + t)
        o = p.oracle_step([0, 1], tk, INF, [0, 0])
        g = p.gpu_step([0, 1], tk, INF, [0, 0])
        assert np.array_equal(g.exit_layer, [0, 0]) and np.array_equal(o.exit_layer, [0, 0])
        p.compare_logits(g.logits, o.logits, f"full-quant step {t}")
    p.compare_kv(0, 12)
    p.compare_kv(1, 9)
    p.close()


def test_batch_min_mode():
    m = model("tiny")
    shape = m[0]
    prompts = [toks(shape, 6 + 3 * b, b) for b in range(4)]
    p = Pair(m, 4, 32, 4, exit_mode=1)
    p.prefill([0, 1, 2, 3], prompts)
    seen = set()
    for t, tau in enumerate([0.5, 0.85, 0.93, 0.97, 0.999]):
        tk = toks(shape, 4, 40 + t)
        o = p.oracle_step([0, 1, 2, 3], tk, tau)
        g = p.gpu_step([0, 1, 2, 3], tk, tau)
        assert len(set(o.exit_layer.tolist())) == 1
        lo = max(shape.entry_layer, 1)
        near = np.abs(o.scores[:, lo - 1:shape.L - 1] - tau).min() <= NEAR
        if not near:
            assert np.array_equal(g.exit_layer, o.exit_layer)
            p.compare_logits(g.logits, o.logits, f"batch-min step {t}")
        else:
            break
        seen.add(int(o.exit_layer[0]))
    assert len(seen) >= 2
    p.close()


def test_cache_is_complete_for_every_token_and_layer():
    # NaN-filled pool: any (token, layer) slot the exit path failed to write stays NaN
    m = model("tiny")
    shape = m[0]
    p = Pair(m, 3, 48, 4, page_shuffle_seed=99)
    p.prefill([0, 2], [toks(shape, 5, 0), toks(shape, 18, 2)], 1)
    for t in range(9):
        fe = synth.forced_exit_schedule(3, t, 2, shape.L, shape.entry_layer).numpy()
        p.gpu_step([2, 0], toks(shape, 2, 50 + t), INF, fe, want_logits=False)
    for slot, n in ((0, 14), (2, 27)):
        assert p.gpu.seq_len(slot) == n
        for l in range(1, shape.L + 1):
            k, v = p.gpu.read_kv(slot, l, 0, n)
            assert torch.isfinite(k.float()).all() and torch.isfinite(v.float()).all()
    # pages of different sequences never alias: release one, the other is untouched
    k_before, _ = p.gpu.read_kv(2, 1, 0, 27)
    p.gpu.release(0)
    assert p.gpu.seq_len(0) == 0
    k_after, _ = p.gpu.read_kv(2, 1, 0, 27)
    assert torch.equal(k_before, k_after)
    p.close()


def test_kv_roundtrip_and_page_table_indices():
    m = model("tiny")
    shape = m[0]
    p = Pair(m, 2, 64, 2, page_shuffle_seed=5)
    w = shape.Hkv * shape.dh
    k = synth.normal(1, 1, (37, w), 1.0, "cuda")
    v = synth.normal(1, 2, (37, w), 1.0, "cuda")
    p.gpu.write_kv(1, 3, 0, k, v)
    assert p.gpu.seq_len(1) == 37
    for pos0, n in ((0, 37), (15, 3), (16, 16), (36, 1)):
        kk, vv = p.gpu.read_kv(1, 3, pos0, n)
        assert torch.equal(kk, k[pos0:pos0 + n]) and torch.equal(vv, v[pos0:pos0 + n])
    p.close()


def test_errors_and_limits():
    from paper_2604_18396_b200 import RiverError
    m = model("tiny")
    shape = m[0]
    p = Pair(m, 2, 32, 2)
    with pytest.raises(RiverError) as e:
        p.gpu_step([0, 0], [1, 2], INF)
    assert e.value.code == -5
    with pytest.raises(RiverError) as e:
        p.gpu_step([0, 1, 1], [1, 2, 3], INF)
    assert e.value.code == -1  # more rows than max_batch
    with pytest.raises(RiverError) as e:
        p.gpu_step([5], [1], INF)
    assert e.value.code == -5
    p.prefill([0], [toks(shape, 31, 0)])
    p.gpu_step([0], [3], INF)
    with pytest.raises(RiverError) as e:
        p.gpu_step([0], [3], INF)  # 32 positions cached: the page table is full
    assert e.value.code == -4
    with pytest.raises(RiverError):
        p.gpu.prefill([0], torch.zeros(4, dtype=torch.int32, device="cuda"), [0, 4])  # slot not empty
    p.gpu.release(0)
    p.gpu.prefill([0], torch.zeros(4, dtype=torch.int32, device="cuda"), [0, 4])
    assert p.gpu.seq_len(0) == 4
    # a bad token id is flagged by the device, not dereferenced
    p.gpu_step([1], [shape.V + 7], INF)
    assert p.gpu.stats().device_error == 2
    p.close()


def test_host_buffer_entry_point_matches_device_one():
    m = model("tiny")
    shape = m[0]
    prompts = [toks(shape, 11, 0), toks(shape, 20, 1), toks(shape, 2, 2)]
    a = Pair(m, 3, 40, 4)
    b = Pair(m, 3, 40, 4)
    a.prefill([0, 1, 2], prompts)
    b.prefill([0, 1, 2], prompts)
    for t in range(4):
        tk = toks(shape, 3, 60 + t)
        ga = a.gpu_step([0, 1, 2], tk, 0.93)
        tok_h = torch.from_numpy(tk.astype(np.int32)).pin_memory()
        tau_h = torch.full((3,), 0.93).pin_memory()
        lg = torch.empty((3, shape.V)).pin_memory()
        nx = torch.empty(3, dtype=torch.int32).pin_memory()
        el = torch.empty(3, dtype=torch.int32).pin_memory()
        sc = torch.empty((3, shape.L)).pin_memory()
        b.gpu.decode_step_host([0, 1, 2], tok_h, tau_h, None, lg, nx, el, sc)
        assert np.array_equal(el.numpy(), ga.exit_layer) and np.array_equal(nx.numpy(), ga.next_tok)
        assert np.array_equal(lg.numpy(), ga.logits)
        assert np.array_equal(np.isnan(sc.numpy()), np.isnan(ga.scores))
    a.close()
    b.close()


# ------------------------------------------------------------------ configs 2-4 (1B / 8B class), reduced runs
# At these depths and widths the 16-bit storage of the KV cache alone (everything else exact) moves the logits of
# the synthetic random-weight models by about 0.5 % / 0.9 % of their standard deviation (max-abs 2.2e-2 / 5.8e-2
# measured), i.e. past the 2e-2 bound before any kernel arithmetic enters.  The method keeps the cache in a 16-bit
# format (paper Section 4.1), so here the oracle stores its cache entries rounded to bf16 (kv_store=1) and the
# stated bounds apply; the deviation from the oracle with an fp32 cache is checked through the cosine bound and
# reported.
def test_1b_class_subbatch():
    r = run_scheduled(model("1b"), [40, 23], 5, "uniform", max_batch=8, kv_store=1)
    print("1b:", r)


def test_8b_class_reduced_run():
    r = run_scheduled(model("8b"), [12], 4, "uniform", max_batch=1, kv_store=1)
    print("8b:", r)


def test_8b_class_batch_rows_on_both_paths():
    # several rows with different exit layers: backbone and exit-layer weights both live in most layers
    r = run_scheduled(model("8b"), [9, 20, 5], 3, "uniform", max_batch=4, kv_store=1, page_seed=3)
    assert r["n_early"] > 0
    print("8b batch:", r)


def test_8b_class_six_rows_tensor_core_paths():
    # from five rows on: backbone rows on the tcgen05 GEMM, exit-layer rows on the dequantising tcgen05 GEMM, at the
    # full 8B layer shape (cluster K-splits of every projection, 128-head-dim cache writes from the GEMM epilogue)
    r = run_scheduled(model("8b"), [6, 11, 3, 9, 4, 7], 2, "uniform", max_batch=8, kv_store=1, page_seed=5)
    assert r["n_early"] > 0
    print("8b six rows:", r)


@pytest.mark.parametrize("lens,flags", [([1024], 1), ([1024, 300, 2050, 17, 640, 1500], 1)])
def test_8b_class_full_size_step_on_synthetic_history(lens, flags):
    # The benchmark's own configuration - all 32 layers of the 8B shape, context ~1024, CUDA-graph replay - checked
    # output by output: an oracle prefill of such prompts would take minutes, so both caches are filled with the same
    # N(0,1) bf16 history through the write hook, then three scheduled steps run on both sides (one row: the
    # small-step kernels the default bench line times; six rows of mixed lengths: the tensor-core GEMMs, the
    # dequantising GEMM and the TMA-fed attention with several splits per row).  Logits, exit layers, scores, row lists
    # and the K/V of every layer and position are compared as in every other test.
    m = model("8b")
    shape = m[0]
    B, n_steps = len(lens), 3
    p = Pair(m, B, max(lens) + n_steps + 1, max(B, 8), page_shuffle_seed=9, kv_store=1, flags=flags)
    w = shape.Hkv * shape.dh
    for b, n in enumerate(lens):
        for l in range(p.L):
            k = synth.normal(31, 1000 * b + 2 * l, (n, w), 1.0, "cuda")
            v = synth.normal(31, 1000 * b + 2 * l + 1, (n, w), 1.0, "cuda")
            p.gpu.write_kv(b, l + 1, 0, k, v)
            p.oracle.write_kv(b, l, 0, k.float().cpu().numpy(), v.float().cpu().numpy())
        p.oracle.set_len(b, n)
        assert p.gpu.seq_len(b) == n
    slots = list(range(B))
    n_early = 0
    for t in range(n_steps):
        tk = toks(shape, B, 300 + t)
        targets = synth.forced_exit_schedule(23, t, B, p.L, shape.entry_layer, "uniform").numpy()
        tau, o = p.oracle_scheduled_step(slots, tk, targets)
        g = p.gpu_step(slots, tk, tau)
        assert np.array_equal(g.exit_layer, o.exit_layer), f"step {t}: exit layers {g.exit_layer} vs {o.exit_layer}"
        p.compare_lists(B)
        p.compare_logits(g.logits, o.logits, f"step {t}")
        ran = ~np.isnan(o.scores)
        assert np.array_equal(ran, ~np.isnan(g.scores))
        assert np.abs(g.scores[ran] - o.scores[ran]).max() < NEAR
        n_early += int((o.exit_layer < p.L).sum())
    for s_ in slots:
        p.compare_kv(s_, p.oracle.seq_len(s_))
        assert p.gpu.seq_len(s_) == p.oracle.seq_len(s_)
    assert p.gpu.stats().device_error == 0
    assert n_early > 0
    p.close()


def test_fp32_cache_oracle_deviation_is_storage_noise():
    # against the oracle with an fp32 cache: direction preserved (cosine bound), max-abs reported
    m = model("8b")
    shape = m[0]
    p = Pair(m, 1, 24, 1, kv_store=0)
    p.prefill([0], [toks(shape, 10, 100)])
    o = p.oracle_step([0], toks(shape, 1, 200), INF)
    g = p.gpu_step([0], toks(shape, 1, 200), INF)
    a, w = g.logits[0].astype(np.float64), o.logits[0].astype(np.float64)
    cos = a @ w / (np.linalg.norm(a) * np.linalg.norm(w))
    err = np.abs(a - w).max()
    print(f"8b vs fp32-cache oracle: cosine {cos:.6f}, max-abs {err:.4f}, logit std {w.std():.3f}")
    assert cos >= 0.999 and err < 0.1 * w.std()
    p.close()

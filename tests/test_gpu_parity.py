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


def toks(shape, n, stream):
    return synth.tokens(shape.seed, stream, n, shape.V).numpy()


def run_scheduled(m, prompt_lens, n_steps, kind="uniform", prefill_exit=None, page_seed=0, max_batch=None,
                  seed=21, kv_store=0, flags=0, storage_yardstick=False, kv_strategy=0):
    shape = m[0]
    B = len(prompt_lens)
    L = len(m[1][0]["layers"])
    p = Pair(m, B, max(prompt_lens) + n_steps + 1, max_batch or max(B, 8), page_shuffle_seed=page_seed,
             kv_store=kv_store, flags=flags, storage_yardstick=storage_yardstick, kv_strategy=kv_strategy)
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


@pytest.mark.parametrize("flags", [0, 1, 32, 33])
def test_launch_modes_agree_with_oracle(flags):
    # 1: CUDA-graph replay; 32: the TMA-fed attention kernel for small steps too (default there: the kernel that
    # fetches the cache early).  Three rows per step: the exit decisions ride in the QKV kernels.
    r = run_scheduled(model("mini8"), [37, 16, 3], 6, "uniform", page_seed=11, flags=flags, max_batch=4)
    assert r["n_early"] > 0


@pytest.mark.parametrize("rows", [1, 2, 4])
def test_small_steps_every_row_count(rows):
    # one, two and four rows per step (each its own kernel instantiation; the decision of block l is taken by the QKV
    # kernel of block l + 1), graph replay on, mixed exit layers
    lens = [29, 5, 18, 40][:rows]
    r = run_scheduled(model("mini8"), lens, 8, "uniform", page_seed=3 + rows, flags=1, max_batch=4)
    assert r["n_early"] > 0


@pytest.mark.parametrize("flags", [0, 16, 2, 64, 1, 65])
def test_mini8_head_dim_128_gqa4(flags):
    # five rows: backbone rows on the tcgen05 GEMM; exit-layer rows on the dequantising tcgen05 GEMM - beside it (0)
    # or behind it (64) -, on the CUDA-core kernel (16), everything on CUDA cores (2); 1, 65: the same two orders
    # replayed from a CUDA graph
    r = run_scheduled(model("mini8"), [70, 16, 31, 48, 5], 18, "uniform", prefill_exit=3, page_seed=7, flags=flags)
    assert r["n_early"] > 0
    print(r)


@pytest.mark.parametrize("rows", [70, 120, 150])
def test_mini8_wide_batches_other_gemm_geometries(rows):
    # 70 rows: operand tiles of 80 rows, three CTAs per SM; 120 rows: 128-row tiles, hi and lo still one TMA box but two
    # MMAs per k-step in the dequantising kernel (its tensor-memory ring leaves no room for a 256-column accumulator
    # twice per SM); 150 rows: 160-row operand tiles, one CTA per SM with deep stages, separate hi / lo boxes; both
    # weight sets live in most layers, lengths mixed so that the attention splits differ per row.  The
    # oracle stores its cache in bf16 here as the large-shape tests do: over millions of cache entries the tail of the
    # fp32-cache deviation (Section 4.1's shared slots hold bf16) reaches the K/V tolerance without any kernel error.
    r = run_scheduled(model("mini8"), [3 + (11 * b) % 29 for b in range(rows)], 3, "uniform", page_seed=rows, max_batch=rows,
                      kv_store=1)
    assert r["n_early"] > 0


@pytest.mark.parametrize("rows", [5, 9, 17, 33, 48, 65, 90, 97, 129, 170, 185, 200, 220, 235, 256])
def test_mini8_row_count_sweep_on_the_tensor_core_kernels(rows):
    # every operand-tile height of the two tcgen05 kernels from 16 to 256 rows (one or two accumulators, hi and lo rows
    # in one TMA box or two, two to four stages, one to three CTAs per SM, with and without K-split clusters), the two
    # GEMMs of a projection side by side, geometric exit layers so that both weight sets are live from the second
    # block on; bf16 cache in the oracle as in the other wide-batch tests
    r = run_scheduled(model("mini8"), [2 + (13 * b + rows) % 41 for b in range(rows)], 2, "geometric", page_seed=100 + rows,
                      max_batch=rows, kv_store=1)
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
    # same weights either way: what differs is the summation order and the 16-bit block-floating-point form the
    # exit-layer kernels give their activations (the A16 of W4A16)
    assert np.abs(outs[0] - outs[1]).max() < 1e-3


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
    # (32 layers of the random-weight 8B shape amplify a single bf16 rounding of a cache entry: deep-layer K/V are held
    # to the plain tolerance or to the distance that 16-bit storage alone produces, whichever is larger)
    r = run_scheduled(model("8b"), [6, 11, 3, 9, 4, 7], 2, "uniform", max_batch=8, kv_store=1, page_seed=5,
                      storage_yardstick=True)
    assert r["n_early"] > 0
    print("8b six rows:", r)


def run_on_history(m, lens, n_steps, flags=1, exit_mode=0, max_batch=None, page_seed=9, sched_seed=23, kv_check=None):
    """Scheduled steps on a synthetic cache history (both caches hold the same N(0,1) bf16 entries): logits, exit
    layers, scores, row lists and the K/V of every layer and position are compared as in every other test."""
    shape = m[0]
    B = len(lens)
    p = Pair(m, B, max(lens) + n_steps + 1, max_batch or max(B, 8), page_shuffle_seed=page_seed, kv_store=1, flags=flags,
             exit_mode=exit_mode, storage_yardstick=shape.name == "8b")
    p.fill_history(lens)
    slots = list(range(B))
    n_early = 0
    for t in range(n_steps):
        tk = toks(shape, B, 300 + t)
        targets = synth.forced_exit_schedule(sched_seed, t, B, p.L, shape.entry_layer, "uniform").numpy()
        tau, o = p.oracle_scheduled_step(slots, tk, targets)
        g = p.gpu_step(slots, tk, tau)
        assert np.array_equal(g.exit_layer, o.exit_layer), f"step {t}: exit layers {g.exit_layer} vs {o.exit_layer}"
        p.compare_lists(B)
        p.compare_logits(g.logits, o.logits, f"step {t}")
        ran = ~np.isnan(o.scores)
        assert np.array_equal(ran, ~np.isnan(g.scores))
        assert np.abs(g.scores[ran] - o.scores[ran]).max() < NEAR
        n_early += int((o.exit_layer < p.L).sum())
    for s_ in (slots if kv_check is None else kv_check):
        p.compare_kv(s_, p.oracle.seq_len(s_))
        assert p.gpu.seq_len(s_) == p.oracle.seq_len(s_)
    assert p.gpu.stats().device_error == 0
    p.close()
    return n_early


@pytest.mark.parametrize("lens", [[1024], [1024, 300, 2050, 17, 640, 1500]])
def test_8b_class_full_size_step_on_synthetic_history(lens):
    # The benchmark's own configuration - all 32 layers of the 8B shape, context ~1024, CUDA-graph replay - checked
    # output by output (one row: the small-step kernels the default bench line times; six rows of mixed lengths: the
    # tensor-core GEMMs, the dequantising GEMM and the TMA-fed attention with several splits per row).
    assert run_on_history(model("8b"), lens, 3) > 0


def test_8b_layer_shape_64_rows_ragged_both_weight_sets():
    # The wide-batch configuration's geometry: the 8B layer shape (its K-splits and 64-row operand tiles in the
    # tensor-core GEMM and in the dequantising GEMM), 64 rows with prompt lengths drawn uniformly from 256-4096 (seed 3,
    # as the benchmark draws them), scheduled exits so that both weight sets are live in most layers.  Eight blocks of
    # that shape instead of 32: depth does not change any kernel's geometry, and the oracle's fp32 cache of 64 x 4096
    # positions x 32 layers would not fit in host memory.  The K/V of eight rows are compared in full.
    lens = synth.prompt_lengths(3, 64, 256, 4096)
    n_early = run_on_history(model("8b", 8), lens, 2, max_batch=64, kv_check=list(range(0, 64, 8)))
    assert 8 < n_early < 120


def test_1b_class_8_rows_context_512():
    # the 1B configuration as stated: 16 layers, 8 rows, context 512
    assert run_on_history(model("1b"), [512] * 8, 3, max_batch=8) > 0


def test_batch_min_mode_on_the_tensor_core_path():
    # Eq. 1 literally (the batch leaves together) with six rows: backbone rows on the tcgen05 GEMM, then all rows on
    # the dequantising GEMM
    m = model("mini8")
    shape = m[0]
    B = 6
    p = Pair(m, B, 64, 8, exit_mode=1, page_shuffle_seed=2)
    slots = list(range(B))
    p.prefill(slots, [toks(shape, 5 + 4 * b, b) for b in range(B)])
    seen = set()
    lo = max(shape.entry_layer, 1)
    for t, tau in enumerate([0.4, 0.8, 0.9, 0.95, 0.98, 0.995, 0.9995]):
        tk = toks(shape, B, 40 + t)
        o = p.oracle_step(slots, tk, tau)
        g = p.gpu_step(slots, tk, tau)
        assert len(set(o.exit_layer.tolist())) == 1
        if np.abs(o.scores[:, lo - 1:p.L - 1] - tau).min() <= NEAR:
            break  # a score within 1e-3 of the threshold may flip the batch's decision: histories would differ
        assert np.array_equal(g.exit_layer, o.exit_layer)
        p.compare_lists(B)
        p.compare_logits(g.logits, o.logits, f"batch-min step {t}")
        seen.add(int(o.exit_layer[0]))
    assert len(seen) >= 2
    p.close()


def free_tau_pass(m, prompt_lens, n_steps, frac, max_batch, kv_store=0, flags=1):
    """One threshold for the whole run, the GPU decides: exit layers must equal the oracle's except for tokens with an
    oracle score within 1e-3 of the threshold (counted and printed).  A row whose decision flipped has a different
    history from then on and leaves the comparison; the other rows go on."""
    shape = m[0]
    B = len(prompt_lens)
    prompts = [toks(shape, n, 100 + b) for b, n in enumerate(prompt_lens)]
    steps = np.stack([toks(shape, B, 200 + t) for t in range(n_steps)])
    tau = natural_tau(m, prompts, steps, frac)
    p = Pair(m, B, max(prompt_lens) + n_steps + 1, max_batch, kv_store=kv_store, flags=flags, page_shuffle_seed=17)
    slots = list(range(B))
    p.prefill(slots, prompts)
    alive = np.ones(B, bool)
    n_cmp = n_near = n_early = 0
    for t in range(n_steps):
        o = p.oracle_step(slots, steps[t], tau)
        g = p.gpu_step(slots, steps[t], tau)
        for b in range(B):
            if not alive[b]:
                continue
            n_cmp += 1
            n_early += int(o.exit_layer[b] < p.L)
            if g.exit_layer[b] != o.exit_layer[b]:
                assert p.near_threshold(o.scores[b], tau, max(g.exit_layer[b], o.exit_layer[b])), \
                    f"step {t} row {b}: exit {g.exit_layer[b]} vs {o.exit_layer[b]} with no score within 1e-3 of tau"
                n_near += 1
                alive[b] = False
        if alive.any():
            p.compare_logits(g.logits[alive], o.logits[alive], f"free step {t}")
    print(f"free-tau pass {shape.name}: tau={tau:.5f}, {n_cmp} decisions compared, {n_early} early exits, "
          f"{n_near} near-threshold flips")
    p.close()
    return n_cmp, n_early, n_near


def test_free_tau_pass_mini8_and_1b():
    n_cmp, n_early, n_near = free_tau_pass(model("mini8"), [21, 9, 33, 14, 5, 27], 12, 0.5, 8)
    assert n_early > 0 and n_near <= n_cmp // 4
    n_cmp, n_early, n_near = free_tau_pass(model("mini8"), [19], 16, 0.5, 1)
    assert n_near <= n_cmp // 4
    n_cmp, n_early, n_near = free_tau_pass(model("1b"), [40, 23], 6, 0.5, 8, kv_store=1)
    assert n_near <= n_cmp // 2


@pytest.mark.parametrize("name,prompt_len", [("1b", 40), ("8b", 12)])
def test_bf16_cache_storage_noise_oracle_vs_oracle_and_gpu(name, prompt_len):
    # Why the large shapes are compared with the oracle whose cache entries are rounded to bf16 (Section 4.1 keeps
    # the KV cache in a 16-bit format): the SAME inputs through the oracle with an fp32 cache and through the oracle
    # with bf16 storage - no kernel involved - already differ by more than the 2e-2 logit bound on these random-weight
    # models.  The GPU, which stores bf16, must sit within the stated bound of the bf16-storage oracle, and its
    # distance from the fp32-cache oracle may exceed the oracle-to-oracle distance by at most that bound.
    m = model(name)
    shape = m[0]
    prompt, steps = toks(shape, prompt_len, 100), toks(shape, 3, 200)
    a = Pair(m, 1, prompt_len + 8, 1, kv_store=0)
    b = Pair(m, 1, prompt_len + 8, 1, kv_store=1)
    a.prefill([0], [prompt])
    b.oracle.prefill(0, prompt)
    worst_oo = worst_g32 = worst_g16 = 0.0
    for t in range(3):
        oa = a.oracle_step([0], [steps[t]], INF)
        ob = b.oracle_step([0], [steps[t]], INF)
        g = a.gpu_step([0], [steps[t]], INF)
        x32, x16, xg = (v.logits[0].astype(np.float64) for v in (oa, ob, g))
        cos = lambda u, v: u @ v / (np.linalg.norm(u) * np.linalg.norm(v))
        assert cos(x32, x16) >= 0.999 and cos(xg, x32) >= 0.999 and cos(xg, x16) >= 0.999
        worst_oo = max(worst_oo, np.abs(x32 - x16).max())
        worst_g32 = max(worst_g32, np.abs(xg - x32).max())
        worst_g16 = max(worst_g16, np.abs(xg - x16).max())
    print(f"{name}: logits max-abs  fp32-cache oracle vs bf16-cache oracle {worst_oo:.4f}   GPU vs fp32-cache oracle "
          f"{worst_g32:.4f}   GPU vs bf16-cache oracle {worst_g16:.4f}   (logit std {x32.std():.3f})")
    assert worst_g16 <= 2e-2
    assert worst_oo <= 0.1 * x32.std()
    assert worst_g32 <= worst_oo + 2e-2
    a.close()
    b.close()


@pytest.mark.parametrize("flags", [0, 1])
def test_free_running_generation_feeds_tokens_back_on_the_device(flags):
    # river_generate against the oracle generating greedily from its own tokens: the token streams must agree up to
    # the first step at which the oracle's choice is ambiguous (top-2 logit gap below twice the logit tolerance) or an
    # exit score lies within 1e-3 of the threshold; at least a few steps have to be comparable
    m = model("mini8")
    shape = m[0]
    prompts = [toks(shape, 12, 0), toks(shape, 30, 1), toks(shape, 5, 2)]
    steps_tok = np.stack([toks(shape, 3, 50 + t) for t in range(6)])
    tau = natural_tau(m, prompts, steps_tok, 0.5)
    n_steps = 24
    p = Pair(m, 3, 30 + n_steps + 2, 4, flags=flags, page_shuffle_seed=2)
    p.prefill([0, 1, 2], prompts)
    tok0 = toks(shape, 3, 77)
    g_tok, g_exit = p.gpu.generate([0, 1, 2], torch.from_numpy(tok0.astype(np.int32)).cuda(),
                                   torch.full((3,), tau, dtype=torch.float32, device="cuda"), n_steps)
    torch.cuda.synchronize()
    g_tok, g_exit = g_tok.cpu().numpy(), g_exit.cpu().numpy()
    alive = np.ones(3, bool)
    cur = tok0.copy()
    compared = 0
    for t in range(n_steps):
        o = p.oracle_step([0, 1, 2], cur, tau)
        top2 = np.sort(o.logits, axis=1)[:, -2:]
        for b in range(3):
            if not alive[b]:
                continue
            if p.near_threshold(o.scores[b], tau, p.L) or top2[b, 1] - top2[b, 0] < 4e-2:
                alive[b] = False  # from here on the two sides may legitimately differ
                continue
            assert g_exit[t, b] == o.exit_layer[b] and g_tok[t, b] == o.next_tok[b], (t, b)
            compared += 1
        cur = np.where(alive, o.next_tok, g_tok[t]).astype(np.int32)
        if not alive.any():
            break
    print(f"free-running generation: {compared} (step, row) pairs compared before ambiguity")
    assert compared >= 6
    for b in range(3):
        assert p.gpu.seq_len(b) == len(prompts[b]) + n_steps
    assert p.gpu.stats().device_error == 0
    p.close()


def test_pool_exhaustion_fails_cleanly_and_the_retry_is_exact():
    # a step that needs more pages than are free takes none (no half-updated page table), and the same rows step
    # correctly once pages have been released
    from paper_2604_18396_b200 import RiverError
    m = model("tiny")
    shape = m[0]
    p = Pair(m, 3, 48, 4, n_pages=4, page_shuffle_seed=8)
    prompts = [toks(shape, 16, b) for b in range(3)]  # one full page each: every row's next token needs a new page
    p.prefill([0, 1, 2], prompts)
    assert p.gpu.stats().pages_in_use == 3
    tk = toks(shape, 3, 70)
    with pytest.raises(RiverError) as e:
        p.gpu_step([0, 1, 2], tk, INF)  # three new pages needed, one free
    assert e.value.code == -4
    assert p.gpu.stats().pages_in_use == 3 and [p.gpu.seq_len(s) for s in range(3)] == [16, 16, 16]
    p.gpu.release(2)
    p.oracle.release(2)
    for t in range(3):
        tk = toks(shape, 2, 71 + t)
        targets = synth.forced_exit_schedule(5, t, 2, shape.L, shape.entry_layer).numpy()
        tau, o = p.oracle_scheduled_step([0, 1], tk, targets)
        g = p.gpu_step([0, 1], tk, tau)
        assert np.array_equal(g.exit_layer, o.exit_layer)
        p.compare_logits(g.logits, o.logits, f"retry step {t}")
    p.compare_kv(0, 19)
    p.compare_kv(1, 19)
    st = p.gpu.stats()
    assert st.device_error == 0 and st.pages_in_use == 4
    with pytest.raises(RiverError) as e:  # prefill: two pages needed, none free
        p.gpu.prefill([2], torch.zeros(20, dtype=torch.int32, device="cuda"), [0, 20])
    assert e.value.code == -4 and p.gpu.seq_len(2) == 0 and p.gpu.stats().pages_in_use == 4
    p.close()


def test_bounded_wait_runs_out_and_is_reported():
    # the library's bounded mbarrier wait on a barrier nobody completes: the kernel returns, the error word says
    # "wait ran out", the call returns RIVER_E_TIMEOUT, further steps are refused until the word is cleared
    from paper_2604_18396_b200 import RiverError
    m = model("tiny")
    shape = m[0]
    p = Pair(m, 1, 32, 1)
    p.prefill([0], [toks(shape, 5, 0)])
    ref = p.gpu_step([0], [3], INF)
    assert p.gpu.selftest_wait_timeout(4000) == -7
    assert p.gpu.stats().device_error == 4
    with pytest.raises(RiverError) as e:
        p.gpu_step([0], [4], INF)
    assert e.value.code == -7 and p.gpu.seq_len(0) == 6
    p.gpu.clear_device_error()
    assert p.gpu.stats().device_error == 0
    o1 = p.oracle_step([0], [3], INF)
    o2 = p.oracle_step([0], [4], INF)
    g2 = p.gpu_step([0], [4], INF)  # the context is usable again
    p.compare_logits(ref.logits, o1.logits, "before the time-out")
    p.compare_logits(g2.logits, o2.logits, "after the time-out")
    p.close()


@pytest.mark.parametrize("depth", [None, 2])
def test_prefill_in_chunks_of_256_positions(depth):
    # prefill_chunk = 256 with max_batch = 4: prompt positions go through the blocks 256 at a time (tensor-core GEMMs
    # with 256-row operand tiles, TMA-fed attention over rows of one sequence at consecutive positions), chunks that
    # hold the end of one prompt and the start of the next, a prompt of one token, and more prompt ends in a chunk
    # than the logits staging has rows for (max_batch).  Last-position logits, every cached K/V and two decode steps
    # afterwards are compared with the oracle.
    m = model("mini8")
    shape = m[0]
    lens = [300, 70, 1, 513, 2, 3, 1, 1, 5, 140]
    B = len(lens)
    p = Pair(m, B, max(lens) + 4, 4, page_shuffle_seed=6, prefill_chunk=256, kv_store=1)
    prompts = [toks(shape, n, 400 + b) for b, n in enumerate(lens)]
    o_logits = np.stack([p.oracle.prefill(b, pr, depth)[0] for b, pr in enumerate(prompts)])
    tok = torch.from_numpy(np.concatenate(prompts).astype(np.int32)).cuda()
    offs = np.concatenate([[0], np.cumsum(lens)]).tolist()
    lg = torch.empty((B, shape.V), dtype=torch.float32, device="cuda")
    nx = torch.empty(B, dtype=torch.int32, device="cuda")
    p.gpu.prefill(list(range(B)), tok, offs, depth, lg, nx)
    torch.cuda.synchronize()
    p.compare_logits(lg.cpu().numpy(), o_logits, "chunked prefill")
    for b in range(B):
        p.compare_kv(b, lens[b])
    for t in range(2):
        sl = [0, 3, 9, 2]
        tk = toks(shape, 4, 500 + t)
        targets = synth.forced_exit_schedule(7, t, 4, p.L, shape.entry_layer).numpy()
        tau, o = p.oracle_scheduled_step(sl, tk, targets)
        g = p.gpu_step(sl, tk, tau)
        assert np.array_equal(g.exit_layer, o.exit_layer)
        p.compare_logits(g.logits, o.logits, f"step {t} after chunked prefill")
    assert p.gpu.stats().device_error == 0
    p.close()


@pytest.mark.parametrize("name,lens", [("tiny", [14, 3, 22]), ("mini8", [40, 9, 75, 18, 31, 6, 12])])
def test_prefill_depth_chosen_by_the_exit_rule(name, lens):
    # prefill_exit_layer = -1: per prompt, the first block after which every position passes Eq. 1.  Thresholds are
    # placed between the per-block minima of the oracle's full-depth scores (never within 2.5e-3 of one), so the depth
    # is unambiguous; depth, last-position logits and the K/V of every layer are compared with the oracle.
    m = model(name)
    shape = m[0]
    B = len(lens)
    prompts = [toks(shape, n, 300 + b) for b, n in enumerate(lens)]
    lo = max(shape.entry_layer, 1)
    L = shape.L
    probe = Pair(m, 1, max(lens) + 2, 4)
    mins = []
    for pr in prompts:  # per-block minima over the prompt's positions, full depth
        sc = []
        for tk in pr:
            sc.append(probe.oracle.decode_step([0], [tk], INF)["scores"][0])
        probe.oracle.release(0)
        mins.append(np.stack(sc)[:, lo - 1:L - 1].min(axis=0))
    probe.close()
    mins = np.stack(mins)  # [B, eligible blocks]
    cands = sorted(set([-1.0, 2.0] + [float(0.5 * (a + b)) for a, b in zip(np.sort(mins.ravel())[:-1], np.sort(mins.ravel())[1:])]))
    cands = [t for t in cands if np.abs(mins - t).min() > 2.5e-3]
    picked = [cands[0], cands[len(cands) // 3], cands[2 * len(cands) // 3], cands[-1]]
    seen = set()
    for tau in picked:
        p = Pair(m, B, max(lens) + 2, 8, page_shuffle_seed=4)
        want, o_logits = [], []
        for b, pr in enumerate(prompts):
            lg, _, depth = p.oracle.prefill_auto(b, pr, tau)
            want.append(depth)
            o_logits.append(lg)
        tok = torch.from_numpy(np.concatenate(prompts).astype(np.int32)).cuda()
        offs = np.concatenate([[0], np.cumsum(lens)]).tolist()
        lg_g = torch.empty((B, shape.V), dtype=torch.float32, device="cuda")
        got = p.gpu.prefill(list(range(B)), tok, offs, -1, lg_g, None, tau)
        torch.cuda.synchronize()
        assert got == want, (tau, got, want)
        p.compare_logits(lg_g.cpu().numpy(), np.stack(o_logits), f"auto prefill tau={tau}")
        for b in range(B):
            p.compare_kv(b, lens[b])
        assert p.gpu.stats().device_error == 0
        seen.update(want)
        p.close()
    assert len(seen) >= 2

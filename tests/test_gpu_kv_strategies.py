"""The KV strategies of skipped blocks other than the exit river (Section 3) on the same kernels: State Propagation
and Mono-Decreasing Exit against the oracle, step by step (exit layers, row lists, scores, logits, every cache entry)."""
import numpy as np
import pytest

from tests.gpu_harness import INF, Pair
from tests.test_gpu_parity import model, run_scheduled, toks

pytestmark = pytest.mark.gpu

SP, MONO, MASK = 1, 2, 3


@pytest.mark.parametrize("rows,flags", [(1, 1), (3, 0), (3, 1), (6, 1)])
def test_state_propagation_steps(rows, flags):
    # one and three rows: streaming kernels (the K / V-only launch runs the bf16 pass over the rows that left); six rows:
    # tensor-core GEMMs over the list of the rows that left.  Prefill stops at block 3: the prompt's deeper K / V are
    # propagated as well.
    # (The oracle stores its cache in bf16 like the library, as in the other multi-row tests of this shape: the rounding
    # of the cache entries alone moves some deep-layer K / V by about the tolerance.)
    lens = [23, 9, 40, 5, 31, 16][:rows]
    r = run_scheduled(model("mini8"), lens, 8, "uniform", prefill_exit=3, page_seed=5 + rows, flags=flags,
                      max_batch=max(rows, 4), kv_strategy=SP, kv_store=1)
    assert r["n_early"] > 0
    print("state propagation:", r)


@pytest.mark.parametrize("rows,flags", [(1, 1), (3, 1), (6, 1)])
def test_mono_decreasing_steps(rows, flags):
    # the requested exit layers vary freely; the library, like the oracle, caps every row at the depth its sequence's
    # previous token reached, writes nothing below, and the cache slots of skipped blocks keep their NaN filling
    lens = [23, 9, 40, 5, 31, 16][:rows]
    r = run_scheduled(model("mini8"), lens, 10, "uniform", page_seed=9 + rows, flags=flags, max_batch=max(rows, 4),
                      kv_strategy=MONO, kv_store=1)
    assert r["n_early"] > 0
    print("mono-decreasing:", r)


def test_mono_decreasing_cap_follows_prefill_depth_and_release():
    m = model("mini8")
    shape = m[0]
    p = Pair(m, 2, 48, 4, kv_strategy=MONO)
    L = p.L
    p.prefill([0], [toks(shape, 12, 3)], 4)  # the prompt stops at block 4: so does every later token of slot 0
    for t in range(3):
        tk = toks(shape, 1, 40 + t)
        o = p.oracle_step([0], tk, INF)
        g = p.gpu_step([0], tk, INF)
        assert g.exit_layer[0] == o.exit_layer[0] == 4
        p.compare_logits(g.logits, o.logits, f"step {t}")
    p.compare_kv(0, p.oracle.seq_len(0))
    # a released slot starts over at full depth
    p.gpu.release(0)
    p.oracle.release(0)
    p.prefill([0], [toks(shape, 7, 4)])
    tk = toks(shape, 1, 50)
    o = p.oracle_step([0], tk, INF)
    g = p.gpu_step([0], tk, INF)
    assert g.exit_layer[0] == o.exit_layer[0] == L
    p.compare_logits(g.logits, o.logits, "after release")
    assert p.gpu.stats().device_error == 0
    p.close()


@pytest.mark.parametrize("rows,flags,steps", [(1, 1, 14), (3, 1, 10), (6, 1, 8)])
def test_kv_mask_steps(rows, flags, steps):
    # exits are free; skipped blocks write nothing; a later token's attention in block l must see exactly the positions
    # whose token ran block l (the small-step kernel for 1-3 rows, the TMA-fed tensor-core kernel for 6): any position
    # seen by mistake would bring the pool's NaN filling into the logits
    lens = [23, 9, 40, 5, 31, 16][:rows]
    r = run_scheduled(model("mini8"), lens, steps, "uniform", prefill_exit=4, page_seed=13 + rows, flags=flags,
                      max_batch=max(rows, 4), kv_strategy=MASK, kv_store=1)
    assert r["n_early"] > 0
    print("kv mask:", r)


def test_kv_mask_long_context_split_attention():
    # one row with a context long enough for the TMA-fed kernel with several splits, early exits in the history
    m = model("mini8")
    shape = m[0]
    p = Pair(m, 1, 400, 4, kv_strategy=MASK, kv_store=1, flags=33)  # 32: the TMA-fed kernel for small steps too
    p.prefill([0], [toks(shape, 300, 3)], 3)  # blocks 4..L see nothing of the prompt
    rng = np.random.default_rng(1)
    for t in range(6):
        tk = toks(shape, 1, 60 + t)
        tau, o = p.oracle_scheduled_step([0], tk, rng.integers(1, p.L + 1, 1))
        g = p.gpu_step([0], tk, tau)
        assert np.array_equal(g.exit_layer, o.exit_layer)
        p.compare_logits(g.logits, o.logits, f"step {t}")
    p.compare_kv(0, p.oracle.seq_len(0))
    assert p.gpu.stats().device_error == 0
    p.close()

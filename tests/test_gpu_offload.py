"""Backbone offloading (Section 4.2): blocks kept in pinned host memory and staged into two device slots give the same
step as the resident model, and a step whose rows have all left before the first offloaded block copies nothing."""
import numpy as np
import pytest
import torch

from tests.gpu_harness import INF, Pair, draw_model
from workloads import synth

pytestmark = pytest.mark.gpu

MATS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")


def offloaded_model(name, first):
    """The drawn model with backbone blocks >= first held on the host: on the device those blocks alias two slots,
    which start out filled with NaN so that any use before staging shows."""
    shape, (bb_c, rv_c), (bb_g, rv_g) = draw_model(name)
    L = len(bb_g["layers"])
    slots = [{n: torch.full_like(bb_g["layers"][first - 1][n], float("nan")) for n in MATS} for _ in range(2)]
    host = [None] * L
    for l in range(first, L + 1):
        host[l - 1] = {n: bb_c["layers"][l - 1][n].contiguous().pin_memory() for n in MATS}
        for n in MATS:
            bb_g["layers"][l - 1][n] = slots[(l - first) & 1][n]
    return (shape, (bb_c, rv_c), (bb_g, rv_g)), host


@pytest.mark.parametrize("B", [1, 3, 6])
def test_offloaded_steps_match_the_oracle(B):
    first = 3
    model, host = offloaded_model("mini8", first)
    # the oracle stores its cache entries in bf16 like the library: with six rows and 40-60 cached positions the storage
    # rounding alone moves some deep-layer K/V of this shape by about 1 % of their rms, the KV tolerance itself
    p = Pair(model, max_seqs=B, max_len=96, max_batch=8, kv_store=1)
    p.gpu.offload(first, host)
    L = p.L
    prompts = [synth.tokens(5, b, 20 + 7 * b, p.shape.V) for b in range(B)]
    slots = list(range(B))
    p.prefill(slots, prompts)
    after_prefill = p.gpu.stats().offload_fetches
    assert after_prefill >= L - first + 1
    tok = np.array([pr[-1] for pr in prompts], np.int32)
    rng = np.random.default_rng(B)
    near = 0
    for t in range(6):
        if t == 2:
            targets = np.full(B, 1)           # every row leaves before the first offloaded block
        elif t == 3:
            targets = np.full(B, L)           # full depth: every offloaded block is staged
        else:
            targets = rng.integers(1, L + 1, B)
        tau, want = p.oracle_scheduled_step(slots, tok, targets)
        before = p.gpu.stats().offload_fetches
        got = p.gpu_step(slots, tok, tau)
        fetched = p.gpu.stats().offload_fetches - before
        deepest = int(want.exit_layer.max())
        risky = any(p.near_threshold(want.scores[b], tau[b], int(want.exit_layer[b])) for b in range(B))
        near += risky
        if not risky:
            assert np.array_equal(got.exit_layer, want.exit_layer), (t, got.exit_layer, want.exit_layer)
            p.compare_logits(got.logits, want.logits, f"step {t}")
            p.compare_lists(B)
            # a block is copied only while some row is still in the backbone (plus one block started ahead)
            assert fetched <= max(0, min(deepest, L) - first + 1) + 1, (t, fetched, deepest)
            if deepest < first:
                assert fetched == 0
        tok = want.next_tok.astype(np.int32)
    for b in range(B):
        p.compare_kv(b, p.oracle.seq_len(b), f"slot {b}")
    assert near <= 2
    assert p.gpu.stats().offload_fetches > after_prefill
    p.close()


def test_offload_rejects_unaliased_layers():
    model = draw_model("tiny")
    p = Pair(model, max_seqs=1, max_len=32, max_batch=1)
    shape, (bb_c, _), _ = model
    L = p.L
    host = [{n: bb_c["layers"][l][n].contiguous().pin_memory() for n in MATS} for l in range(L)]
    if L >= 4:
        with pytest.raises(RuntimeError):
            p.gpu.offload(2, host)  # blocks 2 and 4 have device matrices of their own
    with pytest.raises(RuntimeError):
        p.gpu.offload(1, host)
    p.gpu.offload(0, None)
    p.close()


def test_exit_histogram_and_offload_suggestion():
    # the counters follow the exit layers of the decoded tokens (not the prompt's), and the suggested first offloaded
    # block is the first one that at most the given fraction of them reached
    model = draw_model("mini8")
    p = Pair(model, max_seqs=3, max_len=64, max_batch=4)
    L = p.L
    prompts = [synth.tokens(5, b, 9 + 4 * b, p.shape.V) for b in range(3)]
    p.prefill([0, 1, 2], prompts)
    assert p.gpu.suggest_offload(0.5) == 0 and sum(p.gpu.exit_histogram()) == 0
    tok = np.array([pr[-1] for pr in prompts], np.int32)
    want = np.zeros(L + 1, np.int64)
    schedule = [[2, 2, 6], [1, 3, 2], [2, 6, 2], [2, 1, 4]]
    for forced in schedule:
        o = p.oracle_step([0, 1, 2], tok, INF, forced)
        g = p.gpu_step([0, 1, 2], tok, INF, forced)
        assert np.array_equal(g.exit_layer, o.exit_layer)
        for e in o.exit_layer:
            want[e] += 1
        tok = o.next_tok.astype(np.int32)
    assert p.gpu.exit_histogram() == want.tolist()
    total = int(want.sum())
    for frac in (0.0, 0.1, 0.2, 0.5, 1.0):
        expect = 0
        for l in range(2, L + 1):
            if int(want[l:].sum()) <= frac * total:
                expect = l
                break
        assert p.gpu.suggest_offload(frac) == expect, frac
    assert p.gpu.exit_histogram(reset=True) == want.tolist() and sum(p.gpu.exit_histogram()) == 0
    p.close()


def test_offload_is_refused_under_state_propagation():
    # State Propagation projects K / V with every skipped block's backbone matrices: none of them may live on the host
    model, host = offloaded_model("mini8", 3)
    p = Pair(model, max_seqs=1, max_len=32, max_batch=4, kv_strategy=1)
    with pytest.raises(RuntimeError):
        p.gpu.offload(3, host)
    p.close()

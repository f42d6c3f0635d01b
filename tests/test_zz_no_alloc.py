"""The allocation-free greedy-selection entry point agrees with the decode step's own next tokens.

Some callers of the library cannot allocate device memory where they need a token: a sampling hook in a serving
loop that gave all device memory to the KV cache at start-up, or a latency-critical loop in which an allocation
would stall the device.  river_argmax_noalloc serves them from a fixed scratch array inside the library.  Here it
is called through the C ABI on the logits that river_decode_step produced and must return the very tokens that
river_decode_step returned (same tie rule: lowest id), twice in a row, since every call reuses the one array.
This file sorts last on purpose: a run that stops at the first failure has then run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _decode_logits():
    from tests.gpu_harness import INF, Pair, draw_model
    from workloads import synth
    m = draw_model("tiny")
    shape = m[0]
    p = Pair(m, 5, 40, 8)
    prompts = [synth.tokens(3, b, 4 + 5 * b, shape.V).numpy() for b in range(5)]
    p.prefill(list(range(5)), prompts)
    outs = [p.gpu_step(list(range(5)), synth.tokens(3, 20 + t, 5, shape.V).numpy(), 0.93) for t in range(2)]
    p.close()
    return outs


def test_noalloc_argmax_matches_decode_step_twice_in_a_row():
    from paper_2604_18396_b200 import binding
    lib = binding.load()
    outs = _decode_logits()
    free_before = torch.cuda.mem_get_info()[0]
    for g in outs:  # two calls in a row share the scratch array
        logits = torch.from_numpy(g.logits).cuda()
        # plant exact ties: the lowest id must win, as in the decode step
        top = logits.max(dim=1).values
        logits[0, 7] = top[0]
        logits[0, 3] = top[0]
        want = g.next_tok.copy()
        want[0] = min(3, int(want[0]))
        nxt = torch.full((logits.shape[0],), -1, dtype=torch.int32, device="cuda")
        st = torch.cuda.current_stream()
        rc = lib.river_argmax_noalloc(ctypes.c_void_p(logits.data_ptr()), logits.shape[0], logits.shape[1],
                                      ctypes.c_void_p(nxt.data_ptr()), ctypes.c_void_p(st.cuda_stream))
        assert rc == 0
        torch.cuda.synchronize()
        assert np.array_equal(nxt.cpu().numpy(), want)
    assert torch.cuda.mem_get_info()[0] >= free_before - (8 << 20)  # nothing was allocated behind our back


def test_noalloc_argmax_limits_and_odd_sizes():
    from paper_2604_18396_b200 import argmax_noalloc, binding
    lib = binding.load()
    x = torch.randn(65, 100, device="cuda")
    out = torch.empty(65, dtype=torch.int32, device="cuda")
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert lib.river_argmax_noalloc(ctypes.c_void_p(x.data_ptr()), 65, 100, ctypes.c_void_p(out.data_ptr()), st) == -3
    assert lib.river_argmax_noalloc(None, 1, 100, ctypes.c_void_p(out.data_ptr()), st) == -1
    assert lib.river_argmax_noalloc(ctypes.c_void_p(x.data_ptr()), 1, 0, ctypes.c_void_p(out.data_ptr()), st) == -1
    g = torch.Generator(device="cuda").manual_seed(5)
    for n, V in ((1, 1), (3, 127), (64, 128256), (2, 1000003)):  # fewer columns than CTAs, ragged tails, the full limit
        x = torch.randn(n, V, device="cuda", generator=g)
        out = torch.empty(n, dtype=torch.int32, device="cuda")
        argmax_noalloc(x, out)
        argmax_noalloc(x, out)
        torch.cuda.synchronize()
        assert torch.equal(out.long(), x.argmax(dim=1))

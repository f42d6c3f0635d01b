"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol river.h declares."""
import ctypes
import os
import re

import pytest

from paper_2604_18396_b200 import binding, buildlib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    buildlib.build()
    return binding.load()


def _declared():
    src = open(os.path.join(ROOT, "include", "river.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(river_[a-z0-9_]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_struct_layouts_match_header():
    # field order and count of the ctypes mirrors follow the header text
    src = open(os.path.join(ROOT, "include", "river.h")).read()
    body = re.search(r"typedef struct river_config \{(.*?)\} river_config;", src, re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if decl:
            fields += [f.strip() for f in decl.split(None, 1)[1].split(",")]
    assert fields == [f[0] for f in binding.river_config._fields_]
    assert ctypes.sizeof(binding.river_config) == 4 * len(fields)
    assert ctypes.sizeof(binding.river_layer_weights) == 8 * (9 + 21)
    assert ctypes.sizeof(binding.river_stats_t) == 8 + 8 + 4 * 4 + 8 + 8 + 8


def test_size_queries_and_config_checks_need_no_gpu(lib):
    from workloads import synth
    cfg = binding.make_config(synth.SHAPES["8b"], max_seqs=1, max_pages_per_seq=256, n_pages=256, max_batch=1)
    # 8B shape: 16 tokens/page * 4096 B/token/layer * 32 layers = 2 MiB per page id (cf. the paper's memory table)
    assert lib.river_kv_pool_bytes(ctypes.byref(cfg)) == 256 * 2 * 2 ** 20
    assert lib.river_workspace_bytes(ctypes.byref(cfg)) > 0
    cfg.dh = 96
    assert lib.river_kv_pool_bytes(ctypes.byref(cfg)) == 0 and lib.river_workspace_bytes(ctypes.byref(cfg)) == 0
    h = ctypes.c_void_p()
    assert lib.river_init(ctypes.byref(cfg), None, None, 0, None, 0, None, ctypes.byref(h)) == -2
    assert b"head dim" in lib.river_last_error(None)
    assert lib.river_seq_len(None, 0) == -5

"""ctypes front end of the CPU oracle (river_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the benchmark's
cpu_baseline / reference legs; the product never imports it.  The C file is compiled on
the machine that runs it (the object name carries a hash of the host CPU's feature flags,
because it is built with -march=native).
"""
from __future__ import annotations

import ctypes as C
import hashlib
import os
import subprocess
from typing import List, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "river_oracle.c")
BB_NAMES = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "wg", "wu", "wd")
MAT_NAMES = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")


def _cpu_tag() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            flags = next((ln for ln in f if ln.startswith("flags")), "")
    except OSError:
        flags = ""
    with open(_SRC, "rb") as f:
        src = f.read()
    return hashlib.sha1(flags.encode() + src).hexdigest()[:12]


def build(verbose: bool = False) -> str:
    """Compile river_oracle.c into oracle/liboracle-<tag>.so if that file is missing."""
    so = os.path.join(_HERE, f"liboracle-{_cpu_tag()}.so")
    if not os.path.exists(so):
        tmp = so + f".{os.getpid()}.tmp"
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        if verbose:
            print(" ".join(cmd))
        subprocess.check_call(cmd)
        os.replace(tmp, so)
    return so


class OrcConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("L", "d", "Hq", "Hkv", "dh", "F", "V")] + [
        ("rms_eps", C.c_float), ("rope_theta", C.c_float)] + [
        (n, C.c_int32) for n in ("entry_layer", "group", "max_seqs", "max_len", "exit_mode", "kv_store", "kv_strategy")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.POINTER(OrcConfig), C.c_void_p, C.c_void_p, C.c_void_p,
                                 C.POINTER(C.c_void_p), C.POINTER(C.c_void_p)]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_seq_len.argtypes = [C.c_void_p, C.c_int]
        L.orc_set_len.argtypes = [C.c_void_p, C.c_int, C.c_int]
        L.orc_release.argtypes = [C.c_void_p, C.c_int]
        L.orc_decode_step.argtypes = [C.c_void_p, C.c_int] + [C.c_void_p] * 8
        L.orc_last_lists.argtypes = [C.c_void_p, C.c_int] + [C.c_void_p] * 4
        L.orc_plain_step.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_prefill.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_prefill_auto.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_float, C.c_void_p, C.c_void_p]
        L.orc_read_kv.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_write_kv.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_write_count.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int]
        L.orc_similarity.restype = C.c_float
        L.orc_similarity.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.orc_rope.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_float]
        L.orc_attention.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_float, C.c_void_p]
        L.orc_matvec_bf16.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_matvec_w4.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                    C.c_void_p]
        L.orc_dequant_w4.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]
        L.orc_kv_bytes_16bit.restype = C.c_uint64
        L.orc_kv_bytes_16bit.argtypes = [C.POINTER(OrcConfig), C.c_uint64]
        L.orc_threads.restype = C.c_int
        _lib = L
    return _lib


def _p(a) -> int:
    if a is None:
        return 0
    if isinstance(a, torch.Tensor):
        assert a.device.type == "cpu" and a.is_contiguous()
        return a.data_ptr()
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def make_config(shape, max_seqs: int, max_len: int, exit_mode: int = 0, entry_layer: Optional[int] = None,
                n_layers: Optional[int] = None, kv_store: int = 0, kv_strategy: int = 0) -> OrcConfig:
    return OrcConfig(L=n_layers or shape.L, d=shape.d, Hq=shape.Hq, Hkv=shape.Hkv, dh=shape.dh, F=shape.F,
                     V=shape.V, rms_eps=shape.rms_eps, rope_theta=shape.rope_theta,
                     entry_layer=shape.entry_layer if entry_layer is None else entry_layer, group=shape.group,
                     max_seqs=max_seqs, max_len=max_len, exit_mode=exit_mode, kv_store=kv_store,
                     kv_strategy=kv_strategy)


class Oracle:
    """The oracle over one model (CPU tensors: bf16 backbone, (codes, scale, zero) river)."""

    def __init__(self, shape, backbone: dict, river: List[Optional[dict]], max_seqs: int, max_len: int,
                 exit_mode: int = 0, entry_layer: Optional[int] = None, kv_store: int = 0, kv_strategy: int = 0):
        self.L = len(backbone["layers"])
        self.cfg = make_config(shape, max_seqs, max_len, exit_mode, entry_layer, n_layers=self.L, kv_store=kv_store,
                               kv_strategy=kv_strategy)
        self.shape = shape
        self._keep = (backbone, river)
        bb = (C.c_void_p * (self.L * 9))()
        rv = (C.c_void_p * (self.L * 21))()
        for l, lay in enumerate(backbone["layers"]):
            for j, n in enumerate(BB_NAMES):
                bb[l * 9 + j] = _p(lay[n])
            if river[l] is not None:
                for j, n in enumerate(MAT_NAMES):
                    for t in range(3):
                        rv[l * 21 + 3 * j + t] = _p(river[l][n][t])
        self.h = lib().orc_create(C.byref(self.cfg), _p(backbone["embed"]), _p(backbone["lm_head"]),
                                  _p(backbone["final_norm"]), bb, rv)
        if not self.h:
            raise ValueError("orc_create rejected the configuration")

    def close(self):
        if self.h:
            lib().orc_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def seq_len(self, slot: int) -> int:
        return lib().orc_seq_len(self.h, slot)

    def set_len(self, slot: int, n: int):
        lib().orc_set_len(self.h, slot, n)

    def release(self, slot: int):
        lib().orc_release(self.h, slot)

    def decode_step(self, slots, tok, tau, forced_exit=None, want_logits=True, want_scores=True):
        """-> dict(logits [B,V] f32 | None, next_tok [B], exit_layer [B], scores [B,L] | None)."""
        B = len(slots)
        slots = np.ascontiguousarray(slots, dtype=np.int32)
        tok = np.ascontiguousarray(tok, dtype=np.int32)
        tau = np.ascontiguousarray(np.broadcast_to(np.asarray(tau, dtype=np.float32), (B,)))
        fe = None if forced_exit is None else np.ascontiguousarray(forced_exit, dtype=np.int32)
        logits = np.empty((B, self.cfg.V), np.float32) if want_logits else None
        nxt = np.empty(B, np.int32)
        el = np.empty(B, np.int32)
        sc = np.empty((B, self.L), np.float32) if want_scores else None
        rc = lib().orc_decode_step(self.h, B, _p(slots), _p(tok), _p(tau), _p(fe), _p(logits), _p(nxt), _p(el),
                                   _p(sc))
        if rc:
            raise ValueError(f"orc_decode_step failed: {rc}")
        return {"logits": logits, "next_tok": nxt, "exit_layer": el, "scores": sc}

    def last_lists(self, B: int):
        act = np.empty((self.L + 1, B), np.int32)
        riv = np.empty((self.L + 1, B), np.int32)
        na = np.empty(self.L + 1, np.int32)
        nr = np.empty(self.L + 1, np.int32)
        lib().orc_last_lists(self.h, B, _p(act), _p(na), _p(riv), _p(nr))
        return act, na, riv, nr

    def plain_step(self, slots, tok, use_river: bool = False):
        B = len(slots)
        slots = np.ascontiguousarray(slots, dtype=np.int32)
        tok = np.ascontiguousarray(tok, dtype=np.int32)
        logits = np.empty((B, self.cfg.V), np.float32)
        nxt = np.empty(B, np.int32)
        rc = lib().orc_plain_step(self.h, B, _p(slots), _p(tok), int(use_river), _p(logits), _p(nxt))
        if rc:
            raise ValueError(f"orc_plain_step failed: {rc}")
        return logits, nxt

    def prefill(self, slot: int, tokens, exit_layer: Optional[int] = None):
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        logits = np.empty(self.cfg.V, np.float32)
        nxt = C.c_int32(0)
        e_p = self.L if exit_layer is None else exit_layer
        rc = lib().orc_prefill(self.h, slot, _p(tokens), len(tokens), e_p, _p(logits), C.addressof(nxt))
        if rc:
            raise ValueError(f"orc_prefill failed: {rc}")
        return logits, int(nxt.value)

    def prefill_auto(self, slot: int, tokens, tau: float):
        """Prefill at the depth the exit rule picks for the whole prompt -> (logits, next token, depth)."""
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        logits = np.empty(self.cfg.V, np.float32)
        nxt = C.c_int32(0)
        rc = lib().orc_prefill_auto(self.h, slot, _p(tokens), len(tokens), C.c_float(tau), _p(logits), C.addressof(nxt))
        if rc < 0:
            raise ValueError(f"orc_prefill_auto failed: {rc}")
        return logits, int(nxt.value), rc

    def read_kv(self, slot: int, layer0: int, pos0: int, n: int):
        w = self.cfg.Hkv * self.cfg.dh
        k = np.empty((n, w), np.float32)
        v = np.empty((n, w), np.float32)
        if lib().orc_read_kv(self.h, slot, layer0, pos0, n, _p(k), _p(v)):
            raise ValueError("orc_read_kv: bad range")
        return k, v

    def write_kv(self, slot: int, layer0: int, pos0: int, k, v):
        k = np.ascontiguousarray(k, dtype=np.float32)
        v = np.ascontiguousarray(v, dtype=np.float32)
        if lib().orc_write_kv(self.h, slot, layer0, pos0, k.shape[0], _p(k), _p(v)):
            raise ValueError("orc_write_kv: bad range")

    def attention(self, layer0: int, slot: int, pos: int, q):
        q = np.ascontiguousarray(q, dtype=np.float32)
        out = np.empty_like(q)
        lib().orc_attention(self.h, layer0, slot, pos, _p(q), _p(out))
        return out

    def write_count(self, slot: int, layer0: int, pos: int) -> int:
        return lib().orc_write_count(self.h, slot, layer0, pos)


def threads() -> int:
    return lib().orc_threads()

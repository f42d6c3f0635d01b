"""Thin ctypes binding of include/river.h.

Argument marshalling only: every step of the decode path runs in the CUDA library.  torch is
used for device memory (weights, KV pool, workspace, I/O tensors) and for the stream.  There is
no fallback: without the compiled library, or without a B200, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

from . import buildlib as _build

# ---------------------------------------------------------------- C structs (mirror include/river.h)
RIVER_OK = 0
RIVER_EXIT_PER_TOKEN, RIVER_EXIT_BATCH_MIN = 0, 1
RIVER_F_GRAPH, RIVER_F_NO_TC, RIVER_F_NO_W4TC, RIVER_F_TMA_ATTN, RIVER_F_SERIAL_TC = 1, 2, 16, 32, 64
ERR_NAMES = {-1: "BADARG", -2: "SHAPE", -3: "NOMEM", -4: "NOPAGE", -5: "BADSLOT", -6: "DEVICE", -7: "TIMEOUT"}


class river_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("L", "d", "Hq", "Hkv", "dh", "F", "V")] + [
        ("rms_eps", C.c_float), ("rope_theta", C.c_float)] + [
        (n, C.c_int32) for n in ("entry_layer", "group", "page_size", "max_seqs", "max_pages_per_seq", "n_pages",
                                 "max_batch", "exit_mode")] + [("page_shuffle_seed", C.c_uint32),
                                                               ("flags", C.c_uint32), ("prefill_chunk", C.c_int32), ("kv_strategy", C.c_int32)]


class river_w4(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scale", C.c_void_p), ("zero", C.c_void_p)]


class river_layer_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "wg", "wu", "wd")] + [
        (n, river_w4) for n in ("rq", "rk", "rv", "ro", "rg", "ru", "rd")]


class river_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("layers", C.POINTER(river_layer_weights))]


class river_stats_t(C.Structure):
    _fields_ = [("steps", C.c_int64), ("launches_total", C.c_int64), ("launches_last_step", C.c_int32),
                ("batch_last", C.c_int32), ("device_error", C.c_int32), ("pages_in_use", C.c_int32),
                ("alg_bytes_last_step", C.c_double), ("layers_executed_last", C.c_double),
                ("offload_fetches", C.c_int64)]


class river_kernel_time(C.Structure):
    _fields_ = [("name", C.c_char * 24), ("launches", C.c_int64), ("ms_total", C.c_double),
                ("alg_bytes_total", C.c_double)]


EXPORTS = ("river_argmax_noalloc", "river_profile", "river_profile_read", "river_workspace_bytes", "river_kv_pool_bytes", "river_init", "river_prefill", "river_decode_step",
           "river_decode_step_host", "river_read_kv", "river_write_kv", "river_last_lists", "river_seq_len",
           "river_release", "river_stats", "river_destroy", "river_last_error", "river_clear_device_error",
           "river_selftest_wait_timeout", "river_attention", "river_project_kv", "river_quantize_w4", "river_generate", "river_offload", "river_exit_histogram",
           "river_suggest_offload")

_lib = None


def lib_path() -> str:
    return _build.LIB


def load():
    """Load libriver_b200.so (must have been built; raises otherwise)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_build.LIB):
        raise RuntimeError(f"{_build.LIB} is missing: run paper_2604_18396_b200.build.build() (needs nvcc)")
    L = C.CDLL(_build.LIB)
    vp, i32p = C.c_void_p, C.c_void_p
    L.river_workspace_bytes.restype = C.c_size_t
    L.river_workspace_bytes.argtypes = [C.POINTER(river_config)]
    L.river_kv_pool_bytes.restype = C.c_size_t
    L.river_kv_pool_bytes.argtypes = [C.POINTER(river_config)]
    L.river_init.argtypes = [C.POINTER(river_config), C.POINTER(river_weights), vp, C.c_size_t, vp, C.c_size_t, vp,
                             C.POINTER(vp)]
    L.river_prefill.argtypes = [vp, C.c_int, i32p, vp, i32p, C.c_int, C.c_float, vp, vp, i32p]
    L.river_decode_step.argtypes = [vp, C.c_int, i32p, vp, vp, vp, vp, vp, vp, vp]
    L.river_decode_step_host.argtypes = [vp, C.c_int, i32p, vp, vp, vp, vp, vp, vp, vp]
    L.river_read_kv.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp]
    L.river_write_kv.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp]
    L.river_last_lists.argtypes = [vp, vp, vp, vp, vp]
    L.river_seq_len.argtypes = [vp, C.c_int]
    L.river_release.argtypes = [vp, C.c_int]
    L.river_stats.argtypes = [vp, C.POINTER(river_stats_t)]
    L.river_profile.argtypes = [vp, C.c_int]
    L.river_profile_read.argtypes = [vp, C.POINTER(river_kernel_time), C.c_int, C.POINTER(C.c_int)]
    L.river_argmax_noalloc.argtypes = [vp, C.c_int, C.c_int, vp, vp]
    L.river_attention.argtypes = [vp, C.c_int, C.c_int, i32p, vp, vp]
    L.river_project_kv.argtypes = [vp, C.c_int, C.c_int, C.c_int, i32p, vp, vp]
    L.river_quantize_w4.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp, vp]
    L.river_offload.argtypes = [vp, C.c_int, C.POINTER(river_layer_weights)]
    L.river_exit_histogram.argtypes = [vp, C.POINTER(C.c_int64), C.c_int]
    L.river_suggest_offload.argtypes = [vp, C.c_double]
    L.river_generate.argtypes = [vp, C.c_int, i32p, vp, vp, C.c_int, vp, vp]
    L.river_clear_device_error.argtypes = [vp]
    L.river_selftest_wait_timeout.argtypes = [vp, C.c_int]
    L.river_destroy.argtypes = [vp]
    L.river_destroy.restype = None
    L.river_last_error.argtypes = [vp]
    L.river_last_error.restype = C.c_char_p
    _lib = L
    return L


class RiverError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"river error {ERR_NAMES.get(code, code)}: {msg}")
        self.code = code


def make_config(shape, *, max_seqs: int, max_pages_per_seq: int, n_pages: int, max_batch: int,
                n_layers: Optional[int] = None, entry_layer: Optional[int] = None, exit_mode: int = 0,
                page_shuffle_seed: int = 0, flags: int = 0, prefill_chunk: int = 0,
                kv_strategy: int = 0) -> river_config:
    """river_config from a model shape (anything with L,d,Hq,Hkv,dh,F,V,rms_eps,rope_theta,entry_layer,group)."""
    return river_config(L=n_layers or shape.L, d=shape.d, Hq=shape.Hq, Hkv=shape.Hkv, dh=shape.dh, F=shape.F,
                        V=shape.V, rms_eps=shape.rms_eps, rope_theta=shape.rope_theta,
                        entry_layer=shape.entry_layer if entry_layer is None else entry_layer, group=shape.group,
                        page_size=16, max_seqs=max_seqs, max_pages_per_seq=max_pages_per_seq, n_pages=n_pages,
                        max_batch=max_batch, exit_mode=exit_mode, page_shuffle_seed=page_shuffle_seed, flags=flags,
                        prefill_chunk=prefill_chunk, kv_strategy=kv_strategy)


def _dp(t: Optional[torch.Tensor]) -> int:
    if t is None:
        return 0
    assert t.is_cuda and t.is_contiguous()
    return t.data_ptr()


def _hp(t: Optional[torch.Tensor]) -> int:
    if t is None:
        return 0
    assert (not t.is_cuda) and t.is_contiguous()
    return t.data_ptr()


def _i32_host(xs: Sequence[int]):
    return (C.c_int32 * len(xs))(*[int(v) for v in xs])


def argmax_noalloc(logits: torch.Tensor, next_tok: torch.Tensor, stream=None) -> None:
    """river_argmax_noalloc: next_tok[r] = index of the maximum of logits[r] (ties -> lowest id), no allocation.

    logits: CUDA fp32 [n_rows, V] (n_rows <= 64); next_tok: CUDA int32 [n_rows].  Asynchronous on `stream`
    (default: torch's current stream).  For callers that cannot allocate device memory at this point."""
    assert logits.dtype == torch.float32 and next_tok.dtype == torch.int32 and logits.dim() == 2
    st = stream if stream is not None else torch.cuda.current_stream(logits.device)
    with torch.cuda.device(logits.device):
        rc = load().river_argmax_noalloc(_dp(logits), logits.shape[0], logits.shape[1], _dp(next_tok),
                                         C.c_void_p(st.cuda_stream))
    if rc:
        raise RiverError(rc, "river_argmax_noalloc rejected the call")


def quantize_w4(w: torch.Tensor, group: int = 64, refine_iters: int = 20, stream=None):
    """river_quantize_w4: CUDA bf16 [out, in] -> (codes u8 [out, in/2], scale bf16 [out, in/group], zero bf16 [...])."""
    assert w.is_cuda and w.dtype == torch.bfloat16 and w.dim() == 2 and w.is_contiguous()
    out, inn = w.shape
    codes = torch.empty((out, inn // 2), dtype=torch.uint8, device=w.device)
    scale = torch.empty((out, inn // group), dtype=torch.bfloat16, device=w.device)
    zero = torch.empty_like(scale)
    st = stream if stream is not None else torch.cuda.current_stream(w.device)
    with torch.cuda.device(w.device):
        rc = load().river_quantize_w4(_dp(w), out, inn, group, refine_iters, _dp(codes), _dp(scale), _dp(zero),
                                      C.c_void_p(st.cuda_stream))
    if rc:
        raise RiverError(rc, "river_quantize_w4 rejected the call")
    return codes, scale, zero


class River:
    """A decode context over device-resident weights.

    backbone: {'embed','lm_head','final_norm','layers':[{attn_norm,wq,wk,wv,wo,ffn_norm,wg,wu,wd}]} of CUDA bf16
    tensors; river: per layer None or {name: (codes u8, scale bf16, zero bf16)} CUDA tensors.
    """

    def __init__(self, cfg: river_config, backbone: dict, river: List[Optional[dict]], stream=None):
        L = load()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: this library has no CPU path")
        self.cfg = cfg
        self._keep = (backbone, river)
        nl = cfg.L
        self._layers = (river_layer_weights * nl)()
        for l in range(nl):
            lay = backbone["layers"][l]
            lw = self._layers[l]
            for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "wg", "wu", "wd"):
                setattr(lw, n, _dp(lay[n]))
            if river[l] is not None:
                for short, n in (("rq", "wq"), ("rk", "wk"), ("rv", "wv"), ("ro", "wo"), ("rg", "wg"), ("ru", "wu"),
                                 ("rd", "wd")):
                    c, s, z = river[l][n]
                    setattr(lw, short, river_w4(_dp(c), _dp(s), _dp(z)))
        self._w = river_weights(_dp(backbone["embed"]), _dp(backbone["lm_head"]), _dp(backbone["final_norm"]),
                                self._layers)
        ws = L.river_workspace_bytes(C.byref(cfg))
        kb = L.river_kv_pool_bytes(C.byref(cfg))
        if ws == 0 or kb == 0:
            raise RiverError(-2, "configuration rejected")
        dev = backbone["embed"].device
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=dev)
        # NaN-filled pool: a cache position that is read before it was written shows up at once
        self.kv_pool = torch.full((kb // 2,), float("nan"), dtype=torch.bfloat16, device=dev)
        if stream is None:
            # graph replay cannot be captured on the legacy default stream: give the context a stream of its own
            stream = torch.cuda.Stream(dev) if (cfg.flags & RIVER_F_GRAPH) else torch.cuda.current_stream(dev)
        self.stream = stream
        h = C.c_void_p()
        rc = L.river_init(C.byref(cfg), C.byref(self._w), self.kv_pool.data_ptr(), kb, self.workspace.data_ptr(), ws,
                          C.c_void_p(self.stream.cuda_stream), C.byref(h))
        if rc:
            raise RiverError(rc, L.river_last_error(None).decode())
        self.h = h
        self.device = dev

    # -- helpers
    def _order_after_current(self):
        """Work queued on torch's current stream (input tensors) must precede the step on the context's stream."""
        cur = torch.cuda.current_stream(self.device)
        if cur != self.stream:
            self.stream.wait_stream(cur)

    def _check(self, rc: int):
        if rc:
            raise RiverError(rc, load().river_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None):
            load().river_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- API (same names as the C entry points)
    def prefill(self, slots: Sequence[int], tok: torch.Tensor, offsets: Sequence[int], prefill_exit_layer=None,
                logits_last: Optional[torch.Tensor] = None, next_tok: Optional[torch.Tensor] = None,
                tau: float = float("inf")) -> List[int]:
        """river_prefill; prefill_exit_layer None = the whole backbone, -1 = per prompt by Eq. 1 with threshold tau.
        Returns the depth each prompt left the backbone at."""
        e = self.cfg.L if prefill_exit_layer is None else prefill_exit_layer
        depth = (C.c_int32 * len(slots))()
        self._order_after_current()
        self._check(load().river_prefill(self.h, len(slots), _i32_host(slots), _dp(tok), _i32_host(offsets), e,
                                         C.c_float(tau), _dp(logits_last), _dp(next_tok), depth))
        return list(depth)

    def decode_step(self, slots: Sequence[int], tok: torch.Tensor, tau: torch.Tensor,
                    forced_exit: Optional[torch.Tensor], logits: Optional[torch.Tensor], next_tok: torch.Tensor,
                    exit_layer: torch.Tensor, scores: Optional[torch.Tensor] = None, slots_c=None):
        sc = slots_c if slots_c is not None else _i32_host(slots)
        self._order_after_current()
        self._check(load().river_decode_step(self.h, len(slots), sc, _dp(tok), _dp(tau), _dp(forced_exit),
                                             _dp(logits), _dp(next_tok), _dp(exit_layer), _dp(scores)))

    def decode_step_host(self, slots: Sequence[int], tok: torch.Tensor, tau: torch.Tensor,
                         forced_exit: Optional[torch.Tensor], logits: Optional[torch.Tensor], next_tok: torch.Tensor,
                         exit_layer: torch.Tensor, scores: Optional[torch.Tensor] = None, slots_c=None):
        sc = slots_c if slots_c is not None else _i32_host(slots)
        self._check(load().river_decode_step_host(self.h, len(slots), sc, _hp(tok), _hp(tau), _hp(forced_exit),
                                                  _hp(logits), _hp(next_tok), _hp(exit_layer), _hp(scores)))

    def offload(self, first_offloaded_layer: int, host_layers: Optional[List[dict]] = None):
        """river_offload; host_layers: per layer a dict of pinned CPU bf16 tensors (wq .. wd) or None."""
        nl = self.cfg.L
        arr = (river_layer_weights * nl)()
        if host_layers is not None:
            for l in range(nl):
                if host_layers[l] is not None:
                    for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd"):
                        t = host_layers[l][n]
                        assert t.is_pinned() and t.is_contiguous() and t.dtype == torch.bfloat16
                        setattr(arr[l], n, t.data_ptr())
        self._keep_host = host_layers
        self._check(load().river_offload(self.h, first_offloaded_layer, arr))

    def exit_histogram(self, reset: bool = False):
        """river_exit_histogram -> list of L + 1 counts."""
        buf = (C.c_int64 * (self.cfg.L + 1))()
        self._check(load().river_exit_histogram(self.h, buf, 1 if reset else 0))
        return list(buf)

    def suggest_offload(self, max_deep_fraction: float) -> int:
        rc = load().river_suggest_offload(self.h, float(max_deep_fraction))
        if rc < 0:
            self._check(rc)
        return rc

    def generate(self, slots: Sequence[int], tok0: torch.Tensor, tau: torch.Tensor, n_steps: int):
        """river_generate -> (tokens int32 [n_steps, batch], exit layers int32 [n_steps, batch]), both on the device."""
        B = len(slots)
        out_tok = torch.empty((n_steps, B), dtype=torch.int32, device=self.device)
        out_exit = torch.empty((n_steps, B), dtype=torch.int32, device=self.device)
        self._order_after_current()
        self._check(load().river_generate(self.h, B, _i32_host(slots), _dp(tok0), _dp(tau), n_steps, _dp(out_tok),
                                          _dp(out_exit)))
        return out_tok, out_exit

    def read_kv(self, slot: int, layer: int, pos0: int, n: int):
        w = self.cfg.Hkv * self.cfg.dh
        k = torch.empty((n, w), dtype=torch.bfloat16, device=self.device)
        v = torch.empty((n, w), dtype=torch.bfloat16, device=self.device)
        self._order_after_current()
        self._check(load().river_read_kv(self.h, slot, layer, pos0, n, k.data_ptr(), v.data_ptr()))
        return k, v

    def write_kv(self, slot: int, layer: int, pos0: int, k: torch.Tensor, v: torch.Tensor):
        self._order_after_current()
        self._check(load().river_write_kv(self.h, slot, layer, pos0, k.shape[0], _dp(k), _dp(v)))

    def attention(self, layer: int, slots: Sequence[int], q: torch.Tensor, out: torch.Tensor, slots_c=None):
        sc = slots_c if slots_c is not None else _i32_host(slots)
        self._order_after_current()
        self._check(load().river_attention(self.h, layer, len(slots), sc, _dp(q), _dp(out)))

    def project_kv(self, layer: int, use_exit_layer: bool, slots: Sequence[int], h: torch.Tensor,
                   q_out: Optional[torch.Tensor] = None, slots_c=None):
        sc = slots_c if slots_c is not None else _i32_host(slots)
        self._order_after_current()
        self._check(load().river_project_kv(self.h, layer, int(use_exit_layer), len(slots), sc, _dp(h), _dp(q_out)))

    def last_lists(self, batch: int):
        import numpy as np
        Lp = self.cfg.L + 1
        act = np.empty((Lp, batch), np.int32)
        riv = np.empty((Lp, batch), np.int32)
        na = np.empty(Lp, np.int32)
        nr = np.empty(Lp, np.int32)
        self._check(load().river_last_lists(self.h, act.ctypes.data, na.ctypes.data, riv.ctypes.data, nr.ctypes.data))
        return act, na, riv, nr

    def seq_len(self, slot: int) -> int:
        return load().river_seq_len(self.h, slot)

    def release(self, slot: int):
        self._check(load().river_release(self.h, slot))

    def profile(self, enable: bool):
        self._check(load().river_profile(self.h, int(enable)))

    def profile_read(self):
        """-> [{name, launches, ms_total, alg_bytes_total}] for the kernels timed since profile(True)."""
        buf = (river_kernel_time * 16)()
        n = C.c_int(0)
        self._check(load().river_profile_read(self.h, buf, 16, C.byref(n)))
        return [dict(name=buf[i].name.decode(), launches=buf[i].launches, ms_total=buf[i].ms_total,
                     alg_bytes_total=buf[i].alg_bytes_total) for i in range(n.value)]

    def stats(self) -> river_stats_t:
        """river_stats; a device-error return code (-6, -7) is reported through st.device_error, not raised."""
        st = river_stats_t()
        rc = load().river_stats(self.h, C.byref(st))
        if rc and rc not in (-6, -7):
            self._check(rc)
        return st

    def clear_device_error(self):
        self._check(load().river_clear_device_error(self.h))

    def selftest_wait_timeout(self, poll_limit: int) -> int:
        """river_selftest_wait_timeout: returns the C return code (-7 = the wait ran out, as it should)."""
        return load().river_selftest_wait_timeout(self.h, poll_limit)

#!/usr/bin/env python
"""Benchmark of the early-exit decode step (one JSON line on stdout).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 8b_b1|1b_b8|8b_b64|tiny|attn_micro] [--impl reference]

A step is one decode step of the whole hot path (embed, every block on the backbone or exit-layer weights with
paged GQA attention, exit score, compaction, LM head) over one batch of synthetic, seeded input.  The default
workload is the 8B-class decoder at batch 1 with a 1024-token prompt and thresholds scheduled so that about half
of the tokens leave the backbone early.  value = tokens/s with inputs resident in HBM (CUDA events); e2e = the
same through the host-buffer entry point, host<->device copies inside the timed region.  With --gpus N (under
torchrun) every rank runs an independent replica: the path has no exchange step, so no collective is on it.
--impl reference times the CPU oracle (oracle/) on the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import rtn_w4, synth  # noqa: E402

WORKLOADS = {
    # name: (shape, batch, prompt (lo, hi), seed)
    "tiny": ("tiny", 1, (32, 32), 0),
    "1b_b8": ("1b", 8, (512, 512), 1),
    "8b_b1": ("8b", 1, (1024, 1024), 2),
    "8b_b64": ("8b", 64, (256, 4096), 3),
}
EARLY_FRACTION = 0.5   # share of decode tokens that leave the backbone early
EARLY_MEAN_LAYER = 3.0  # their mean exit layer (the paper's benchmark table reports about 3 of 16 / 32 at tau = 0.5)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for ln in self.proc.stdout:
            self.rows.append([c.strip() for c in ln.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            self.t.join(timeout=2)

    def summary(self):
        mhz, mx, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                mhz.append(float(r[0])); mx = max(mx, float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(mhz)}


def alg_bytes_step(shape, L, exit_layers, positions, want_logits=True, kv_strategy=0):
    """Algorithmic HBM bytes of one decode step from its exit pattern: weights of every (layer, weight set) that
    ran, KV read by every row in every layer it attends in (exit-layer rows attend too), KV written, LM head,
    embedding rows.  kv_strategy 1 (State Propagation): a skipped block costs its bf16 K and V matrices and a KV
    write, no attention; 2 (Mono-Decreasing Exit) and 3 (KV Mask): nothing (KV Mask rows read fewer cache entries than
    counted here: positions without an entry in a block are skipped)."""
    P = shape.layer_params()
    B = len(exit_layers)
    kv_tok = 2.0 * shape.Hkv * shape.dh * 2.0
    total = 0.0
    for l in range(1, L + 1):
        n_act = sum(1 for e in exit_layers if e >= l)
        if n_act > 0:
            total += 2.0 * P
        if n_act < B:
            if kv_strategy == 0:
                total += P / 2.0 + 4.0 * P / shape.group
            elif kv_strategy == 1:
                total += 2.0 * 2.0 * shape.Hkv * shape.dh * shape.d
        for e, p in zip(exit_layers, positions):
            if kv_strategy == 0 or e >= l:
                total += (p + 1) * kv_tok + kv_tok
            elif kv_strategy == 1:
                total += kv_tok
    total += 2.0 * shape.V * shape.d + B * shape.d * 2.0 + (4.0 * B * shape.V if want_logits else 0.0)
    return total


def exit_targets(seed, n, L, entry):
    """Seeded target exit layers: EARLY_FRACTION of the tokens leave early (geometric, mean EARLY_MEAN_LAYER)."""
    early = synth.uniform_int(seed, 5000, n, 0, 1000).numpy() < int(1000 * EARLY_FRACTION)
    geo = synth.forced_exit_schedule(seed, 77, n, L - 1, entry, "geometric", EARLY_MEAN_LAYER).numpy()
    return np.where(early, np.minimum(geo, L - 1), L).astype(np.int32)


def draw_model(shape, device):
    bb = synth.make_backbone(shape, device)
    rv = rtn_w4.make_river(bb, shape.group)
    return bb, rv


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu capture summarised under
# profiles/ (taken on a 4-layer model of the same layer shape: kernel, geometry and operands per launch are those of
# the full model).  Missing key: no capture of that kernel is on file (traffic is then reported as null).
NCU_TRAFFIC = {("8b", "gateup_swiglu"): 235068160.0}  # profiles/stream_proj_kernel_8b4L_b1.md


# ---------------------------------------------------------------------------------------------- CPU oracle timing
def time_oracle(shape, bb_cpu, rv_cpu, B, ctx_len, n_steps, n_warm, seed):
    """Oracle decode steps at context ctx_len on the host cores.  The KV history is synthetic N(0,1) (an oracle
    prefill of the whole prompt would take minutes); exits are forced at the scheduled layers."""
    from oracle import river_oracle as orc
    L = len(bb_cpu["layers"])
    o = orc.Oracle(shape, bb_cpu, rv_cpu, B, ctx_len + n_steps + n_warm + 1)
    w = shape.Hkv * shape.dh
    for b in range(B):
        k = synth.normal(seed, 9000 + b, (ctx_len, w), 1.0, "cpu", torch.float32).numpy()
        for l in range(L):
            o.write_kv(b, l, 0, k, k)
        o.set_len(b, ctx_len)
    targets = exit_targets(seed, (n_steps + n_warm) * B, L, shape.entry_layer).reshape(-1, B)
    toks = synth.tokens(seed, 50, (n_steps + n_warm) * B, shape.V).numpy().reshape(-1, B)
    slots = list(range(B))
    times = []
    for t in range(n_warm + n_steps):
        t0 = time.perf_counter()
        o.decode_step(slots, toks[t], float("inf"), targets[t], want_logits=True, want_scores=False)
        times.append(time.perf_counter() - t0)
    o.close()
    dt = float(np.sum(times[n_warm:]))
    return {"tokens_per_s": B * n_steps / dt, "seconds": dt, "threads": orc.threads(),
            "layers_executed": float(targets[n_warm:].mean() / L)}


def reference_arm(args, wl):
    shape_name, B, (plo, phi), seed = WORKLOADS[wl]
    shape = synth.SHAPES[shape_name]
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    bb, rv = draw_model(shape, dev)
    to_cpu = lambda x: x.cpu() if isinstance(x, torch.Tensor) else (
        {k: to_cpu(v) for k, v in x.items()} if isinstance(x, dict) else type(x)(to_cpu(v) for v in x))
    bb, rv = to_cpu(bb), to_cpu(rv)
    ctx = (plo + phi) // 2
    # bound the run to a few minutes: time one step, then fit the row count of the sample
    Bs = min(B, 4)
    r = time_oracle(shape, bb, rv, Bs, ctx, args.steps, args.warmup, seed)
    from oracle import river_oracle as orc
    cores = orc.threads()
    sample = (f"{args.steps} oracle decode steps, {Bs} of {B} rows, {shape_name} shape, context {ctx} "
              f"(synthetic N(0,1) KV history instead of an oracle prefill), exits forced at the scheduled layers")
    line = {"impl": "reference", "metric": "decode_tokens_per_s", "value": r["tokens_per_s"], "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * r["seconds"] / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl, "shape": shape_name, "batch": Bs, "context": ctx},
            "cpu_baseline": {"value": r["tokens_per_s"], "unit": "tokens/s", "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": r["tokens_per_s"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "layers_executed_fraction": r["layers_executed"]}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- distributed glue
def dist_setup(n_gpus):
    """Replicas only: torch.distributed serves the barrier and the max over ranks of the timed region."""
    import torch.distributed as dist
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        if torch.cuda.is_available():
            torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
        dist.init_process_group(backend)
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def dist_barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def dist_max(x: float) -> float:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        t = torch.tensor([x], dtype=torch.float64, device="cuda" if dist.get_backend() == "nccl" else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())
    return x


def dist_sum(x: float) -> float:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        t = torch.tensor([x], dtype=torch.float64, device="cuda" if dist.get_backend() == "nccl" else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())
    return x


# ---------------------------------------------------------------------------------------------- our arm
def timed_steps(rv, slots_c, slots, toks, taus, logits, nxt, exits, t0, n):
    """n decode steps with device-resident inputs, timed with CUDA events on the launching stream."""
    torch.cuda.synchronize()
    dist_barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(t0, t0 + n):
        rv.decode_step(slots, toks[t], taus[t], None, logits, nxt, exits[t], None, slots_c=slots_c)
    e1.record()
    torch.cuda.synchronize()
    dist_barrier()
    return e0.elapsed_time(e1)


def ours(args, wl):
    import ctypes
    from paper_2604_18396_b200 import River, buildlib, make_config
    rank, world = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    buildlib.build()
    dev = torch.device("cuda", torch.cuda.current_device())
    shape_name, B, (plo, phi), seed = WORKLOADS[wl]
    seed = seed + 1000 * rank  # replicas draw their own prompts; the model is the same
    shape = synth.SHAPES[shape_name]
    if args.layers:
        import dataclasses
        shape = dataclasses.replace(shape, L=args.layers)
    if args.prompt:
        plo = phi = args.prompt
    if args.batch:
        B = args.batch
    L = shape.L
    K, W = args.steps, args.warmup
    n_cal, n_prof, n_e2e = 8, 4, min(K, 64)
    total_steps = n_cal + 2 * (W + K) + 2 * n_prof + (W + n_e2e) + 4
    bb, rvw = draw_model(shape, dev)
    off_host, off_saved = None, 0
    if args.offload_from:  # backbone blocks >= offload_from live in pinned host memory, staged through two slots
        first = args.offload_from
        off_host = [None] * L
        slot_w = [{n: torch.empty_like(bb["layers"][first - 1][n]) for n in synth.MATS} for _ in range(2)]
        for l in range(first, L + 1):
            off_host[l - 1] = {n: bb["layers"][l - 1][n].cpu().contiguous().pin_memory() for n in synth.MATS}
            for n in synth.MATS:
                off_saved += bb["layers"][l - 1][n].numel() * 2
                bb["layers"][l - 1][n] = slot_w[(l - first) & 1][n]
        off_saved -= sum(t.numel() * 2 for s in slot_w for t in s.values())
        torch.cuda.empty_cache()
    lens = synth.prompt_lengths(WORKLOADS[wl][3] + 1000 * rank, B, plo, phi) if plo != phi else [plo] * B
    max_len = max(lens) + total_steps
    pages_per_seq = (max_len + 15) // 16
    n_pages = sum((l + total_steps + 15) // 16 for l in lens)
    flags = args.flags
    cfg = make_config(shape, max_seqs=B, max_pages_per_seq=pages_per_seq, n_pages=n_pages, max_batch=max(B, 8),
                      page_shuffle_seed=seed + 1, flags=flags, prefill_chunk=256, kv_strategy=args.kv_strategy)
    rv = River(cfg, bb, rvw)
    if off_host is not None:
        rv.offload(args.offload_from, off_host)
    torch.cuda.synchronize()
    # everything below runs on the context's stream (its own stream when graph replay is on)
    stream_ctx = torch.cuda.stream(rv.stream)
    stream_ctx.__enter__()
    slots = list(range(B))
    slots_c = (ctypes.c_int32 * B)(*slots)

    # ---- prefill (untimed; whole backbone)
    prompt = torch.cat([synth.tokens(seed, 100 + b, n, shape.V) for b, n in enumerate(lens)]).to(dev)
    offs = np.concatenate([[0], np.cumsum(lens)]).tolist()
    t_pf = time.perf_counter()
    rv.prefill(slots, prompt, offs)
    torch.cuda.synchronize()
    t_pf = time.perf_counter() - t_pf

    toks = synth.tokens(seed, 50, total_steps * B, shape.V).view(total_steps, B).to(dev)
    logits = torch.empty((B, shape.V), dtype=torch.float32, device=dev)
    nxt = torch.empty(B, dtype=torch.int32, device=dev)
    exits = torch.full((total_steps, B), -1, dtype=torch.int32, device=dev)
    inf = torch.full((total_steps, B), float("inf"), dtype=torch.float32, device=dev)

    # ---- calibration: full-depth steps with score read-out give the mean score per layer
    sc = torch.empty((B, L), dtype=torch.float32, device=dev)
    acc = []
    step = 0
    for _ in range(n_cal):
        rv.decode_step(slots, toks[step], inf[step], None, logits, nxt, exits[step], sc, slots_c=slots_c)
        acc.append(sc.clone())
        step += 1
    torch.cuda.synchronize()
    s_mean = torch.stack(acc).float().mean(dim=(0, 1)).cpu().numpy()  # [L]
    lo = max(shape.entry_layer, 1)
    targets = exit_targets(seed, total_steps * B, L, shape.entry_layer).reshape(total_steps, B)
    run_max = np.maximum.accumulate(np.concatenate([[-1.0], s_mean[lo - 1:L - 1]]))  # max score below layer e
    tau_np = np.full((total_steps, B), np.inf, np.float32)
    for e in range(lo, L):
        prev = run_max[e - lo]
        tau_e = 0.5 * (s_mean[e - 1] + prev) if prev > -1.0 else s_mean[e - 1] - 0.05
        tau_np[targets == e] = tau_e
    taus = torch.from_numpy(tau_np).to(dev)

    # ---- timed: early-exit run, then the same kernels at full depth
    timed_steps(rv, slots_c, slots, toks, taus, logits, nxt, exits, step, W)
    step += W
    pos0 = [rv.seq_len(s) for s in slots]
    launches0 = rv.stats().launches_total
    off_fetches0 = rv.stats().offload_fetches
    torch.cuda.profiler.start()  # marks the timed region for `ncu --profile-from-start off`; a no-op otherwise
    with ClockSampler(torch.cuda.current_device()) as clk:
        ms = timed_steps(rv, slots_c, slots, toks, taus, logits, nxt, exits, step, K)
    torch.cuda.profiler.stop()
    launches = rv.stats().launches_total - launches0
    off_fetches = rv.stats().offload_fetches
    ex = exits[step:step + K].cpu().numpy()
    step += K
    ms = dist_max(ms)
    bytes_exit = sum(alg_bytes_step(shape, L, ex[t], [p + t for p in pos0], kv_strategy=args.kv_strategy)
                     for t in range(K)) / K

    timed_steps(rv, slots_c, slots, toks, inf, logits, nxt, exits, step, W)
    step += W
    pos1 = [rv.seq_len(s) for s in slots]
    ms_full = timed_steps(rv, slots_c, slots, toks, inf, logits, nxt, exits, step, K)
    step += K
    ms_full = dist_max(ms_full)
    bytes_full = sum(alg_bytes_step(shape, L, [L] * B, [p + t for p in pos1]) for t in range(K)) / K

    # ---- end to end: host buffers in, results out, every step
    tok_h = toks.cpu().pin_memory()
    tau_h = taus.cpu().pin_memory()
    lg_h = torch.empty((B, shape.V), dtype=torch.float32).pin_memory()
    nx_h = torch.empty(B, dtype=torch.int32).pin_memory()
    el_h = torch.empty(B, dtype=torch.int32).pin_memory()
    for t in range(step, step + W):
        rv.decode_step_host(slots, tok_h[t], tau_h[t], None, lg_h, nx_h, el_h, None, slots_c=slots_c)
    step += W
    torch.cuda.synchronize()
    dist_barrier()
    t0 = time.perf_counter()
    for t in range(step, step + n_e2e):
        rv.decode_step_host(slots, tok_h[t], tau_h[t], None, lg_h, nx_h, el_h, None, slots_c=slots_c)
    torch.cuda.synchronize()
    dist_barrier()
    ms_e2e = dist_max((time.perf_counter() - t0) * 1e3)
    step += n_e2e

    # ---- per-kernel timing passes (outside every timed region): events around every launch.  Full depth, then
    # scheduled exits.
    def profile_pass(thresholds):
        nonlocal step
        rv.profile(True)
        for t in range(step, step + n_prof):
            rv.decode_step(slots, toks[t], thresholds[t], None, logits, nxt, exits[t], None, slots_c=slots_c)
        step += n_prof
        out = rv.profile_read()
        rv.profile(False)
        return out
    prof = profile_pass(inf)
    prof_exit = profile_pass(taus)
    st = rv.stats()

    peak, peak_kind = peaks()
    tok_s = world * B * K / (ms / 1e3)
    line = None
    if rank == 0:
        def table(pr):
            tot = sum(r["ms_total"] for r in pr)
            return {r["name"]: {"launches_per_step": r["launches"] // n_prof, "ms_per_step": round(r["ms_total"] / n_prof, 4),
                                "share": round(r["ms_total"] / tot, 4),
                                "GBps": round(r["alg_bytes_total"] / max(r["ms_total"], 1e-9) / 1e6, 1)} for r in pr}
        dom = max(prof, key=lambda r: r["ms_total"])
        per_launch_ms = dom["ms_total"] / dom["launches"]
        ach = dom["alg_bytes_total"] / dom["launches"] / (per_launch_ms * 1e-3) / 1e9
        kernels = table(prof)
        kernels_exit = table(prof_exit)
        step_gbs = bytes_exit / (ms / K * 1e-3) / 1e9
        full_gbs = bytes_full / (ms_full / K * 1e-3) / 1e9
        line = {
            "metric": "decode_tokens_per_s", "value": tok_s, "unit": "tokens/s", "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl, "shape": shape_name, "batch": B, "prompt": [plo, phi], "context_at_start": pos0[:4],
                       "early_exit_target_fraction": EARLY_FRACTION, "thresholds": "per-step, from calibrated mean scores",
                       "l2": "inputs (weights + KV) larger than L2, no flush", "flags": flags, "layers": L,
                       "parallelism": "replicas only" if world > 1 else "1 GPU", "prefill_s": round(t_pf, 3),
                       "kv_strategy": ["exit river", "state propagation", "mono-decreasing exit", "kv mask"][args.kv_strategy],
                       **({"offload": {"first_offloaded_layer": args.offload_from, "device_bytes_saved": off_saved,
                                       "block_copies_per_step": (off_fetches - off_fetches0) / K}}
                          if args.offload_from else {})},
            "layers_executed_fraction": float(ex.mean() / L), "early_exit_fraction": float((ex < L).mean()),
            "mean_exit_layer": float(ex.mean()),
            "alg_bytes_per_step": bytes_exit,
            "hbm_roofline_step": {"achieved_GBps": step_gbs, "frac_of_measured_peak": step_gbs / peak,
                                  "frac_of_8TBps": step_gbs / 8000.0, "peak_GBps": peak, "peak_kind": peak_kind},
            "full_depth": {"tokens_per_s": world * B * K / (ms_full / 1e3), "ms_per_step": ms_full / K,
                           "alg_bytes_per_step": bytes_full, "achieved_GBps": full_gbs,
                           "frac_of_measured_peak": full_gbs / peak, "frac_of_8TBps": full_gbs / 8000.0},
            "early_exit_speedup_vs_full_depth": ms_full / ms,
            "roofline": {"bound": "hbm", "kernel": dom["name"], "achieved": ach, "peak": peak, "unit": "GB/s",
                         "frac": ach / peak,
                         "traffic": NCU_TRAFFIC.get((shape_name, dom["name"])),
                         "peak_kind": peak_kind,
                         "launch_ms": per_launch_ms, "alg_bytes_per_launch": dom["alg_bytes_total"] / dom["launches"],
                         "pass": "full depth, events around every launch"},
            "kernels": kernels,
            "kernels_exit_run": kernels_exit,
            "e2e": {"value": world * B * n_e2e / (ms_e2e / 1e3), "unit": "tokens/s", "steps": n_e2e,
                    "h2d_bytes_per_step": B * 8, "d2h_bytes_per_step": B * (4 * shape.V + 8)},
            "gpu_launches": int(launches),
            "clocks": clk.summary(),
            "device_error": st.device_error,
        }
    # ---- the oracle on the host cores, rank 0 at N = 1 only
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        to_cpu = lambda x: x.cpu() if isinstance(x, torch.Tensor) else (
            {k: to_cpu(v) for k, v in x.items()} if isinstance(x, dict) else type(x)(to_cpu(v) for v in x))
        Bs = min(B, 2)
        n_or = 12 if shape_name == "8b" else 24
        r = time_oracle(shape, to_cpu(bb), to_cpu(rvw), Bs, int(np.mean(pos0)), n_or, 1, WORKLOADS[wl][3])
        line["cpu_baseline"] = {
            "value": r["tokens_per_s"], "unit": "tokens/s", "cores": r["threads"], "kind": "oracle",
            "sample": f"{n_or} oracle decode steps after 1 warm-up, {Bs} of {B} rows, {shape_name} shape, context "
                      f"{int(np.mean(pos0))} (synthetic N(0,1) KV history), exits forced at the scheduled layers"}
    if rank == 0 and "cpu_baseline" not in line:
        line["cpu_baseline"] = None
    stream_ctx.__exit__(None, None, None)
    rv.close()
    if rank == 0:
        print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- attention microbenchmark
def attn_micro(args):
    """Exit-aware decode-attention microbenchmark (8B-class GQA geometry: 32/8 heads, head dim 128, bf16 cache).

    For every (context, batch, skip density) point the rows of the batch get exit layers drawn (seed 4) so that the
    mean share of bypassed blocks equals the skip density; masks are sticky in depth.  Per block l three pieces are
    timed with CUDA events through the library's single-stage entry points and summed over the blocks:
      M1  attention over the compacted rows still in the backbone (river_attention on A_l),
      M2  exit-layer K/V generation + RoPE + paged cache write for the rows that left it (river_project_kv on R_l),
      M3  attention of those rows (river_attention on R_l): an exit layer is a whole block, so they attend too.
    The method's total is M1 + M2 + M3; M1 + M2 alone would be a K/V-only exit path.  Prints one JSON line."""
    import ctypes
    import dataclasses
    from paper_2604_18396_b200 import River, buildlib, make_config
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    buildlib.build()
    dev = torch.device("cuda", 0)
    peak, peak_kind = peaks()
    shape0 = synth.SHAPES["8b"]
    contexts = [int(x) for x in args.micro_contexts.split(",")]
    batches = [int(x) for x in args.micro_batches.split(",")]
    densities = [float(x) for x in args.micro_densities.split(",")]
    pool_cap = args.micro_pool_gib * 2 ** 30
    kv_tok_layer = 2 * shape0.Hkv * shape0.dh * 2  # bytes of K+V per token and block
    qkv_rows = (shape0.Hq + 2 * shape0.Hkv) * shape0.dh
    w4_qkv_bytes = qkv_rows * shape0.d * (0.5 + 4.0 / shape0.group)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    results = []
    models = {}
    for ctx in contexts:
        for B in batches:
            per_layer = B * (ctx + 16) * kv_tok_layer
            L = int(max(1, min(shape0.L, pool_cap // per_layer)))
            shape = dataclasses.replace(shape0, L=L)
            if L not in models:
                models.clear()
                torch.cuda.empty_cache()
                models[L] = draw_model(shape, dev)
            bb, rvw = models[L]
            pages_per_seq = (ctx + 15) // 16
            cfg = make_config(shape, max_seqs=B, max_pages_per_seq=pages_per_seq, n_pages=B * pages_per_seq,
                              max_batch=max(B, 8), page_shuffle_seed=5, flags=0)
            rv = River(cfg, bb, rvw)
            with torch.cuda.stream(rv.stream):
                w = shape.Hkv * shape.dh
                z = torch.zeros((ctx, w), dtype=torch.bfloat16, device=dev)
                for b in range(B):
                    rv.write_kv(b, 1, 0, z, z)  # allocates the row's pages and sets its length
                del z
                flat = rv.kv_pool.view(-1)
                for i0 in range(0, flat.numel(), 1 << 30):  # N(0,1) bf16 everywhere: every block's K and V
                    flat[i0:i0 + (1 << 30)].normal_()
                q = torch.randn((B, shape.Hq * shape.dh), device=dev)
                h = torch.randn((B, shape.d), device=dev)
                out = torch.empty_like(q)
                torch.cuda.synchronize()
                for dens in densities:
                    # exit layer per row: mean (L - e) / L = dens, e in [1, L]; rows with e = L never leave
                    u = synth.uniform_int(4, int(1000 * dens) + 7 * B + ctx, B, 0, 10 ** 6).numpy() / 1e6
                    frac_left = u ** ((1.0 - dens) / dens) if dens > 0 else np.zeros(B)  # mean dens: E[u^k] = 1 / (k + 1)
                    depth_left = np.clip(np.round(frac_left * shape0.L), 0, shape0.L - 1)
                    e_rel = 1.0 - depth_left / shape0.L
                    t = {"M1": 0.0, "M2": 0.0, "M3": 0.0}
                    by = {"M1": 0.0, "M2": 0.0, "M3": 0.0}
                    n_riv_total = 0
                    for rep in range(2):  # first pass warms up (launch geometry, attributes), second is timed
                        for l in range(1, L + 1):
                            rel = l / L
                            riv = [b for b in range(B) if e_rel[b] < rel - 1e-9]
                            act = [b for b in range(B) if not e_rel[b] < rel - 1e-9]
                            pieces = (("M1", act), ("M2", riv), ("M3", riv))
                            for name, rows in pieces:
                                if not rows:
                                    continue
                                if per_layer < (256 << 20):
                                    flush.zero_()  # the block's cache would otherwise sit in the L2 from the last pass
                                sc = (ctypes.c_int32 * len(rows))(*rows)
                                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                                e0.record()
                                if name == "M2":
                                    rv.project_kv(l, True, rows, h[:len(rows)], None, slots_c=sc)
                                else:
                                    rv.attention(l, rows, q[:len(rows)], out[:len(rows)], slots_c=sc)
                                e1.record()
                                if rep == 1:
                                    torch.cuda.synchronize()
                                    t[name] += e0.elapsed_time(e1) * 1e-3
                                    by[name] += (w4_qkv_bytes + len(rows) * kv_tok_layer) if name == "M2" else \
                                        len(rows) * ctx * kv_tok_layer
                                    if name == "M2":
                                        n_riv_total += len(rows)
                    tot_t, tot_b = sum(t.values()), sum(by.values())
                    results.append({
                        "context": ctx, "batch": B, "skip_density": dens, "blocks": L,
                        "achieved_skip": n_riv_total / (B * L),
                        "us_per_block": {k: round(1e6 * v / L, 2) for k, v in t.items()},
                        "us_per_block_sum": round(1e6 * tot_t / L, 2),
                        "GBps": {k: (round(by[k] / t[k] / 1e9, 1) if t[k] > 0 else None) for k in t},
                        "frac_of_peak_sum": round(tot_b / tot_t / 1e9 / peak, 4) if tot_t > 0 else None,
                        "frac_of_peak_attention": round((by["M1"] + by["M3"]) / max(t["M1"] + t["M3"], 1e-12) / 1e9 / peak, 4),
                    })
                st = rv.stats()
                assert st.device_error == 0, st.device_error
            rv.close()
            del rv
            torch.cuda.empty_cache()
    line = {"metric": "exit_aware_decode_attention", "unit": "us per block (M1 + M2 + M3)", "n_gpus": 1, "dtype": "bf16",
            "data": "synthetic", "peak_GBps": peak, "peak_kind": peak_kind,
            "config": {"workload": "attn_micro", "shape": "8b (32/8 heads, head dim 128, 16-token pages)",
                       "contexts": contexts, "batches": batches, "skip_densities": densities, "seed": 4,
                       "pool_cap_GiB": args.micro_pool_gib,
                       "l2": "cache of a block flushed from the L2 before each timed call when it is below 256 MB",
                       "timing": "CUDA events around each single-stage call (metadata upload + kernels)"},
            "points": results}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8b_b1", choices=sorted(WORKLOADS) + ["attn_micro"])
    ap.add_argument("--micro-contexts", default="1024,8192,32768")
    ap.add_argument("--micro-batches", default="1,16,128")
    ap.add_argument("--micro-densities", default="0,0.2,0.4,0.6,0.8")
    ap.add_argument("--micro-pool-gib", type=int, default=64, help="attn_micro: cap of the KV pool (fewer blocks are run when a point needs more)")
    ap.add_argument("--flags", type=int, default=1, help="river_config.flags (1 = CUDA-graph replay)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kv-strategy", type=int, default=0, choices=[0, 1, 2, 3],
                    help="what a skipped block does: 0 = the 4-bit exit river (the method), 1 = State Propagation, "
                         "2 = Mono-Decreasing Exit, 3 = KV Mask (river_config.kv_strategy)")
    ap.add_argument("--offload-from", type=int, default=0,
                    help="keep backbone blocks >= this layer in pinned host memory (river_offload); 0 = all resident")
    ap.add_argument("--layers", type=int, default=0, help="profiling aid: keep only the first N layers of the shape")
    ap.add_argument("--prompt", type=int, default=0, help="profiling aid: override the prompt length")
    ap.add_argument("--batch", type=int, default=0, help="profiling aid: override the row count (attention sweeps)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.workload == "attn_micro":
        attn_micro(args)
    elif args.impl == "reference":
        reference_arm(args, args.workload)
    else:
        ours(args, args.workload)


if __name__ == "__main__":
    main()

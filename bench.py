#!/usr/bin/env python
"""Benchmark of the STEM FFN layer hot path on B200.

One step = dedup of the batch's token ids + forward + backward of one layer (all steps of
the path) on one batch of synthetic input.  Prints ONE JSON line (rank 0).

    python bench.py --gpus 1 --steps 30 --warmup 5
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference ...        # the CPU checker, timed on the host cores

N > 1 runs N independent replicas (the path has no exchange step): every rank processes
its own batch, no data-path collective; the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2601_10639_b200 import synth  # noqa: E402

METRIC = "STEM-FFN fwd+bwd tokens/sec (1B-class layer, dedup + forward + backward)"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def layer_flops(T: int, d: int, F: int, backward: bool) -> float:
    """FLOPs (2 per multiply-accumulate) the layer's contractions perform on T tokens: two d x d_ff
    products per token forward (the up-projection STEM removes is not counted: paper Table 1),
    and twice that again backward (each forward product has a data and a weight gradient)."""
    return (12.0 if backward else 4.0) * T * d * F


def rank_seed(seed: int, rank: int) -> int:
    """Every rank is an independent replica with its own batch: same shapes, different draws."""
    return seed + rank


def max_over_ranks(values, device):
    """Element-wise maximum over the ranks of a list of floats (multi-GPU times are the slowest rank's)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        out = {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
        under = (d.get("clocks_under_load") or {}).get("sm_mhz_median")
        if under:
            out["sm_mhz_under_load"] = float(under)
        return out
    return dict(FALLBACK_PEAKS, source="fallback")


def source_digest(files) -> str:
    """Short digest of kernel sources: ties stored DRAM counters to the code they were taken from."""
    import hashlib
    h = hashlib.sha256()
    for name in files:
        with open(os.path.join(ROOT, "paper_2601_10639_b200", "csrc", name), "rb") as f:
            text = f.read()
        # device code only: the launch code after this marker does not change what a kernel moves
        h.update(text.split(b"// ---- host side", 1)[0])
    return h.hexdigest()[:12]


def load_traffic(step: str):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum, one ncu capture) of the
    kernel behind `step`, scaled to this workload's launch; None when no capture is stored or the
    kernel's source has changed since it was taken.  File lines: step tokens_captured bytes digest."""
    p = os.path.join(ROOT, "profiles", "ncu_traffic.txt")
    if not os.path.exists(p):
        return None
    digest = source_digest(["gemm_sm100.cu", "ptx_sm100.cuh"] if step.endswith("_gemm") else ["segreduce.cu"])
    for line in open(p):
        parts = line.split()
        if len(parts) >= 4 and not line.startswith("#") and parts[0] == step and parts[3] == digest:
            return int(parts[1]), float(parts[2])
    return None


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while a region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def __exit__(self, *exc):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, t0: float, t1: float) -> dict:
        sm, mx, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        rows = [l for (t, l) in self.lines if t0 - 0.05 <= t <= t1 + 0.2] or [l for (_, l) in self.lines]
        for line in rows:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": max(mx), "power_w_max": max(power),
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_tokens_per_sec(inputs: dict, Tc: int) -> tuple[float, float]:
    """Time the CPU checker (as it stands) on the first Tc tokens of the batch."""
    from oracle import stem_oracle as O
    sl = {k: (v[:Tc] if k in ("x", "dy", "ids") else v) for k, v in inputs.items()}
    t = time.perf_counter()
    O.dedup(sl["ids"])
    O.forward(sl["x"], sl["ids"], sl["W_gate"], sl["E"], sl["W_down"])
    O.backward(sl["dy"], sl["x"], sl["ids"], sl["W_gate"], sl["E"], sl["W_down"])
    dt = time.perf_counter() - t
    return Tc / dt, dt


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, w):
    """The CPU checker as the reference arm: rank 0 only, bounded token sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    Tc = args.ref_tokens
    inputs = synth.make_inputs(w, T=Tc)
    for _ in range(args.warmup):
        oracle_tokens_per_sec(inputs, Tc)
    t = time.perf_counter()
    for _ in range(args.steps):
        oracle_tokens_per_sec(inputs, Tc)
    dt = time.perf_counter() - t
    value = Tc * args.steps / dt
    sample = f"first {Tc} tokens of the batch per step (every stage is linear in T), all weights and the full table"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "T": w.T, "d_model": w.d_model, "d_ff": w.d_ff, "V": w.V, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_host_stack(args, w, steps=None, warmup=None):
    """Workload with the tables of a stack of independent layers in pinned host memory: a step is
    forward + backward of every layer, rows prefetched and gradient rows written back on side
    streams.  Reports tokens/s (all layers) and the exposed copy time: the time of the same stack
    with device-resident tables subtracted from the host-table time."""
    import torch
    from paper_2601_10639_b200 import binding as B
    from paper_2601_10639_b200 import runner

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    B.lib()
    dt = torch.bfloat16
    steps = args.steps if steps is None else steps
    warmup = args.warmup if warmup is None else warmup
    T, d, F, V, L = (args.tokens or w.T), w.d_model, w.d_ff, w.V, w.layers
    gcode = B.DTYPE_BF16 if args.grad_bf16 else B.DTYPE_FP32
    gen = torch.Generator(device=dev).manual_seed(args.seed)
    shape = B.make_shape(T, d, F, V, B.DTYPE_BF16, gcode, 0)
    W_gate = (torch.randn(F, d, generator=gen, device=dev) * d ** -0.5).to(dt)
    W_down = (torch.randn(d, F, generator=gen, device=dev) * F ** -0.5).to(dt)
    xs = [torch.randn(T, d, generator=gen, device=dev).to(dt) for _ in range(L)]
    dys = [torch.randn(T, d, generator=gen, device=dev).to(dt) for _ in range(L)]
    idss = [torch.from_numpy(synth.token_ids(args.seed, T, V, w.id_dist, layer=l)).to(dev) for l in range(L)]
    dev_tables, host_tables = [], []
    for l in range(L):
        E = torch.empty(V, F, device=dev, dtype=dt)
        for r0 in range(0, V, 4096):
            r1 = min(V, r0 + 4096)
            E[r0:r1] = (torch.randn(r1 - r0, F, generator=gen, device=dev) * 0.02).to(dt)
        dev_tables.append(E)
        h = torch.empty(V, F, dtype=dt).pin_memory()
        h.copy_(E)
        host_tables.append(h)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    results = {}
    for name, resident in (("resident", True), ("host", False)):
        stack = runner.HostTableStack(shape, L, dev_tables if resident else host_tables, W_gate, W_down, resident)
        for _ in range(warmup):
            stack.step(xs, idss, dys)
        stack.finish()
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = B.stem_launch_count()
        with ClockSampler(0) as clocks:
            t0 = time.time()
            ev0.record(stream)
            for _ in range(steps):
                stack.step(xs, idss, dys)
            stack.finish()
            ev1.record(stream)
            torch.cuda.synchronize()
            t1 = time.time()
        assert B.stem_query_status(stack.ws) == B.OK
        results[name] = {"ms": ev0.elapsed_time(ev1) / steps, "launches": B.stem_launch_count() - l0,
                         "clocks": clocks.summary(t0, t1),
                         "n_unique": [int(k["n_unique"].item()) for k in stack.slots]}
        if not resident:
            k = stack.slots[(L - 1) % 3]
            n = int(k["host_n"][0])
            assert n == int(k["n_unique"].item())
            assert torch.equal(k["host_rows"][:n], k["dE_rows"][:n].cpu())      # what reached the host is the gradient
        del stack

    # ---- the host link by itself: plain pinned copies (the denominator), then the row movers alone
    def timed(fn, n=5):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n
    nbytes = 256 << 20
    hbuf = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    dbuf = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    link = {"h2d_gbs": nbytes / timed(lambda: dbuf.copy_(hbuf, non_blocking=True)) / 1e6,
            "d2h_gbs": nbytes / timed(lambda: hbuf.copy_(dbuf, non_blocking=True)) / 1e6}
    probe = runner.HostTableStack(shape, L, host_tables, W_gate, W_down, False)
    k = probe.slots[0]
    B.stem_dedup_ids(shape, idss[0], k["unique_ids"], k["n_unique"], k["inverse"], k["perm"], k["seg_offsets"], probe.ws)
    n0 = int(k["n_unique"].item())
    gsz = 2 if args.grad_bf16 else 4
    t_pf = timed(lambda: B.stem_prefetch_rows(shape, k["unique_ids"], k["n_unique"], host_tables[0], k["cache"], probe.ws))
    t_wb = timed(lambda: B.stem_writeback_rows(shape, k["dE_rows"], k["unique_ids"], k["n_unique"], k["host_rows"],
                                               k["host_ids"], k["host_n"]))
    t_dma = timed(lambda: B.stem_writeback_rows_dma(shape, k["dE_rows"], k["unique_ids"], n0, k["host_rows"], k["host_ids"]))
    link.update(prefetch_rows_gbs=n0 * F * 2 / t_pf / 1e6, writeback_rows_kernel_gbs=n0 * F * gsz / t_wb / 1e6,
                writeback_rows_dma_gbs=n0 * F * gsz / t_dma / 1e6, prefetch_rows_ms=t_pf, writeback_rows_dma_ms=t_dma)
    del probe
    host_ms, res_ms = results["host"]["ms"], results["resident"]["ms"]
    n_u = float(np.mean(results["host"]["n_unique"]))
    peaks = load_peaks()
    tf = 12.0 * L * T * d * F / (host_ms * 1e-3) / 1e12
    return {
        "metric": METRIC, "value": L * T / (host_ms * 1e-3), "unit": "tokens/s", "n_gpus": 1, "steps": steps,
        "warmup": warmup, "ms_per_step": host_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "layers": L, "T": T, "d_model": d, "d_ff": F, "V": V, "ids": w.id_dist,
                   "tables": "pinned host memory, one per layer", "grad_dtype": "bf16" if args.grad_bf16 else "f32",
                   "l2": "working set exceeds L2; no flush"},
        "gpu_launches": int(results["host"]["launches"]), "clocks": results["host"]["clocks"], "tflops_step": tf,
        "host_tables": {"ms_per_step": host_ms, "ms_per_layer": host_ms / L},
        "device_tables": {"ms_per_step": res_ms, "ms_per_layer": res_ms / L, "clocks": results["resident"]["clocks"]},
        "exposed_copy_ms_per_step": host_ms - res_ms, "exposed_copy_ms_per_layer": (host_ms - res_ms) / L,
        "host_link": link, "rows_prefetched_per_layer": n_u, "prefetch_bytes_per_layer": n_u * F * 2,
        "writeback_bytes_per_layer": n_u * F * gsz,
        "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                     "frac": tf / peaks["bf16_tflops_sustained"], "traffic": None,
                     "peak_source": peaks["source"] + " (sustained bf16 GEMM, of measured)",
                     "kernel": "whole step (six contractions per layer)"},
    }


def run_prefill_stack(args, w):
    """Forward-only pass of one long sequence through a stack of layers with host-resident tables:
    ids deduplicated once, rows prefetched a layer ahead, with and without an on-device hot set."""
    import torch
    from paper_2601_10639_b200 import binding as B
    from paper_2601_10639_b200 import runner

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    B.lib()
    dt = torch.bfloat16
    T, d, F, V, L = (args.tokens or w.T), w.d_model, w.d_ff, w.V, w.layers
    gen = torch.Generator(device=dev).manual_seed(args.seed)
    shape = B.make_shape(T, d, F, V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    W_gate = (torch.randn(F, d, generator=gen, device=dev) * d ** -0.5).to(dt)
    W_down = (torch.randn(d, F, generator=gen, device=dev) * F ** -0.5).to(dt)
    xs = [torch.randn(T, d, generator=gen, device=dev).to(dt) for _ in range(L)]
    ids_np = synth.token_ids(args.seed, T, V, w.id_dist)
    ids = torch.from_numpy(ids_np).to(dev)
    dev_tables, host_tables = [], []
    for l in range(L):
        E = torch.empty(V, F, device=dev, dtype=dt)
        for r0 in range(0, V, 4096):
            r1 = min(V, r0 + 4096)
            E[r0:r1] = (torch.randn(r1 - r0, F, generator=gen, device=dev) * 0.02).to(dt)
        dev_tables.append(E)
        h = torch.empty(V, F, dtype=dt).pin_memory()
        h.copy_(E)
        host_tables.append(h)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    uniq = np.unique(ids_np)
    n_u = int(uniq.size)
    results = {}
    # hot sets: the K most frequent ids of the token distribution (ids are frequency-ranked, so 0..K-1)
    modes = [("resident", None), ("host", None)] + [(f"host+hot{K}", K) for K in args.hot_rows]
    for name, K in modes:
        hot = None
        if K:
            hot = [runner.build_hot_set(t, torch.arange(0, K)) for t in host_tables]
        stack = runner.HostTablePrefill(shape, L, dev_tables if name == "resident" else host_tables, W_gate, W_down,
                                        name == "resident", hot)
        for _ in range(args.warmup):
            stack.run(xs, ids)
        torch.cuda.synchronize()
        stack.stats.zero_()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(0) as clocks:
            t0 = time.time()
            ev0.record(stream)
            for _ in range(args.steps):
                stack.run(xs, ids)
            ev1.record(stream)
            torch.cuda.synchronize()
            t1 = time.time()
        assert B.stem_query_status(stack.ws) == B.OK and int(stack.n_unique.item()) == n_u
        ms = ev0.elapsed_time(ev1) / args.steps
        r = {"ms_per_step": ms, "ms_per_layer": ms / L, "clocks": clocks.summary(t0, t1)}
        if K:
            hits, misses = stack.stats.tolist()
            assert hits + misses == args.steps * L * n_u
            r.update(hot_rows=K, hot_bytes_per_layer=K * F * 2, unique_row_hit_rate=hits / (hits + misses),
                     token_hit_rate=float((ids_np < K).mean()), rows_over_link_per_layer=misses / (args.steps * L))
        results[name] = r
        del stack, hot
    res_ms = results["resident"]["ms_per_step"]
    for name, r in results.items():
        r["exposed_copy_ms_per_layer"] = (r["ms_per_step"] - res_ms) / L
    best = min((r["ms_per_step"], n) for n, r in results.items() if n != "resident")[1]
    ms = results[best]["ms_per_step"]
    peaks = load_peaks()
    tf = layer_flops(T, d, F, False) * L / (ms * 1e-3) / 1e12
    print(json.dumps({
        "metric": "STEM-FFN forward tokens/sec (prefill through a stack with host-resident tables)",
        "value": L * T / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": w.name, "layers": L, "T": T, "d_model": d, "d_ff": F, "V": V, "ids": w.id_dist,
                   "n_unique": n_u, "reported_mode": best, "l2": "working set exceeds L2; no flush"},
        "clocks": results[best]["clocks"], "tflops_step": tf, "modes": results,
        "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                     "frac": tf / peaks["bf16_tflops_sustained"], "traffic": None,
                     "peak_source": peaks["source"] + " (sustained bf16 GEMM, of measured)",
                     "kernel": "whole pass (two contractions per layer)"},
    }))


def run_decode(args, w):
    """Decode steps with the table in host memory and a frequency-ranked row cache on the device
    (paper Section 3.4; Table 1, decoding: communication B_uniq * d_ff per step).  A step = count
    the lookups, deduplicate the step's ids, gather their rows (cache or host link), forward."""
    import torch
    from paper_2601_10639_b200 import binding as B
    from paper_2601_10639_b200 import runner

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    B.lib()
    dt = torch.bfloat16
    Bt, d, F, V = (args.tokens or w.T), w.d_model, w.d_ff, w.V
    steps, refresh_every = max(args.steps, 400), 20
    gen = torch.Generator(device=dev).manual_seed(args.seed)
    shape = B.make_shape(Bt, d, F, V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    cshape = B.make_shape(Bt, d, F, min(Bt, V), B.DTYPE_BF16, B.DTYPE_FP32, 0)
    W_gate = (torch.randn(F, d, generator=gen, device=dev) * d ** -0.5).to(dt)
    W_down = (torch.randn(d, F, generator=gen, device=dev) * F ** -0.5).to(dt)
    x = torch.randn(Bt, d, generator=gen, device=dev).to(dt)
    E = torch.empty(V, F, device=dev, dtype=dt)
    for r0 in range(0, V, 4096):
        r1 = min(V, r0 + 4096)
        E[r0:r1] = (torch.randn(r1 - r0, F, generator=gen, device=dev) * 0.02).to(dt)
    table = torch.empty(V, F, dtype=dt).pin_memory()
    table.copy_(E)
    del E
    all_ids = torch.from_numpy(synth.token_ids(args.seed, steps * Bt, V, w.id_dist)).to(dev)   # every step's ids
    st = runner.LayerState(shape, device=dev).allocate(backward=False)
    st.x, st.W_gate, st.W_down = x, W_gate, W_down
    b = st.bufs
    cache = torch.empty(min(Bt, V), F, dtype=dt, device=dev)
    stream = torch.cuda.current_stream()
    out = {}
    for K in args.hot_rows:
        freq = torch.zeros(V, dtype=torch.int32, device=dev)
        hot_slot = torch.full((V,), -1, dtype=torch.int32, device=dev)
        hot_ids = torch.full((K,), -1, dtype=torch.int32, device=dev)
        hot_rows = torch.zeros(K, F, dtype=dt, device=dev)
        stats, rows = torch.zeros(2, dtype=torch.int32, device=dev), torch.zeros(2, dtype=torch.int32, device=dev)
        n_inst = torch.zeros(1, dtype=torch.int32, device=dev)
        lws = torch.empty(B.stem_lfu_workspace_bytes(V, K), dtype=torch.uint8, device=dev)

        def step(i):
            ids = all_ids[i * Bt:(i + 1) * Bt]
            B.stem_lfu_touch(Bt, V, ids, freq, hot_slot, stats)
            B.stem_dedup_ids(shape, ids, b["unique_ids"], b["n_unique"], b["inverse"], b["perm"], b["seg_offsets"], b["ws"])
            B.stem_prefetch_rows_hot(shape, b["unique_ids"], b["n_unique"], table, hot_rows, hot_slot, cache, rows, b["ws"])
            B.stem_ffn_forward(cshape, x, b["inverse"], W_gate, cache, W_down, b["y"], None, None, b["ws"])
            if i % refresh_every == refresh_every - 1:
                B.stem_lfu_refresh(shape, K, freq, hot_slot, hot_ids, hot_rows, table, n_inst, lws)

        half = steps // 2
        for i in range(half):                       # warm the counters and the cache
            step(i)
        torch.cuda.synchronize()
        stats.zero_(); rows.zero_()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for i in range(half, steps):
            step(i)
        ev1.record(stream)
        torch.cuda.synchronize()
        assert st.status() == B.OK
        hits, misses = stats.tolist()
        rhit, rmiss = rows.tolist()
        n = steps - half
        out[f"hot{K}"] = {"hot_rows": K, "hot_bytes": K * F * 2, "token_hit_rate": hits / (hits + misses),
                          "unique_row_hit_rate": rhit / (rhit + rmiss), "unique_rows_per_step": (rhit + rmiss) / n,
                          "rows_over_link_per_step": rmiss / n, "link_bytes_per_step": rmiss / n * F * 2,
                          "ms_per_step": ev0.elapsed_time(ev1) / n, "refresh_every_steps": refresh_every}
    # the same step with the table on the device (no cache, no link): the compute floor of this path
    dev_table = table.to(dev)
    def resident_step(i):
        ids = all_ids[i * Bt:(i + 1) * Bt]
        B.stem_ffn_forward(shape, x, ids, W_gate, dev_table, W_down, b["y"], None, None, b["ws"])
    for i in range(20):
        resident_step(i)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for i in range(200):
        resident_step(i)
    ev1.record(stream)
    torch.cuda.synchronize()
    res_ms = ev0.elapsed_time(ev1) / 200

    # The same two loops replayed from CUDA graphs: a decode step is a handful of short launches,
    # so how fast the host can issue them is part of the eager figures above.  The step's ids are
    # copied into a fixed buffer before each replay; the cache refresh stays outside the graph.
    def replay_ms(body, n, before=None):
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(3):
                body()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            body()
        for i in range(10):
            if before:
                before(i)
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n):
            if before:
                before(i)
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    ids_now = all_ids[:Bt].clone()
    res_graph_ms = replay_ms(lambda: B.stem_ffn_forward(shape, x, ids_now, W_gate, dev_table, W_down, b["y"], None, None,
                                                       b["ws"]), 200)

    def graph_body():
        B.stem_lfu_touch(Bt, V, ids_now, freq, hot_slot, stats)
        B.stem_dedup_ids(shape, ids_now, b["unique_ids"], b["n_unique"], b["inverse"], b["perm"], b["seg_offsets"], b["ws"])
        B.stem_prefetch_rows_hot(shape, b["unique_ids"], b["n_unique"], table, hot_rows, hot_slot, cache, rows, b["ws"])
        B.stem_ffn_forward(cshape, x, b["inverse"], W_gate, cache, W_down, b["y"], None, None, b["ws"])

    half = steps // 2
    step_graph_ms = replay_ms(graph_body, steps - half, lambda i: ids_now.copy_(all_ids[(half + i) * Bt:(half + i + 1) * Bt]))
    assert st.status() == B.OK
    best = min(out.values(), key=lambda r: r["ms_per_step"])
    peaks = load_peaks()
    wbytes = 2 * d * F * 2
    print(json.dumps({
        "metric": "STEM-FFN decode steps: tokens/sec of one layer with a host-resident table and an LFU row cache",
        "value": Bt / (best["ms_per_step"] * 1e-3), "unit": "tokens/s", "n_gpus": 1, "steps": steps - steps // 2,
        "warmup": steps // 2, "ms_per_step": best["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "tokens_per_step": Bt, "d_model": d, "d_ff": F, "V": V, "ids": w.id_dist,
                   "paper_hit_rate": "> 80 % (Section 3.4, hardware and cache size not stated)"},
        "modes": out, "device_table_forward_ms": res_ms,
        "cuda_graph": {"device_table_forward_ms": res_graph_ms, "step_ms": step_graph_ms, "hot_rows": args.hot_rows[-1],
                       "tokens_per_s": Bt / (step_graph_ms * 1e-3),
                       "note": "the step (count, dedup, gather, forward) captured once and replayed; ids copied in before each replay"},
        "roofline": {"bound": "hbm", "achieved": wbytes / (res_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": wbytes / (res_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                     "kernel": "forward with a device table (both weight matrices read once per step: 2 d d_ff elements, Table 1)",
                     "peak_source": peaks["source"] + " (copy bandwidth, of measured)"},
    }))


def run_unique_growth(args):
    """Distinct table rows touched as a function of context length (paper Section 3.2.5: the STEM
    parameters a sequence activates are |S| d_ff L_uniq, and L_uniq grows sublinearly): one sequence
    of L positions with the long-context id mix, deduplicated on the GPU, L = 4k ... 128k."""
    import torch
    from paper_2601_10639_b200 import binding as B
    from paper_2601_10639_b200 import runner

    torch.cuda.set_device(0)
    w = synth.WORKLOADS["1b_long_fwd"]
    rows = []
    for L in (4096, 8192, 16384, 32768, 65536, 131072):
        ids = synth.token_ids(args.seed, L, w.V, w.id_dist)
        st = runner.LayerState(B.make_shape(L, 8, 8, w.V, B.DTYPE_BF16, B.DTYPE_FP32, 0)).allocate(backward=False)
        st.ids = torch.from_numpy(ids).cuda()
        for _ in range(3):
            st.dedup()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            st.dedup()
        e1.record()
        torch.cuda.synchronize()
        n_u = int(st.bufs["n_unique"].item())
        assert n_u == len(np.unique(ids)) and st.status() == B.OK
        rows.append({"L": L, "unique_rows": n_u, "unique_fraction": n_u / L, "dedup_us": 1e3 * e0.elapsed_time(e1) / 20,
                     "row_bytes_per_layer": n_u * w.d_ff * 2})
    print(json.dumps({"metric": "distinct table rows touched vs context length", "unit": "rows", "data": "synthetic",
                      "config": {"workload": "unique_growth", "V": w.V, "d_ff": w.d_ff, "ids": w.id_dist}, "rows": rows}))


def run_sharded(args, w):
    """The layer with its table sharded over G ranks (paper Section 3.4, "parallel embeddings"),
    as G virtual ranks stepped in lock step on one GPU: the device time each step of a rank's
    path takes, and the bytes its exchanges would carry.  The exchange itself is slice copies
    here; its time over NVLink is projected, not measured."""
    import torch
    from paper_2601_10639_b200 import binding as B
    from paper_2601_10639_b200 import runner, sharded

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    B.lib()
    G = args.shard_ranks
    dt = torch.bfloat16
    T, d, F, V = (args.tokens or w.T), w.d_model, w.d_ff, w.V
    gen = torch.Generator(device=dev).manual_seed(args.seed)
    shape = B.make_shape(T, d, F, V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    W_gate = (torch.randn(F, d, generator=gen, device=dev) * d ** -0.5).to(dt)
    W_down = (torch.randn(d, F, generator=gen, device=dev) * F ** -0.5).to(dt)
    E = torch.empty(V, F, device=dev, dtype=dt)
    for r0 in range(0, V, 4096):
        r1 = min(V, r0 + 4096)
        E[r0:r1] = (torch.randn(r1 - r0, F, generator=gen, device=dev) * 0.02).to(dt)
    ranks = [sharded.ShardedRank(r, G, shape, E[r::G].contiguous(), W_gate, W_down, device=dev) for r in range(G)]
    xs = [torch.randn(T, d, generator=gen, device=dev).to(dt) for _ in range(G)]
    dys = [torch.randn(T, d, generator=gen, device=dev).to(dt) for _ in range(G)]
    idss = [torch.from_numpy(synth.token_ids(rank_seed(args.seed, r), T, V, w.id_dist)).to(dev) for r in range(G)]
    ex = sharded.LocalExchange(G)
    steps = min(args.steps, 20)
    for _ in range(3):
        sharded.step_local(ranks, ex, xs, idss, dys)
    torch.cuda.synchronize()
    launches0 = B.stem_launch_count()
    events = []

    def timed(name, fn):      # CUDA events around one rank's phase: the exchange's copies stay outside
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = fn()
        e1.record()
        events.append((name, e0, e1))
        return out

    t0 = time.perf_counter()
    for _ in range(steps):
        owned = sharded.step_local(ranks, ex, xs, idss, dys, timed)
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    assert all(r.status() == B.OK for r in ranks)
    per_rank_step = {}
    for name, e0, e1 in events:
        per_rank_step[name] = per_rank_step.get(name, 0.0) + e0.elapsed_time(e1) / (steps * G)
    # route = dedup + requests (+ the count read-back); serve = the owner's gather; layer = forward,
    # backward and the gradient rows put in request order; reduce = the owner's dedup + per-row sums
    layer = per_rank_step["layer"]
    extra = per_rank_step["route"] + per_rank_step["serve"] + per_rank_step["reduce"]
    n_u = sum(r.h_send_counts[g] for r in ranks for g in range(G)) / G
    remote = sum(r.h_send_counts[g] for r in ranks for g in range(G) if g != r.rank) / G
    fwd_bytes, bwd_bytes = remote * F * 2, remote * F * 4
    nvlink_gbs = 770.0
    print(json.dumps({
        "metric": "STEM-FFN fwd+bwd with the table sharded over G ranks: device time per rank per step",
        "value": T / ((layer + extra) * 1e-3), "unit": "tokens/s per rank (exchange time excluded)",
        "n_gpus": 1, "virtual_ranks": G, "steps": steps, "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "tokens_per_rank": T, "d_model": d, "d_ff": F, "V": V, "ids": w.id_dist,
                   "rows_by": "id mod G", "exchange": "in-process slice copies (one GPU); NVLink time projected"},
        "ms_per_rank_step": {"layer": layer, "route_serve_reduce": extra, **per_rank_step},
        "distinct_rows_per_rank": n_u, "rows_from_other_ranks": remote,
        "exchange_bytes_per_rank": {"rows_in": fwd_bytes, "grad_rows_out_fp32": bwd_bytes},
        "projected_exchange_ms_at_770GBs": {"rows_in": fwd_bytes / nvlink_gbs / 1e6, "grad_rows_out": bwd_bytes / nvlink_gbs / 1e6},
        "owner_rows_reduced": [int(o[1].item()) for o in owned],
        "gpu_launches": B.stem_launch_count() - launches0, "wall_ms_per_step_all_ranks": wall / steps * 1e3,
    }))


TWO_PRODUCTS = ("dw_pair_gemm", "gate_up_gemm")
TRAFFIC_SHAPE = (2048, 8192)     # (d_model, d_ff) of the captures behind profiles/ncu_traffic.txt
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}   # dense bf16 and HBM3e figures of the data sheet


def roofline_regime(region_s: float, sm_mhz, peaks) -> str:
    """Which measured tensor peak a timed region is compared with: the burst figure when the region
    is too short to settle under the power cap (under a second) or ran at clocks well above those
    the sustained figure was measured at, else the sustained one."""
    under_load = peaks.get("sm_mhz_under_load")
    if region_s < 1.0:
        return "burst"
    if sm_mhz and under_load and sm_mhz > 1.15 * under_load:
        return "burst"
    return "sustained"


def measure_layer(w, T, steps, warmup, args, rank, local, dev, barrier, variant, profile=True):
    """Device-resident timing of dedup + forward (+ backward) of one layer: synthetic inputs made on
    the device, `warmup` untimed steps, `steps` timed ones between two CUDA events, per-step-of-the-
    path event records, clocks sampled meanwhile."""
    import torch
    from paper_2601_10639_b200 import binding as B
    from paper_2601_10639_b200 import runner

    dcode = B.DTYPE_BF16 if w.dtype == "bf16" else B.DTYPE_FP32
    dt = runner.torch_dtype(dcode)
    d, F, V, backward = w.d_model, w.d_ff, w.V, w.backward
    gen = torch.Generator(device=dev).manual_seed(args.seed + 1000 * rank)
    flags = B.FLAG_DAGGER_FUSED if variant == "dagger_fused" else 0
    st = runner.LayerState(B.make_shape(T, d, F, V, dcode, B.DTYPE_FP32, flags), device=dev)
    st.x = torch.randn(T, d, generator=gen, device=dev, dtype=torch.float32).to(dt)
    st.dy = torch.randn(T, d, generator=gen, device=dev, dtype=torch.float32).to(dt)
    st.W_gate = (torch.randn(F, d, generator=gen, device=dev, dtype=torch.float32) * d ** -0.5).to(dt)
    st.W_down = (torch.randn(d, F, generator=gen, device=dev, dtype=torch.float32) * F ** -0.5).to(dt)
    st.E = torch.empty(V, F, device=dev, dtype=dt)
    for r0 in range(0, V, 4096):
        r1 = min(V, r0 + 4096)
        st.E[r0:r1] = (torch.randn(r1 - r0, F, generator=gen, device=dev, dtype=torch.float32) * 0.02).to(dt)
    ids_np = synth.token_ids(rank_seed(args.seed, rank), T, V, w.id_dist)
    st.ids = torch.from_numpy(ids_np).to(dev)
    st.allocate(backward)
    stream = torch.cuda.current_stream()
    run_step = lambda: st.step(backward=backward)
    if variant.startswith("dagger"):
        # STEM-dagger (Appendix): the up-projection is kept; 3 contractions forward, 6 backward
        W_up = (torch.randn(F, d, generator=gen, device=dev, dtype=torch.float32) * d ** -0.5).to(dt)
        U = torch.empty(T, F, dtype=dt, device=dev)
        dW_up = torch.empty(F, d, dtype=torch.float32, device=dev)
        b_ = st.bufs

        def run_step():
            st.dedup()
            B.stem_dagger_forward(st.shape, st.x, st.ids, st.W_gate, W_up, st.E, st.W_down, b_["y"], b_["G"], b_["H"], U,
                                  b_["ws"])
            if backward:
                B.stem_dagger_backward(st.shape, st.dy, st.x, st.W_gate, W_up, st.W_down, b_["G"], b_["H"], U, b_["perm"],
                                       b_["seg_offsets"], b_["n_unique"], b_["dx"], b_["dW_gate"], dW_up, b_["dW_down"],
                                       b_["dE_rows"], b_["ws"])

    for _ in range(warmup):
        run_step()
    barrier()
    assert st.status() == B.OK, B.status_string(st.status())
    n_u = int(st.bufs["n_unique"].item())
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = B.stem_launch_count()
    with ClockSampler(local) as clocks:
        B.stem_profile_enable(profile)
        barrier()
        t0 = time.time()
        ev0.record(stream)
        for _ in range(steps):
            run_step()
        ev1.record(stream)
        barrier()
        t1 = time.time()
        B.stem_profile_enable(False)
    launches = B.stem_launch_count() - launches0
    ms_total = ev0.elapsed_time(ev1)
    records = B.stem_profile_records()
    assert st.status() == B.OK, B.status_string(st.status())
    return {"state": st, "n_unique": n_u, "ids_np": ids_np, "dcode": dcode, "ms_total": ms_total, "records": records,
            "launches": launches, "clocks": clocks.summary(t0, t1)}


def measure_gather(st, n_u, T, V, F, esz, dev):
    """cache[r] = E[unique_ids[r]] on the device, back to back, outside the timed step."""
    import torch
    from paper_2601_10639_b200 import binding as B
    cache = torch.empty(min(T, V), F, dtype=st.E.dtype, device=dev)
    b = st.bufs
    stream = torch.cuda.current_stream()
    for _ in range(3):
        B.stem_prefetch_rows(st.shape, b["unique_ids"], b["n_unique"], st.E, cache, b["ws"])
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 20
    g0.record(stream)
    for _ in range(reps):
        B.stem_prefetch_rows(st.shape, b["unique_ids"], b["n_unique"], st.E, cache, b["ws"])
    g1.record(stream)
    torch.cuda.synchronize()
    return {"rows": n_u, "ms": g0.elapsed_time(g1) / reps, "bytes": 2 * n_u * F * esz}     # rows read once, written once


def gather_entry(gather, peaks):
    gbs = gather["bytes"] / (gather["ms"] * 1e-3) / 1e9
    return {"launch_sets": 20, "avg_ms": gather["ms"], "rows": gather["rows"], "bytes": gather["bytes"], "gbs": gbs,
            "frac_of_measured_hbm": gbs / peaks["hbm_gbs"], "frac_of_nominal_hbm": gbs / NOMINAL["hbm_gbs"],
            "note": "cache[r] = E[unique_ids[r]] on the device, back to back, outside the timed step"}


def kernel_table(records, ms_total, T, d, F, n_u, esz, grad_fp32, peaks):
    """Per step of the path: average event time, share of the timed region, and the achieved rate
    against the measured (burst and sustained) and nominal peaks."""
    by_name: dict[str, list] = {}
    for name, ms in records:
        by_name.setdefault(name, []).append(ms)
    flops_gemm = 2.0 * T * d * F
    seg_bytes = T * F * esz + n_u * F * (4 if grad_fp32 else 2) + 4 * (T + n_u + 1)
    kernels = {}
    for name, v in by_name.items():
        avg = float(np.mean(v))
        k = {"launch_sets": len(v), "avg_ms": avg, "share": float(np.sum(v)) / ms_total}
        if name.endswith("_gemm"):
            # launches that carry two products (the two weight gradients; gate and up of the dagger variant)
            k["tflops"] = (2.0 if name in TWO_PRODUCTS else 1.0) * flops_gemm / (avg * 1e-3) / 1e12
            k["frac_of_measured_sustained"] = k["tflops"] / peaks["bf16_tflops_sustained"]
            k["frac_of_measured_burst"] = k["tflops"] / peaks["bf16_tflops"]
            k["frac_of_nominal"] = k["tflops"] / NOMINAL["bf16_tflops"]
        elif name == "seg_reduce":
            k["bytes"] = seg_bytes
            k["gbs"] = seg_bytes / (avg * 1e-3) / 1e9
            k["frac_of_measured_hbm"] = k["gbs"] / peaks["hbm_gbs"]
            k["frac_of_nominal_hbm"] = k["gbs"] / NOMINAL["hbm_gbs"]
        kernels[name] = k
    return kernels


def rooflines(kernels, regime, peaks, T, d, F, bf16):
    """The two roofline objects of a bench line: the slowest contraction against the measured tensor
    peak of the run's regime, and the slower of the two HBM-bound kernels against the measured copy
    bandwidth."""
    gemms = {n: k for n, k in kernels.items() if n.endswith("_gemm")}
    roofline = None
    if gemms and bf16:
        dom = min(gemms, key=lambda n: gemms[n]["tflops"])      # the contraction furthest from the peak
        # The stored counters were taken at the 1B-class shape.  DRAM traffic grows in proportion to
        # the tokens of a launch (every [T,.] operand does; the weights are the small remainder), so
        # a capture at fewer tokens is scaled by T / T_captured; other shapes have no counters.
        cap = load_traffic(dom) if (d, F) == TRAFFIC_SHAPE else None
        traffic = cap[1] * T / cap[0] if cap else None
        key = "bf16_tflops" if regime == "burst" else "bf16_tflops_sustained"
        g = gemms[dom]
        roofline = {"kernel": dom, "bound": "tensor", "achieved": g["tflops"], "peak": peaks[key], "unit": "TFLOP/s",
                    "frac": g["tflops"] / peaks[key], "regime": regime,
                    "frac_burst": g["frac_of_measured_burst"], "frac_sustained": g["frac_of_measured_sustained"],
                    "frac_nominal": g["frac_of_nominal"], "traffic": traffic,
                    "peak_source": f"{peaks['source']} ({regime} bf16 GEMM, of measured); nominal 2250 TFLOP/s",
                    "flops_per_launch": (2.0 if dom in TWO_PRODUCTS else 1.0) * 2.0 * T * d * F}
    hbm = {n: k for n, k in kernels.items() if "frac_of_measured_hbm" in k}
    roofline_hbm = None
    if hbm:
        worst = min(hbm, key=lambda n: hbm[n]["frac_of_measured_hbm"])
        k = hbm[worst]
        cap = load_traffic(worst) if (d, F) == TRAFFIC_SHAPE else None
        roofline_hbm = {"kernel": worst, "bound": "hbm", "achieved": k["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": k["frac_of_measured_hbm"], "frac_nominal": k["frac_of_nominal_hbm"],
                        "bytes_per_launch": k["bytes"], "traffic": cap[1] * T / cap[0] if cap else None,
                        "peak_source": f"{peaks['source']} (copy bandwidth, of measured); nominal 8000 GB/s",
                        "all": {n: v["frac_of_measured_hbm"] for n, v in hbm.items()}}
    return roofline, roofline_hbm


def shard_plan(V: int, world: int, rank: int) -> dict:
    """Which rows of a V-row table rank `rank` of `world` holds (row id lives on rank id mod world at
    local index id // world) and how a batch's distinct ids spread over the owners on average."""
    from paper_2601_10639_b200 import sharded
    return {"rank": rank, "world": world, "rows_owned": sharded.shard_rows(V, world, rank),
            "first_id": rank, "id_stride": world}


def shard_rows_of_block(r0: int, r1: int, rank: int, world: int):
    """Of the table rows [r0, r1) drawn as one block, which belong to `rank` (id mod world == rank):
    (offset of the first one inside the block, its local row index, how many)."""
    first = (rank - r0) % world
    count = len(range(r0 + first, r1, world))
    return first, (r0 + first) // world, count


def sharded_line(args, w, T, world, ms_total, phase_ms, plan, sent, launches, clocks) -> dict:
    """The JSON line of the sharded mode from rank 0's view: times are maxima over ranks already."""
    F = w.d_ff
    n_u, remote = sum(sent), sum(c for g, c in enumerate(sent) if g != plan["rank"])
    ms_per_step = ms_total / args.steps
    return {
        "metric": "STEM-FFN fwd+bwd tokens/sec with the table sharded over the GPUs (id mod N), replicated weights",
        "value": world * T * args.steps / (ms_total * 1e-3), "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "T": T, "d_model": w.d_model, "d_ff": F, "V": w.V, "ids": w.id_dist,
                   "parallelism": f"table sharded id mod {world} + replicas x{world}", "exchange": "NCCL all-to-all-v",
                   "rows_owned_rank0": plan["rows_owned"],
                   "l2": "per-step working set exceeds the 126 MB L2; no flush"},
        "gpu_launches": int(launches), "clocks": clocks,
        "tflops_step": world * layer_flops(T, w.d_model, F, True) / (ms_per_step * 1e-3) / 1e12,
        "ms_per_phase_max_over_ranks": phase_ms,
        "rank0_rows": {"distinct": n_u, "from_other_ranks": remote},
        "rank0_exchange_bytes": {"ids_out": 4 * remote, "rows_in": remote * F * 2, "grad_rows_out_fp32": remote * F * 4},
        "host_round_trips_per_step": 1,
    }


def run_sharded_dist(args, w):
    """The layer with its table sharded over the ranks of a torch.distributed job (paper Section 3.4,
    "parallel embeddings"): one process per GPU, rows and gradient rows exchanged by NCCL all-to-all-v,
    every rank its own batch.  A step = route, exchange, forward, backward, exchange, the owner's
    reduce.  Times are CUDA-event times, maximum over ranks; rank 0 prints the line."""
    import socket
    import torch
    import torch.distributed as dist
    from paper_2601_10639_b200 import binding as B
    from paper_2601_10639_b200 import sharded

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    os.environ.setdefault("NCCL_DEBUG", "INFO")               # keep the communicator's own log (stderr)
    os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    if "MASTER_ADDR" not in os.environ:                       # a plain `python bench.py --sharded`: a group of one
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    B.lib()
    dt = torch.bfloat16
    T, d, F, V = (args.tokens or w.T), w.d_model, w.d_ff, w.V
    plan = shard_plan(V, world, rank)
    shape = B.make_shape(T, d, F, V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    gen = torch.Generator(device=dev).manual_seed(args.seed)         # weights and table: the same on every rank
    W_gate = (torch.randn(F, d, generator=gen, device=dev) * d ** -0.5).to(dt)
    W_down = (torch.randn(d, F, generator=gen, device=dev) * F ** -0.5).to(dt)
    shard = torch.empty(plan["rows_owned"], F, device=dev, dtype=dt)
    for r0 in range(0, V, 4096):                                     # the whole table is drawn, this rank keeps its rows
        r1 = min(V, r0 + 4096)
        blk = (torch.randn(r1 - r0, F, generator=gen, device=dev) * 0.02).to(dt)
        first, lo, count = shard_rows_of_block(r0, r1, rank, world)
        shard[lo:lo + count] = blk[first::world]
    gen_r = torch.Generator(device=dev).manual_seed(args.seed + 1000 * (rank + 1))    # the batch: every rank its own
    x = torch.randn(T, d, generator=gen_r, device=dev).to(dt)
    dy = torch.randn(T, d, generator=gen_r, device=dev).to(dt)
    ids = torch.from_numpy(synth.token_ids(rank_seed(args.seed, rank), T, V, w.id_dist)).to(dev)
    rk = sharded.ShardedRank(rank, world, shape, shard, W_gate, W_down, device=dev)
    ex = sharded.DistExchange()
    stream = torch.cuda.current_stream()

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        rk.step_dist(ex, x, ids, dy)
    barrier()
    assert rk.status() == B.OK
    events = []

    def timed(name, fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        out = fn()
        e1.record(stream)
        events.append((name, e0, e1))
        return out

    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = B.stem_launch_count()
    with ClockSampler(local) as clocks:
        barrier()
        t0 = time.time()
        ev0.record(stream)
        for _ in range(args.steps):
            rk.step_dist(ex, x, ids, dy, timed)
        ev1.record(stream)
        barrier()
        t1 = time.time()
    launches = B.stem_launch_count() - launches0
    assert rk.status() == B.OK
    names = ["route", "counts", "x_ids", "serve", "x_rows", "layer", "x_grads", "reduce"]
    sums = {n: 0.0 for n in names}
    for name, e0, e1 in events:
        sums[name] += e0.elapsed_time(e1) / args.steps
    t = max_over_ranks([ev0.elapsed_time(ev1)] + [sums[n] for n in names], dev)
    if rank == 0:
        print(json.dumps(sharded_line(args, w, T, world, t[0], dict(zip(names, t[1:])), plan, rk.h_send_counts, launches,
                                      clocks.summary(t0, t1))))
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="stem", choices=["stem", "reference"])
    ap.add_argument("--workload", default="1b", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--cpu-tokens", type=int, default=8192, help="tokens in the CPU-baseline sample (0 = skip)")
    ap.add_argument("--ref-tokens", type=int, default=1024, help="tokens per step of --impl reference")
    ap.add_argument("--seed", type=int, default=synth.BASE_SEED)
    ap.add_argument("--tokens", type=int, default=0,
                    help="override the workload's token count (small cases for profiler captures; not a bench line)")
    ap.add_argument("--hot-rows", type=int, nargs="*", default=[2048, 8192],
                    help="prefill workload: sizes of the on-device hot set to try")
    ap.add_argument("--unique-growth", action="store_true", help="print distinct rows vs context length and exit")
    ap.add_argument("--grad-bf16", action="store_true", help="host-table workload: bf16 weight and table gradients")
    ap.add_argument("--variant", default="stem", choices=["stem", "dagger", "dagger_fused"],
                    help="dagger: the paper's STEM-dagger ablation (up-projection kept, table row added); "
                         "dagger_fused: its gate and up products as one launch with two accumulators")
    ap.add_argument("--no-profile", action="store_true",
                    help="do not record per-step events inside the timed region (checks what they cost)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiler captures)")
    ap.add_argument("--no-host-config", action="store_true",
                    help="default workload only: skip the host-table stack among the other configurations")
    ap.add_argument("--no-configs", action="store_true",
                    help="default workload only: skip the short timings of the other single-layer configurations")
    ap.add_argument("--sharded", action="store_true",
                    help="the table sharded over the --gpus ranks of this job (one process per GPU, NCCL all-to-all-v)")
    ap.add_argument("--shard-ranks", type=int, default=0,
                    help="G > 0: the table sharded over G virtual ranks on one GPU (per-rank device times)")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.warmup < 3:
        args.warmup = 3

    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.unique_growth:
        run_unique_growth(args)
        return

    if args.sharded:
        if w.host_tables or not w.backward or w.dtype != "bf16":
            raise SystemExit("--sharded runs the single-layer bf16 training workloads")
        run_sharded_dist(args, w)
        return
    if args.shard_ranks > 0:
        if int(os.environ.get("WORLD_SIZE", "1")) > 1:
            raise SystemExit("--shard-ranks steps virtual ranks on one GPU")
        run_sharded(args, w)
        return
    if w.host_tables:
        if int(os.environ.get("WORLD_SIZE", "1")) > 1:
            raise SystemExit("the host-table workload is a one-GPU measurement")
        if w.note == "decode":
            run_decode(args, w)
        elif w.backward:
            print(json.dumps(run_host_stack(args, w)))
        else:
            run_prefill_stack(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2601_10639_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.lib()  # fail loudly here if the extension is missing

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = load_peaks()
    T = args.tokens or w.T
    head = measure_layer(w, T, args.steps, args.warmup, args, rank, local, dev, barrier, args.variant,
                         profile=not args.no_profile)
    st, n_u, ids_np = head["state"], head["n_unique"], head["ids_np"]
    d, F, V, backward, dcode = w.d_model, w.d_ff, w.V, w.backward, head["dcode"]
    esz = 2 if dcode == B.DTYPE_BF16 else 4
    stream = torch.cuda.current_stream()

    # ---- end to end through the host-buffer entry point -------------------------------------
    e2e = None
    if backward and not args.no_e2e and args.variant == "stem":
        hx, hdy = st.x.cpu().pin_memory(), st.dy.cpu().pin_memory()
        hids = st.ids.cpu().pin_memory()
        hy, hdx = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory()
        hn = torch.zeros(1, dtype=torch.int32).pin_memory()
        arena = torch.empty(B.stem_step_arena_bytes(st.shape), dtype=torch.uint8, device=dev)
        B.stem_init_workspace(arena)
        b = st.bufs

        def host_step():
            B.stem_ffn_step_host(st.shape, hx, hids, hdy, st.W_gate, st.E, st.W_down, hy, hdx, b["dW_gate"],
                                 b["dW_down"], b["dE_rows"], b["unique_ids"], b["n_unique"], hn, arena)
        for _ in range(3):
            host_step()
        B.stem_ffn_step_host_flush()
        barrier()
        ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ee0.record(stream)
        for _ in range(args.steps):
            host_step()
        B.stem_ffn_step_host_flush()       # the stream waits for the last output copies: they are timed
        ee1.record(stream)
        barrier()
        e2e_ms = ee0.elapsed_time(ee1)
        assert B.stem_query_status(arena) == B.OK
        assert int(hn[0]) == n_u
        assert torch.equal(hy, st.bufs["y"].cpu())       # same result as the device-resident path
        e2e = {"ms": e2e_ms, "h2d": 2 * T * d * esz + T * 4, "d2h": 2 * T * d * esz + 4}
        # what the host link gives with both directions busy: plain pinned copies of the same sizes
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        dx_dev, dx2_dev = torch.empty_like(st.x), torch.empty_like(st.x)
        torch.cuda.synchronize()
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0.record(stream)
        s_in.wait_stream(stream); s_out.wait_stream(stream)
        reps = 4
        for _ in range(reps):
            with torch.cuda.stream(s_in):
                dx_dev.copy_(hx, non_blocking=True); dx2_dev.copy_(hdy, non_blocking=True)
            with torch.cuda.stream(s_out):
                hy.copy_(dx_dev, non_blocking=True); hdx.copy_(dx2_dev, non_blocking=True)
        stream.wait_stream(s_in); stream.wait_stream(s_out)
        l1.record(stream)
        torch.cuda.synchronize()
        e2e["link_ms"] = l0.elapsed_time(l1) / reps       # per step's worth of copies, both directions at once
        del arena, dx_dev, dx2_dev

    # ---- compact row gather from the device-resident table (the standalone gather figure) ------------
    gather = None
    if rank == 0 and dcode == B.DTYPE_BF16:
        gather = measure_gather(st, n_u, T, V, F, esz, dev)

    # ---- max over ranks ------------------------------------------------------------------------
    ms_total, launches = head["ms_total"], int(head["launches"])
    if world > 1:
        t = max_over_ranks([ms_total, e2e["ms"] if e2e else 0.0], dev)
        ms_total = t[0]
        if e2e:
            e2e["ms"] = t[1]
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = ms_total / args.steps
    value = world * T * args.steps / (ms_total * 1e-3)
    clock_summary = head["clocks"]
    regime = roofline_regime(ms_total * 1e-3, clock_summary.get("sm_mhz"), peaks)
    kernels = kernel_table(head["records"], ms_total, T, d, F, n_u, esz, st.shape.grad_dtype == B.DTYPE_FP32, peaks)
    if gather:
        kernels["compact_gather"] = gather_entry(gather, peaks)
    if "gate_gemm" in kernels:
        # rows the fused lookup hands to the epilogue, per second (not a roofline: the kernel is MMA-bound)
        kernels["gate_gemm"]["fused_lookup_gbs"] = T * F * esz / (kernels["gate_gemm"]["avg_ms"] * 1e-3) / 1e9
    roofline, roofline_hbm = rooflines(kernels, regime, peaks, T, d, F, dcode == B.DTYPE_BF16)

    # ---- the CPU checker timed beside it (rank 0, N = 1 only) -----------------------------------------
    cpu = None
    if world == 1 and args.cpu_tokens > 0 and backward:
        Tc = min(args.cpu_tokens, T)
        host_inputs = {"x": st.x[:Tc].float().cpu().numpy(), "dy": st.dy[:Tc].float().cpu().numpy(),
                       "ids": ids_np[:Tc], "W_gate": st.W_gate.float().cpu().numpy(),
                       "W_down": st.W_down.float().cpu().numpy(), "E": st.E.float().cpu().numpy()}
        tps, secs = oracle_tokens_per_sec(host_inputs, Tc)
        cpu = {"value": tps, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle", "seconds": secs,
               "cores_note": "threads of the BLAS library numpy's matrix products run on",
               "sample": f"first {Tc} of {T} tokens, full weights and table, dedup + forward + backward in fp64"}

    # ---- the other single-layer configurations, shorter, outside the headline's timed region --------
    configs = None
    if (world == 1 and args.workload == "1b" and args.variant == "stem" and not args.tokens and not args.no_configs):
        configs = {}
        del st, head
        torch.cuda.empty_cache()
        for name in ("350m", "1b_long_fwd"):
            wc = synth.WORKLOADS[name]
            steps_c = max(20, min(args.steps, 50))
            m = measure_layer(wc, wc.T, steps_c, 5, args, rank, local, dev, barrier, "stem", profile=True)
            es = 2
            kern = kernel_table(m["records"], m["ms_total"], wc.T, wc.d_model, wc.d_ff, m["n_unique"], es, True, peaks)
            g = measure_gather(m["state"], m["n_unique"], wc.T, wc.V, wc.d_ff, es, dev)
            kern["compact_gather"] = gather_entry(g, peaks)
            reg = roofline_regime(m["ms_total"] * 1e-3, m["clocks"].get("sm_mhz"), peaks)
            rf, rf_hbm = rooflines(kern, reg, peaks, wc.T, wc.d_model, wc.d_ff, True)
            ms_c = m["ms_total"] / steps_c
            configs[name] = {
                "T": wc.T, "d_model": wc.d_model, "d_ff": wc.d_ff, "V": wc.V, "ids": wc.id_dist, "backward": wc.backward,
                "n_unique": m["n_unique"], "steps": steps_c, "warmup": 5, "ms_per_step": ms_c,
                "value": wc.T / (ms_c * 1e-3), "unit": "tokens/s",
                "tflops_step": layer_flops(wc.T, wc.d_model, wc.d_ff, wc.backward) / (ms_c * 1e-3) / 1e12,
                "gpu_launches": m["launches"], "clocks": m["clocks"], "roofline": rf, "roofline_hbm": rf_hbm, "kernels": kern}
            del m
            torch.cuda.empty_cache()
        if not args.no_host_config:
            # the host-table configuration: every layer of the stack, three timed passes
            wh = synth.WORKLOADS["1b_host_x16"]
            h = run_host_stack(args, wh, steps=3, warmup=3)
            configs[wh.name] = {k: h[k] for k in ("value", "unit", "steps", "warmup", "ms_per_step", "tflops_step", "config",
                                                   "gpu_launches", "clocks", "host_tables", "device_tables",
                                                   "exposed_copy_ms_per_layer", "host_link", "rows_prefetched_per_layer",
                                                   "prefetch_bytes_per_layer", "writeback_bytes_per_layer")}
            torch.cuda.empty_cache()

    out = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if dcode == B.DTYPE_BF16 else "f32", "data": "synthetic",
        "config": {"workload": w.name, "T": T, "d_model": d, "d_ff": F, "V": V, "ids": w.id_dist,
                   "n_unique": n_u, "backward": backward, "variant": args.variant, "parallelism": f"replicas x{world}",
                   "l2": "per-step working set (~2.5 GB at 1b shapes) exceeds the 126 MB L2; no flush"},
        "gpu_launches": launches,
        "tflops_step": layer_flops(T, d, F, backward) * (1.5 if args.variant.startswith("dagger") else 1.0) / (ms_per_step * 1e-3) / 1e12,
        # the ids are the same for every STEM layer of a model, so their dedup can be paid once per batch
        "value_dedup_amortised": (world * T / ((ms_per_step - kernels["dedup"]["avg_ms"]) * 1e-3)
                                  if kernels.get("dedup") else None),
        "clocks": clock_summary,
        "roofline": roofline,
        "roofline_hbm": roofline_hbm,
        "kernels": kernels,
        "cpu_baseline": cpu,
    }
    if configs is not None:
        out["configs"] = configs
    if e2e:
        e2e_step = e2e["ms"] / args.steps
        link_gbs = (e2e["h2d"] + e2e["d2h"]) / (e2e["link_ms"] * 1e-3) / 1e9
        out["e2e"] = {"value": world * T * args.steps / (e2e["ms"] * 1e-3), "unit": "tokens/s",
                      "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                      "ms_per_step": e2e_step,
                      # the copies of a step, alone, both directions at once, against the kernels of a step
                      "link_ms_per_step": e2e["link_ms"], "link_gbs_both_directions": link_gbs,
                      "bound": "host link" if e2e["link_ms"] >= 0.9 * ms_per_step else "kernels"}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the selective-FFN hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2] [--impl ours|reference]

One "step" = one pass of the whole decode hot path over one batch of synthetic input: all
tokens of the workload through all FFN layers, each layer running the selective FFN on that
token's active list (one persistent launch through the C ABI).  The store is built once by
the loader before timing.  Metric: selective-FFN decode tokens/s at batch 1.

Prints ONE JSON line (rank 0).  The headline is configuration 2 with the (token, layer) steps
independent of one another (every step's input given up front) and worked through in order.
Beside it, in the same line: `chained` -- the same launch size with every layer reading the
output of the layer before it, as inside a decoder; `steps_any_order`; and `configs` -- the other
four configurations (c1 latency, c3 batch sizes, c4 prefill, the sixteen c5 cells), each measured
on a stated reduced number of layers whose weights still exceed L2.

With N > 1 each rank is an independent replica decoding its own tokens against its own copy of
the store: no data-path collective, weak scaling, time = max over ranks.  Started without a
launcher, `--gpus N` starts its own N ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_18081_b200 import replicas, workloads as wl  # noqa: E402

METRIC = "selective_ffn_decode_tokens_per_s_batch1"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of si_decode_persistent_kernel per (token, layer) step of
# the config-2 shape: an ncu capture of an 8-layer x 32-token launch (256 steps) read 9.6434e9 and wrote
# 0.2278e9 bytes; traffic grows in proportion to the steps (every step reads its own records once)
NCU_DRAM_BYTES_PER_C2_STEP = (9.6434e9 + 0.2278e9) / 256
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        mhz, mx, reasons = [], None, set()
        inside = [l for (t, l) in self.lines if t0 - 0.05 <= t <= t1 + 0.15] or [l for _, l in self.lines]
        for l in inside:
            parts = [p.strip() for p in l.split(",")]
            if len(parts) < 6:
                continue
            try:
                mhz.append(float(parts[0])); mx = float(parts[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                               parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(mhz)}


def cell_config(args):
    cfg = wl.CONFIGS[args.config]
    kw = {}
    if args.layers:
        kw["n_layers"] = args.layers
    if args.tokens:
        kw["tokens"] = args.tokens
    if args.loaded_pct:
        kw["loaded_pct"] = args.loaded_pct
    if args.active_pct:
        kw["active_pct"] = args.active_pct
    if args.batch:
        kw["batch"] = args.batch
    return cfg.with_(**kw) if kw else cfg


def workload_name(cfg):
    return (f"{cfg.name}: {cfg.n_layers} layers d_model={cfg.d_model} d_ff={cfg.d_ff} {cfg.dtype}, "
            f"{cfg.loaded_pct}% loaded ({cfg.n_loaded}), {cfg.active_pct}% of loaded active ({cfg.k_active}) "
            f"per token by Zipf(1.1), batch 1, {cfg.tokens} decode tokens")


# ----------------------------------------------------------------------------- reference arm

def run_reference(args):
    """Times the float64 CPU oracle, as it stands, on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import selectinfer_oracle as so
    cfg = cell_config(args)
    cores = so.host_threads()
    n_layers_sample = min(cfg.n_layers, 4)
    layers = [wl.layer_weights(cfg, l) for l in range(n_layers_sample)]
    ids = [wl.loaded_ids(cfg, l) for l in range(n_layers_sample)]

    def one_step(step):
        for l in range(n_layers_sample):
            lst = wl.zipf_lists(cfg, l, 1, slot_of_rank=ids[l][1], first_token=step)[0]
            x = wl.x_tokens(cfg, l, 1, first_token=step)[0]
            so.ffn(*layers[l], x, ids[l][0][lst], dtype=cfg.dtype, threads=cores)

    for w in range(args.warmup):
        one_step(w)
    t0 = time.perf_counter()
    for s in range(args.steps):
        one_step(args.warmup + s)
    dt = time.perf_counter() - t0
    # one step = one token through n_layers_sample of the n_layers layers
    tok_s = args.steps * (n_layers_sample / cfg.n_layers) / dt
    sample = (f"{args.steps} tokens x first {n_layers_sample} of {cfg.n_layers} layers "
              f"(list and input generation included), scaled to all layers")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": tok_s, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg)},
        "cpu_baseline": {"value": tok_s, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tok_s, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))



# ----------------------------------------------------------------------------- measuring helpers

def device_ms(torch, fn, reps, warm=3):
    """Mean CUDA-event time of fn() over reps calls on the current stream, after warm-up."""
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def graphed(torch, fn):
    """fn() captured once into a CUDA graph (host launch overhead out of the picture); returns a
    callable that replays it, or fn itself if the capture is not possible."""
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g.replay, True
    except Exception:                                   # pragma: no cover
        torch.cuda.synchronize()
        return fn, False


def load_store(api, torch, cfg, n_layers, device):
    tdt = api.torch_dtype(cfg.dtype)
    store = api.NeuronStore(n_layers, cfg.d_model, cfg.d_ff, [cfg.n_loaded] * n_layers, cfg.dtype, device=device)
    for l in range(n_layers):
        wg, wu, wd = wl.layer_weights(cfg, l)
        ids, _ = wl.loaded_ids(cfg, l)
        to_dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(tdt)
        store.load(l, to_dev(wg), to_dev(wu), to_dev(wd), ids, cfg.n_base)
        del wg, wu, wd
    torch.cuda.synchronize()
    return store


CHAIN_EPS = 1e-5


def measure_chained(api, torch, store, cfg, heads_dev, idx_dev, ws, status, peaks, reps):
    """The same launch size as the headline with every layer reading the output of the layer before it
    (one chain per token, pre-norm + residual): microseconds per (token, layer) step and the rate the
    selected bytes stream at."""
    L, d, k, tokens = cfg.n_layers, cfg.d_model, cfg.k_active, cfg.tokens
    n_steps = tokens * L
    y = torch.empty(n_steps, d, dtype=api.torch_dtype(cfg.dtype), device="cuda")
    flags = api.SI_FLAG_PRENORM | api.SI_FLAG_RESIDUAL

    def launch():
        api.si_decode_chain_forward(store.handle, n_steps, None, L, heads_dev, idx_dev, None, k, y, None, CHAIN_EPS,
                                    flags, ws, status)

    ms = device_ms(torch, launch, reps)
    us_step = ms * 1e3 / n_steps
    gbs = k * cfg.record_bytes / us_step / 1e3

    # the same launch through the diagnostics call with no weight copied at all (skip_mask bits 3 and 4: neither the
    # records nor the down slices; its y is meaningless and goes to a buffer of its own): what the exchanges between
    # the SMs and the arithmetic of the dependent steps cost by themselves
    y_floor = torch.empty_like(y)

    def launch_no_weights():
        api.si_debug_decode_chain_forward(store.handle, n_steps, None, L, heads_dev, idx_dev, None, k, y_floor, None,
                                          CHAIN_EPS, flags, ws, status, skip_mask=24)

    ms_floor = device_ms(torch, launch_no_weights, max(2, reps // 2))
    return {"value": tokens / (ms * 1e-3), "unit": UNIT, "us_per_step": us_step, "achieved_gbs": gbs,
            "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS, "launch_ms": ms,
            "us_per_step_without_weight_traffic": ms_floor * 1e3 / n_steps,
            "note": "si_decode_chain_forward: one chain per token through all layers, each layer's input = the rounded "
                    "output of the layer before it (pre-norm + residual); no arithmetic of a step starts before the "
                    "step before it is complete on every SM, only the weight stream runs ahead"}, y


def extra_configs(api, torch, args, device, peaks, peak_kind):
    """The four configurations beside the headline, each on a reduced number of layers whose weights
    still exceed L2 (stated per entry), timed with CUDA events; per-layer calls replayed from CUDA graphs."""
    out = {}
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    hbm = peaks["hbm_gbs"]

    # ---- c1: one small fp16 layer, 16 decode tokens; the whole store (2.1 MB) is L2-resident
    try:
        cfg = wl.CONFIGS["c1"]
        store = load_store(api, torch, cfg, 1, device)
        _, sor = wl.loaded_ids(cfg, 0)
        tdt = api.torch_dtype(cfg.dtype)
        x = torch.from_numpy(wl.x_tokens(cfg, 0, cfg.tokens).view(np.int16)).cuda().view(tdt)
        idx = torch.from_numpy(wl.zipf_lists(cfg, 0, cfg.tokens, slot_of_rank=sor)).cuda()
        y = torch.empty(cfg.tokens, cfg.d_model, dtype=tdt, device="cuda")
        ws = store.workspace(1, cfg.k_active, cfg.tokens)
        one, g1 = graphed(torch, lambda: api.si_ffn_forward(store.handle, 0, x[0], 1, idx[0], None, cfg.k_active, y[0], 0, ws, status))
        allt, g2 = graphed(torch, lambda: api.si_decode_stack_forward(store.handle, cfg.tokens, [0] * cfg.tokens, x, idx, None,
                                                                      cfg.k_active, y, 0, ws, status))
        ms_one, ms_all = device_ms(torch, one, 200), device_ms(torch, allt, 100)
        out["c1"] = {"workload": "c1: 1 layer d_model=512 d_ff=1376 f16, 688 loaded, 172 active, batch 1, 16 decode tokens",
                     "us_per_token_single_call": ms_one * 1e3, "us_per_token_in_one_16_token_launch": ms_all * 1e3 / cfg.tokens,
                     "tokens_per_s": cfg.tokens / (ms_all * 1e-3), "selected_bytes_per_token": cfg.k_active * cfg.record_bytes,
                     "replayed_from_cuda_graph": bool(g1 and g2),
                     "note": "the whole store (2.1 MB) is L2-resident: launch- and latency-bound, an HBM roofline does not apply"}
        store.close(); del store, ws
    except Exception as e:                              # pragma: no cover
        out["c1"] = {"error": repr(e)}

    # ---- c3 (batched decode over the union) and c4 (prefill, one shared list): per-layer calls, 4 layers
    def multitoken(cfg, T, n_layers, groups, shared):
        tdt = api.torch_dtype(cfg.dtype)
        d, k = cfg.d_model, cfg.k_active
        store = load_store(api, torch, cfg, n_layers, device)
        x = torch.empty(groups, n_layers, T, d, dtype=torch.int16)
        for l in range(n_layers):
            x[:, l] = torch.from_numpy(wl.x_tokens(cfg, l, groups * T).view(np.int16)).view(groups, T, d)
        x = x.cuda().view(tdt)
        if shared:
            idx, flags, usz = torch.arange(k, dtype=torch.int32, device="cuda"), api.SI_FLAG_SHARED_LIST, [k]
        else:
            blk = (T * k + 3) // 4 * 4                          # every (group, layer) block of lists starts 16-byte aligned
            lists = np.zeros((groups, n_layers, blk), dtype=np.int32)
            for l in range(n_layers):
                lists[:, l, :T * k] = wl.zipf_lists(cfg, l, groups * T).reshape(groups, T * k)
            usz = [len(np.unique(lists[g, l, :T * k])) for g in range(groups) for l in range(n_layers)]
            idx, flags = torch.from_numpy(lists).cuda(), 0
        y = torch.empty(groups, n_layers, T, d, dtype=tdt, device="cuda")
        ws = store.workspace(max(T, 2), k, max(T, 1))

        def run():
            for g in range(groups):
                for l in range(n_layers):
                    api.si_ffn_forward(store.handle, l, x[g, l], T, idx if shared else idx[g, l, :T * k], None, k, y[g, l], flags, ws, status)

        fn, was_graph = graphed(torch, run)
        ms = device_ms(torch, fn, 10)
        us_call = ms * 1e3 / (groups * n_layers)
        store.close()
        return us_call, float(np.mean(usz)), was_graph

    try:
        cfg3 = wl.CONFIGS["c3"]
        cells = []
        for B in wl.C3_BATCHES:
            us_call, u, was_graph = multitoken(cfg3.with_(batch=B), B, 4, max(1, 8 // B) if B < 8 else 1, False)
            tok_s = B / (us_call * 1e-6 * cfg3.n_layers)
            ubytes = u * cfg3.record_bytes
            cells.append({"batch": B, "tokens_per_s": tok_s, "us_per_layer_call": us_call, "mean_union": u,
                          "union_overlap": 1.0 - u / (B * cfg3.k_active), "union_coverage_of_loaded": u / cfg3.n_loaded,
                          "union_gbs": ubytes / us_call / 1e3, "frac": ubytes / us_call / 1e3 / hbm,
                          "route": "decode kernel" if B == 1 else "union + tensor-core contractions (K split over thread-block clusters)",
                          "replayed_from_cuda_graph": was_graph})
        out["c3"] = {"workload": "c3: 7B-shaped stack (d_model=4096, d_ff=11008, bf16, 7705 loaded), own 1541-slot Zipf list per "
                                 "token, batch sizes 1..32; measured on 4 layers (757 MB of records), tokens/s scaled to 32 layers",
                     "bound": "hbm", "peak": hbm, "peak_kind": f"of {peak_kind}", "cells": cells}
    except Exception as e:                              # pragma: no cover
        out["c3"] = {"error": repr(e)}
    try:
        cfg4 = wl.CONFIGS["c4"]
        us_call, u, was_graph = multitoken(cfg4, cfg4.tokens, 4, 1, True)
        tflops = 6.0 * cfg4.d_model * cfg4.k_active * cfg4.tokens / us_call / 1e6
        out["c4"] = {"workload": "c4: 7B-shaped stack, 512 prefill tokens, one shared list of 3082 slots per layer; measured on 4 "
                                 "layers, tokens/s scaled to 32 layers",
                     "tokens_per_s": cfg4.tokens / (us_call * 1e-6 * cfg4.n_layers), "us_per_layer_call": us_call,
                     "bound": "tensor", "achieved_tflops": tflops, "peak": peaks["bf16_tflops_sustained"],
                     "frac": tflops / peaks["bf16_tflops_sustained"], "peak_kind": f"of {peak_kind} (sustained)",
                     "replayed_from_cuda_graph": was_graph,
                     "kernels": "CTA pairs (tcgen05.mma.cta_group::2): tokens on M, store columns on N, weight tiles by tensor copies"}
        # the same call over ALL loaded neurons (what the prefill of a prompt runs before it votes: Section 5)
        cfg4a = cfg4.with_(active_pct=100)
        us_all, _, _ = multitoken(cfg4a, cfg4a.tokens, 4, 1, True)
        tf_all = 6.0 * cfg4a.d_model * cfg4a.k_active * cfg4a.tokens / us_all / 1e6
        out["c4"]["all_loaded"] = {"k": cfg4a.k_active, "us_per_layer_call": us_all, "achieved_tflops": tf_all,
                                   "frac": tf_all / peaks["bf16_tflops_sustained"]}
    except Exception as e:                              # pragma: no cover
        out["c4"] = {"error": repr(e)}

    # ---- c5: 16 cells (loaded x active), 4 layers x 64 tokens per launch.  The loaded set of a cell is the
    # first n_loaded ids of the layer's ranking, slot = rank, so one store holding every neuron serves all cells.
    try:
        n_layers = 4
        base = wl.CONFIGS["c5"].with_(n_layers=n_layers, loaded_pct=100)
        store = load_store(api, torch, base, n_layers, device)
        tdt = api.torch_dtype(base.dtype)
        d, tokens = base.d_model, base.tokens
        n_steps = tokens * n_layers
        x = torch.empty(tokens, n_layers, d, dtype=torch.int16)
        for l in range(n_layers):
            x[:, l] = torch.from_numpy(wl.x_tokens(base, l, tokens).view(np.int16))
        x = x.cuda().view(tdt).view(n_steps, d)
        heads = x.view(tokens, n_layers, d)[:, 0].contiguous()
        y = torch.empty(n_steps, d, dtype=tdt, device="cuda")
        cells = []
        for lp in wl.C5_LOADED:
            for ap in wl.C5_ACTIVE:
                cfg = base.with_(loaded_pct=lp, active_pct=ap)
                k = cfg.k_active
                lists = np.empty((tokens, n_layers, k), dtype=np.int32)
                for l in range(n_layers):
                    lists[:, l] = wl.zipf_lists(cfg, l, tokens)
                idx = torch.from_numpy(lists.reshape(n_steps, k)).cuda()
                ws = store.workspace(1, k, n_steps)
                ms = device_ms(torch, lambda: api.si_decode_stack_forward(store.handle, n_steps, None, x, idx, None, k, y, 0, ws, status), 5)
                ms_any = device_ms(torch, lambda: api.si_decode_stack_forward(store.handle, n_steps, None, x, idx, None, k, y,
                                                                              api.SI_FLAG_STEPS_ANY_ORDER, ws, status), 5)
                ms_ch = device_ms(torch, lambda: api.si_decode_chain_forward(store.handle, n_steps, None, n_layers, heads, idx, None, k, y,
                                                                             None, CHAIN_EPS, api.SI_FLAG_PRENORM | api.SI_FLAG_RESIDUAL,
                                                                             ws, status), 3)
                bytes_step = k * cfg.record_bytes
                cell = {"loaded_pct": lp, "active_pct": ap, "k": k}
                for name, m in (("in_order", ms), ("any_order", ms_any), ("chained", ms_ch)):
                    us = m * 1e3 / n_steps
                    cell[name] = {"us_per_step": us, "gbs": bytes_step / us / 1e3, "frac_of_nominal_8TBs": bytes_step / us / 1e3 / NOMINAL_HBM_GBS,
                                  "tokens_per_s_32_layers": 1e6 / (us * 32)}
                cells.append(cell)
                del ws, idx
        out["c5"] = {"workload": "c5: 8B-shaped FFN (d_model=4096, d_ff=14336, bf16), loaded {30,50,70,100}% x active {5,10,20,50}% of "
                                 "loaded, Zipf lists, batch 1, 64 tokens; measured on 4 layers per launch (256 steps), tokens/s scaled "
                                 "to 32 layers", "bound": "hbm", "cells": cells}
        store.close()
    except Exception as e:                              # pragma: no cover
        out["c5"] = {"error": repr(e)}
    if int(status.item()) != 0:
        out["device_status"] = int(status.item())
    return out

# ----------------------------------------------------------------------------- our arm

def run_ours(args):
    import torch
    import torch.distributed as dist

    rank, world, local_rank = replicas.rank_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the selective-FFN library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    from paper_2607_18081_b200 import api, build
    build.build()

    cfg = cell_config(args)
    if cfg.name in ("c3", "c4"):
        return run_multitoken(args, cfg, rank, world, local_rank)
    L, d, k, tokens = cfg.n_layers, cfg.d_model, cfg.k_active, cfg.tokens
    tdt = api.torch_dtype(cfg.dtype)
    host_threads = max(1, len(os.sched_getaffinity(0)) // world)

    # ---- load the model: selective loading of every layer (not timed; once per model)
    t_load0 = time.perf_counter()
    store = api.NeuronStore(L, d, cfg.d_ff, [cfg.n_loaded] * L, cfg.dtype, device=f"cuda:{local_rank}")
    cpu_samples = []
    cpu_tokens = args.cpu_tokens if (rank == 0 and world == 1 and not args.no_cpu_baseline) else 0
    oracle = None
    if cpu_tokens:
        from oracle import selectinfer_oracle as oracle  # cpu_baseline leg only
    cpu_time = 0.0
    cpu_time_1t, cpu_layers_1t = 0.0, 0
    parity = []
    for l in range(L):
        wg, wu, wd = wl.layer_weights(cfg, l)
        ids, sor = wl.loaded_ids(cfg, l)
        to_dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(tdt)
        store.load(l, to_dev(wg), to_dev(wu), to_dev(wd), ids, cfg.n_base)
        if cpu_tokens:
            lists = wl.zipf_lists(cfg, l, cpu_tokens, slot_of_rank=sor)
            xs = wl.x_tokens(cfg, l, cpu_tokens)
            t0 = time.perf_counter()
            for t in range(cpu_tokens):
                y_ref = oracle.ffn(wg, wu, wd, xs[t], ids[lists[t]], dtype=cfg.dtype, threads=host_threads)
            cpu_time += time.perf_counter() - t0
            if l < 4:                                     # one token on four layers with a single thread
                t0 = time.perf_counter()
                oracle.ffn(wg, wu, wd, xs[0], ids[lists[0]], dtype=cfg.dtype, threads=1)
                cpu_time_1t += time.perf_counter() - t0
                cpu_layers_1t += 1
            if l in (0, L - 1):
                cpu_samples.append((l, cpu_tokens - 1, y_ref))
        del wg, wu, wd
    torch.cuda.synchronize()
    load_s = time.perf_counter() - t_load0

    # ---- synthetic decode inputs for this rank (pinned host memory)
    first_token, _ = replicas.token_range(rank, world, tokens)
    x_host = torch.empty(tokens, L, d, dtype=torch.int16).pin_memory()
    idx_host = torch.empty(tokens, L, k, dtype=torch.int32).pin_memory()
    for l in range(L):
        _, sor = wl.loaded_ids(cfg, l)
        x_host[:, l] = torch.from_numpy(wl.x_tokens(cfg, l, tokens, first_token).view(np.int16))
        idx_host[:, l] = torch.from_numpy(wl.zipf_lists(cfg, l, tokens, slot_of_rank=sor, first_token=first_token))
    n_steps = tokens * L
    y_host = torch.empty(n_steps, d, dtype=tdt).pin_memory()
    x_dev = x_host.cuda().view(tdt).view(n_steps, d)
    idx_dev = idx_host.cuda().view(n_steps, k)
    y_dev = torch.empty(n_steps, d, dtype=tdt, device="cuda")
    ws = store.workspace(1, k, n_steps)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    flags = api.SI_FLAG_SIMPLE_KERNELS if args.simple else 0

    def step_device():
        api.si_decode_stack_forward(store.handle, n_steps, None, x_dev, idx_dev, None, k, y_dev, flags, ws, status)

    # the same launch with the caller's statement that the steps are independent (every step's x is an input),
    # which lets the SMs work in step groups: reported beside the headline, which keeps the steps in order
    def step_device_any_order():
        api.si_decode_stack_forward(store.handle, n_steps, None, x_dev, idx_dev, None, k, y_dev,
                                    flags | api.SI_FLAG_STEPS_ANY_ORDER, ws, status)

    # End to end: the step's x and lists start in pinned host memory and y ends there.  The tokens go
    # through in chunks so that the copies of one chunk run beside the decode launch of another
    # (copy-in stream -> launch stream -> copy-out stream, two device input buffers).
    # The first and the last chunk are small: the first copy-in and the last copy-out are the only copies
    # that nothing overlaps.
    if args.e2e_sizes:
        sizes = [int(v) for v in args.e2e_sizes.split(",")]
        if sum(sizes) != tokens:
            raise SystemExit("--e2e-sizes must add up to the tokens of a step")
    elif tokens >= 32:
        # a small first and last chunk: the first copy-in and the last copy-out are the only copies nothing
        # overlaps (measured at 128 tokens: [8, 112, 8] 5.71 k tokens/s, four equal chunks 5.55 k, one chunk 5.40 k)
        edge = tokens // 16
        sizes = [edge, tokens - 2 * edge, edge]
    else:
        sizes = [tokens]
    sizes = [c for c in sizes if c > 0]
    n_chunk = len(sizes)
    starts = [sum(sizes[:i]) for i in range(n_chunk)]
    cs_max = max(sizes) * L                                  # (token, layer) steps of the largest chunk
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    xd_buf = [torch.empty(cs_max, d, dtype=tdt, device="cuda") for _ in range(2)]
    idd_buf = [torch.empty(cs_max, k, dtype=torch.int32, device="cuda") for _ in range(2)]
    x_host_f = x_host.view(tdt).view(n_steps, d)
    idx_host_f = idx_host.view(n_steps, k)
    buf_free = [None, None]

    def step_e2e():
        cur = torch.cuda.current_stream()
        s_in.wait_stream(cur)
        for c in range(n_chunk):
            b = c % 2
            lo, n = starts[c] * L, sizes[c] * L
            with torch.cuda.stream(s_in):
                if buf_free[b] is not None:
                    s_in.wait_event(buf_free[b])             # the launch that read this buffer is done
                xd_buf[b][:n].copy_(x_host_f[lo:lo + n], non_blocking=True)
                idd_buf[b][:n].copy_(idx_host_f[lo:lo + n], non_blocking=True)
                arrived = torch.cuda.Event()
                arrived.record(s_in)
            cur.wait_event(arrived)
            api.si_decode_stack_forward(store.handle, n, None, xd_buf[b][:n], idd_buf[b][:n], None, k, y_dev[lo:lo + n], flags,
                                        ws, status)
            done = torch.cuda.Event()
            done.record(cur)
            buf_free[b] = done
            with torch.cuda.stream(s_out):
                s_out.wait_event(done)
                y_host[lo:lo + n].copy_(y_dev[lo:lo + n], non_blocking=True)
        cur.wait_stream(s_out)                               # the step ends when y is back on the host

    def barrier():
        torch.cuda.synchronize()
        replicas.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup, sampler=None):
        for _ in range(warmup):
            fn()
        barrier()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        t0 = time.time()
        ev[0].record()
        for i in range(steps):
            fn()
            ev[i + 1].record()
        barrier()
        t1 = time.time()
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        total_ms = ev[0].elapsed_time(ev[steps])
        total_ms = replicas.max_over_ranks(total_ms, device="cuda")
        return total_ms, per, (t0, t1)

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.3)
    total_ms, per_step_ms, (t0, t1) = timed(step_device, args.steps, max(args.warmup, 3))
    clocks = sampler.stop(t0, t1) if sampler else None
    side_steps = max(3, min(args.steps, 20))               # the figures beside the headline need no long region
    any_ms, any_per, _ = timed(step_device_any_order, side_steps, 3)
    e2e_ms, _, _ = timed(step_e2e, args.steps, max(args.warmup, 3))
    if int(status.item()) != 0:
        raise SystemExit(f"device status {status.item()}: {api.strerror(int(status.item()))}")
    chained = None
    if rank == 0 and not args.simple and not args.no_chained:
        peaks_c, _ = measured_peaks()
        heads_dev = x_dev.view(tokens, L, d)[:, 0].contiguous()         # a token's chain starts from its layer-0 input
        chained, y_chain = measure_chained(api, torch, store, cfg, heads_dev, idx_dev, ws, status, peaks_c, side_steps)
        if int(status.item()) != 0:
            raise SystemExit(f"device status {status.item()} in the chained launch: {api.strerror(int(status.item()))}")
        if cpu_tokens:
            # parity of the chained launch: sampled steps against the oracle fed with the very input the device read
            xn = torch.empty(n_steps, d, dtype=tdt, device="cuda")
            api.si_decode_chain_forward(store.handle, n_steps, None, L, heads_dev, idx_dev, None, k, y_chain, xn, CHAIN_EPS,
                                        api.SI_FLAG_PRENORM | api.SI_FLAG_RESIDUAL, ws, status)
            torch.cuda.synchronize()
            bits = lambda t_: t_.view(torch.int16).cpu().numpy().view(np.uint16)
            t_s = cpu_tokens - 1
            errs = []
            for l in (0, L - 1):
                s_ = t_s * L + l
                wg, wu, wd = wl.layer_weights(cfg, l)
                ids, sor = wl.loaded_ids(cfg, l)
                x_in = bits(heads_dev[t_s]) if l == 0 else bits(y_chain[s_ - 1])
                xin64 = oracle.widen_bits(x_in, cfg.dtype)
                xn_ref = oracle.rmsnorm(xin64, CHAIN_EPS)
                xn_dev = oracle.widen_bits(bits(xn[s_]), cfg.dtype)
                lst = idx_host.view(n_steps, k)[s_].numpy()
                ref = oracle.ffn(wg, wu, wd, bits(xn[s_]), ids[lst], dtype=cfg.dtype, threads=host_threads) + xin64
                e = oracle.error_metrics(oracle.widen_bits(bits(y_chain[s_]), cfg.dtype), ref)
                errs.append({"step": [t_s, l], "max_rel": e[0], "mean_rel": e[1],
                             "norm_max_rel_dev": float(np.max(np.abs(xn_dev - xn_ref) / np.maximum(np.abs(xn_ref), 1e-30)))})
                del wg, wu, wd
            chained["parity_samples"] = errs
            del xn

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        tok_s = replicas.aggregate_throughput(tokens * args.steps, world, total_ms)
        e2e_tok_s = replicas.aggregate_throughput(tokens * args.steps, world, e2e_ms)
        alg_bytes = wl.selected_bytes_per_token(cfg) * tokens          # per launch (= per step), per GPU
        launch_ms = statistics.mean(per_step_ms)
        achieved = alg_bytes / (launch_ms * 1e-3) / 1e9
        # practical ceiling beside it: one kernel that only reads the store once with plain loads
        chk = torch.zeros(1, dtype=torch.int32, device="cuda")
        rb_bytes = store.nbytes - store.nbytes % 16
        for _ in range(2):
            api.si_debug_read_bandwidth(store.mem_aligned, rb_bytes, chk)
        torch.cuda.synchronize()
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        r0.record()
        for _ in range(3):
            api.si_debug_read_bandwidth(store.mem_aligned, rb_bytes, chk)
        r1.record()
        torch.cuda.synchronize()
        read_ceiling = rb_bytes * 3 / (r0.elapsed_time(r1) * 1e-3) / 1e9
        out = {
            "metric": METRIC, "value": tok_s, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": workload_name(cfg), "tokens_per_step": tokens, "layers": L,
                       "parallelism": f"replicas x{world} (no data-path collective)",
                       "l2": ("inputs exceed L2: %.0f MB of selected records per launch, no flush needed"
                              if wl.selected_bytes_per_token(cfg) * tokens > 2 * 126e6 else
                              "%.0f MB of selected records per launch: partly L2-resident, see traffic")
                             % (wl.selected_bytes_per_token(cfg) * tokens / 1e6),
                       "kernel": "simple" if args.simple else "persistent"},
            "e2e": {"value": e2e_tok_s, "unit": UNIT, "h2d_bytes_per_step": x_host.numel() * 2 + idx_host.numel() * 4,
                    "d2h_bytes_per_step": y_host.numel() * y_host.element_size(),
                    "launches_per_step": n_chunk if not args.simple else 2 * n_steps,
                    "pipeline": f"chunks of {sizes} tokens: copies of one chunk overlap the launch of another"},
            "gpu_launches": args.steps * (1 if not args.simple else 2 * n_steps),     # (headline region; the side figures launch more)
            "clocks": clocks,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}",
                         "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                         "kernel": "si_decode_persistent_kernel" if not args.simple else "si_decode_partial_kernel",
                         "algorithmic_bytes_per_launch": alg_bytes, "launch_ms": launch_ms,
                         "launch_ms_median": statistics.median(per_step_ms), "launch_ms_best": min(per_step_ms),
                         "read_only_kernel_gbs": read_ceiling,
                         "frac_of_read_only_kernel": achieved / read_ceiling,
                         "traffic": (args.traffic_bytes if args.traffic_bytes is not None else
                                     (NCU_DRAM_BYTES_PER_C2_STEP * n_steps
                                      if (cfg.name == "c2" and not args.simple) else None))},
            "load_seconds": load_s,
        }
        out["config"]["steps"] = "independent: every (token, layer) step's input is given up front; worked through in order"
        if clocks and clocks.get("sm_mhz"):
            out["ms_per_step_x_sm_mhz"] = total_ms / args.steps * clocks["sm_mhz"]       # comparable across GPUs that clock differently
        if chained is not None:
            out["chained"] = chained
        any_launch_ms = statistics.mean(any_per)
        out["steps_any_order"] = {
            "value": replicas.aggregate_throughput(tokens * side_steps, world, any_ms), "unit": UNIT,
            "achieved_gbs": alg_bytes / (any_launch_ms * 1e-3) / 1e9,
            "frac": alg_bytes / (any_launch_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "frac_of_read_only_kernel": alg_bytes / (any_launch_ms * 1e-3) / 1e9 / read_ceiling,
            "note": "same launch with SI_FLAG_STEPS_ANY_ORDER: the SMs work in four groups that each take every "
                    "fourth step; not the headline, which keeps every SM on the steps in their order"}
        if cpu_tokens:
            # parity spot check of the timed configuration against the oracle samples
            errs = []
            for (l, t, y_ref) in cpu_samples:
                yg = y_dev[t * L + l].double().cpu().numpy()
                errs.append(oracle.error_metrics(yg, y_ref))
            out["parity_samples"] = [{"max_rel": e[0], "mean_rel": e[1]} for e in errs]
            out["cpu_baseline"] = {
                "value": cpu_tokens / cpu_time, "unit": UNIT, "cores": host_threads, "kind": "oracle",
                "sample": f"{cpu_tokens} tokens x all {L} layers, float64 oracle as it stands, "
                          f"{host_threads} OpenMP threads",
                "single_thread": {"value": (cpu_layers_1t / L) / cpu_time_1t if cpu_time_1t > 0 else None, "unit": UNIT,
                                  "sample": f"1 token x {cpu_layers_1t} layers with one thread, scaled to {L} layers"}}
        if world == 1 and not args.no_extra_configs and cfg.name == "c2":
            store.close()
            del store
            torch.cuda.empty_cache()
            out["configs"] = extra_configs(api, torch, args, f"cuda:{local_rank}", peaks, peak_kind)
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_multitoken(args, cfg, rank, world, local_rank):
    """Configs 3 (batched decode: the union of B lists per layer) and 4 (512-token prefill with one
    shared list): per-layer si_ffn_forward calls with T > 1 on the tensor-core path.  Not the
    headline line; reports tokens/s, union size / overlap and achieved GB/s or TFLOP/s."""
    import torch
    from paper_2607_18081_b200 import api
    L, d = cfg.n_layers, cfg.d_model
    tdt = api.torch_dtype(cfg.dtype)
    prefill = cfg.shared_list
    T = cfg.tokens if prefill else cfg.batch
    k = cfg.k_active
    n_groups = 1 if prefill else max(1, cfg.tokens // T if cfg.tokens >= T else 1)
    store = api.NeuronStore(L, d, cfg.d_ff, [cfg.n_loaded] * L, cfg.dtype, device=f"cuda:{local_rank}")
    for l in range(L):
        wg, wu, wd = wl.layer_weights(cfg, l)
        ids, _ = wl.loaded_ids(cfg, l)
        to_dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(tdt)
        store.load(l, to_dev(wg), to_dev(wu), to_dev(wd), ids, cfg.n_base)
        del wg, wu, wd
    first_token, _ = replicas.token_range(rank, world, n_groups * T)
    x = torch.empty(n_groups, L, T, d, dtype=torch.int16)
    for l in range(L):
        xs = wl.x_tokens(cfg, l, n_groups * T, first_token)
        x[:, l] = torch.from_numpy(xs.view(np.int16)).view(n_groups, T, d)
    x = x.cuda().view(tdt)
    union_sizes = []
    if prefill:
        idx = torch.arange(k, dtype=torch.int32, device="cuda")
        flags = api.SI_FLAG_SHARED_LIST
        union_sizes = [k]
    else:
        lists = np.empty((n_groups, L, T, k), dtype=np.int32)
        for l in range(L):
            ll = wl.zipf_lists(cfg, l, n_groups * T, first_token=first_token)
            lists[:, l] = ll.reshape(n_groups, T, k)
        union_sizes = [len(np.unique(lists[g, l])) for g in range(n_groups) for l in range(min(L, 4))]
        idx = torch.from_numpy(lists).cuda()
        flags = api.SI_FLAG_UNION_PATH     # config 3 is about the union path (a single token would otherwise take the decode kernel)
    y = torch.empty(n_groups, L, T, d, dtype=tdt, device="cuda")
    ws = store.workspace(T, k, 1)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def step():
        for g in range(n_groups):
            for l in range(L):
                api.si_ffn_forward(store.handle, l, x[g, l], T, idx if prefill else idx[g, l], None, k, y[g, l],
                                   flags, ws, status)

    warm = max(args.warmup, 3)
    for _ in range(warm):
        step()
    torch.cuda.synchronize(); replicas.barrier(); torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize(); replicas.barrier(); torch.cuda.synchronize()
    total_ms = replicas.max_over_ranks(e0.elapsed_time(e1), device="cuda")
    if int(status.item()) != 0:
        raise SystemExit(f"device status {status.item()}: {api.strerror(int(status.item()))}")
    if rank == 0:
        peaks, peak_kind = measured_peaks()
        tokens_per_step = n_groups * T
        tok_s = replicas.aggregate_throughput(tokens_per_step * args.steps, world, total_ms)
        u = float(np.mean(union_sizes))
        layer_calls = args.steps * n_groups * L
        us_per_layer = total_ms * 1e3 / layer_calls
        union_bytes = u * cfg.record_bytes
        flops = 6.0 * d * u * T
        out = {
            "metric": "selective_ffn_multitoken_tokens_per_s", "value": tok_s, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": warm, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": f"{cfg.name}: {L} layers d_model={d} d_ff={cfg.d_ff} {cfg.dtype}, "
                                   f"{cfg.n_loaded} loaded, T={T} tokens per call, "
                                   + ("one shared list of %d slots (prefill)" % k if prefill else
                                      "own %d-slot Zipf list per token (batched decode)" % k),
                       "mean_union": u, "union_overlap": None if prefill else 1.0 - u / (T * k),
                       "union_coverage_of_loaded": u / cfg.n_loaded, "us_per_layer_call": us_per_layer,
                       "l2": "weights of one pass exceed L2"},
            "gpu_launches": layer_calls * 3,
            "roofline": ({"bound": "tensor", "achieved": flops / us_per_layer / 1e6, "peak": peaks["bf16_tflops_sustained"],
                          "unit": "TFLOP/s", "frac": flops / us_per_layer / 1e6 / peaks["bf16_tflops_sustained"],
                          "peak_kind": f"of {peak_kind} (sustained)", "traffic": None} if prefill else
                         {"bound": "hbm", "achieved": union_bytes / us_per_layer / 1e3, "peak": peaks["hbm_gbs"],
                          "unit": "GB/s", "frac": union_bytes / us_per_layer / 1e3 / peaks["hbm_gbs"],
                          "peak_kind": f"of {peak_kind}", "traffic": None}),
        }
        print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=80, help="timed steps (launches) of the headline: 80 x 25 ms = 2 s")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c2", choices=sorted(wl.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (smaller captures)")
    ap.add_argument("--tokens", type=int, default=0, help="override the number of decode tokens per step")
    ap.add_argument("--loaded-pct", type=int, default=0)
    ap.add_argument("--active-pct", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0, help="c3: tokens processed together per step")
    ap.add_argument("--cpu-tokens", type=int, default=8, help="tokens of the oracle cpu_baseline sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-chained", action="store_true", help="skip the chained launch beside the headline")
    ap.add_argument("--no-extra-configs", action="store_true", help="skip the configs object (c1, c3, c4, c5)")
    ap.add_argument("--e2e-sizes", default="", help="tokens per chunk of the end-to-end pipeline, comma separated (default: derived)")
    ap.add_argument("--simple", action="store_true", help="time the per-step plain-load kernels instead")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="DRAM bytes per launch from an ncu capture (default: the committed capture of the "
                         "persistent kernel, scaled by the number of steps)")
    args = ap.parse_args()
    # started without a launcher: start the N ranks ourselves (each re-enters here with WORLD_SIZE set)
    rc = replicas.ensure_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:])
    if rc is not None:
        raise SystemExit(rc)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

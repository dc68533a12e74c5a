#!/usr/bin/env python
"""Benchmark of the selective-FFN hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2] [--impl ours|reference]

One "step" = one pass of the whole decode hot path over one batch of synthetic input: all
tokens of the workload through all FFN layers, each layer running the selective FFN on that
token's active list (one persistent launch through the C ABI).  The store is built once by
the loader before timing.  Metric: selective-FFN decode tokens/s at batch 1.

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) each rank is an independent replica
decoding its own tokens against its own copy of the store: no data-path collective, weak
scaling, time = max over ranks.
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
# dram__bytes_read.sum + dram__bytes_write.sum of si_decode_persistent_kernel per (token, layer) step
# of the config-2 shape, from the capture summarised in
# profiles/decode_persistent_c2_8layers_32tokens_full.md: (9.6461e9 + 0.2290e9) / 256 steps
NCU_DRAM_BYTES_PER_C2_STEP = (9.6454e9 + 0.2272e9) / 256
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
    any_ms, any_per, _ = timed(step_device_any_order, args.steps, max(args.warmup, 3))
    e2e_ms, _, _ = timed(step_e2e, args.steps, max(args.warmup, 3))
    if int(status.item()) != 0:
        raise SystemExit(f"device status {status.item()}: {api.strerror(int(status.item()))}")

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
            "gpu_launches": args.steps * (1 if not args.simple else 2 * n_steps),
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
        any_launch_ms = statistics.mean(any_per)
        out["steps_any_order"] = {
            "value": replicas.aggregate_throughput(tokens * args.steps, world, any_ms), "unit": UNIT,
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
        flags = api.SI_FLAG_UNION_PATH     # config 3 is about the union path (few tokens would otherwise take the decode route)
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
    ap.add_argument("--steps", type=int, default=10)
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
    ap.add_argument("--e2e-sizes", default="", help="tokens per chunk of the end-to-end pipeline, comma separated (default: derived)")
    ap.add_argument("--simple", action="store_true", help="time the per-step plain-load kernels instead")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="DRAM bytes per launch from an ncu capture (default: the committed capture of the "
                         "persistent kernel, scaled by the number of steps)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

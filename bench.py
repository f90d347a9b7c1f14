#!/usr/bin/env python
"""Benchmark of the chunked gated delta-rule prefill on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload long] [--impl ours|reference]

One step = one pass of the whole hot path (one layer's prefill call) over one batch
of seeded synthetic input.  Prints ONE JSON line.  The path does not shard (one GPU,
no collectives): with N > 1 every rank runs an independent replica of the workload
and the line reports the aggregate.  `--impl reference` times the fp64 CPU oracle on
the host cores instead (rank 0 only).
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

from workloads import get_config, make_inputs, widen  # noqa: E402

METRIC = "gdn_chunk_prefill_tokens_per_s_per_layer"
UNIT = "tokens/s"


# --------------------------------------------------------------------------------------------
# algorithmic work of one call (what the method itself must do; restructurings get no credit)
# --------------------------------------------------------------------------------------------
def algorithmic_work(cfg, lengths, with_initial_state):
    C, dk, dv, H = cfg.chunk, cfg.d_k, cfg.d_v, cfg.H
    e = 2 if cfg.dtype == "bf16" else 4
    tokens = int(sum(lengths))
    flops_per_th = 6 * C * dk + 4 * C * dv + 6 * dk * dv
    bytes_per_th = (2 * dk + dv) * e + dv * e + 8
    state_bytes = 4 * dk * dv * len(lengths) * H * (2 if with_initial_state else 1)
    return {"tokens": tokens, "flops": tokens * H * flops_per_th,
            "bytes": tokens * H * bytes_per_th + state_bytes}


def aggregate_over_ranks(local_ms, tokens_per_rank, steps, dist=None, device=None):
    """Replicas-only aggregation: every rank ran `steps` steps over its own copy of the workload.
    Job time = MAX over ranks of each local time; job tokens = sum over ranks.  `local_ms` is a
    list of per-rank-local millisecond totals (e.g. [device-resident, end-to-end]); returns
    (list of max-over-ranks ms, total tokens processed by the job)."""
    import torch
    world = dist.get_world_size() if dist is not None and dist.is_initialized() else 1
    ms = [float(x) for x in local_ms]
    tokens = float(tokens_per_rank) * steps
    if world > 1:
        t = torch.tensor(ms, dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = [float(x) for x in t]
        n = torch.tensor([tokens], dtype=torch.float64, device=device)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
        tokens = float(n[0])
    return ms, tokens


def ncu_traffic_bytes(workload):
    """DRAM bytes of one call (sum over its kernels) from the committed ncu summary, or None."""
    path = os.path.join(ROOT, "profiles", f"{workload}_dram_traffic.txt")
    if not os.path.exists(path):
        return None
    for line in open(path):
        parts = line.split()
        if len(parts) >= 2 and parts[0] == "total_bytes_per_call":
            return float(parts[1])
    return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


# --------------------------------------------------------------------------------------------
# clocks during the timed region
# --------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        rows = [r for (t, r) in self.rows if t0 - 0.05 <= t <= t1 + 0.15] or [r for (_, r) in self.rows]
        for r in rows:
            parts = [x.strip() for x in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax = float(parts[1])
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": smax,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------
# reference arm: the oracle, as it stands, on the host cores
# --------------------------------------------------------------------------------------------
def oracle_sample(cfg, x, budget_heads=None, form="sequential"):
    """Run the fp64 oracle (the sequential recurrence, or its chunked form) on a bounded sample
    (whole (sequence, head) chains).  Returns (seconds, tokens of full-H work the sample stands for, heads, threads)."""
    import oracle
    H = cfg.H
    heads = H if budget_heads is None else min(H, budget_heads)
    sl = (slice(None),) * (x.q.ndim - 2) + (slice(0, heads),)
    q, k, v = widen(x.q[sl]), widen(x.k[sl]), widen(x.v[sl])
    la, be = x.log_alpha[sl], x.beta[sl]
    s0 = None if x.initial_state is None else x.initial_state[:, :heads]
    t0 = time.perf_counter()
    if form == "sequential":
        oracle.sequential(q, k, v, la, be, s0, x.cu_seqlens)
    else:
        oracle.chunked(q, k, v, la, be, s0, x.cu_seqlens, chunk=cfg.chunk)
    dt = time.perf_counter() - t0
    tokens_equiv = sum(x.lengths) * heads / H        # tokens of full-H work this sample stands for
    return dt, tokens_equiv, heads, oracle.num_threads()


def cpu_baseline(cfg, x, reps=3):
    """The oracle as it stands on the host cores: one untimed warm-up call, then the median of `reps` calls,
    for the sequential recurrence (the definition) and for its chunked form."""
    heads = cfg.H if cfg.d_v <= 128 and sum(x.lengths) <= 16384 else 4
    res = {}
    for form in ("sequential", "chunked"):
        oracle_sample(cfg, x, 1, form)
        runs, spent = [], 0.0
        while len(runs) < reps and (not runs or spent < 8.0):      # bounded: large samples are not repeated
            runs.append(oracle_sample(cfg, x, heads, form))
            spent += runs[-1][0]
        dt = float(np.median([r[0] for r in runs]))
        res[form] = (runs[0][1] / dt, dt, runs[0][2], runs[0][3])
    v, dt, heads, cores = res["sequential"]
    return {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{heads} of {cfg.H} heads, all tokens, sequential fp64 recurrence, median of up to {reps} warmed calls "
                      f"({dt:.2f} s each); tokens scaled by heads/H",
            "chunked_oracle_value": res["chunked"][0],
            "chunked_oracle_sample": f"same sample through the fp64 chunked form ({res['chunked'][1]:.2f} s per call)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = get_config(args.workload)
    x = make_inputs(cfg)
    heads = cfg.H if cfg.d_v <= 128 and sum(x.lengths) <= 16384 else 4
    for _ in range(args.warmup):
        oracle_sample(cfg, x, 1)
    total_t, total_tok, cores = 0.0, 0.0, 1
    for _ in range(args.steps):
        dt, tok, heads, cores = oracle_sample(cfg, x, heads)
        total_t += dt
        total_tok += tok
    value = total_tok / total_t
    sample = f"{heads} of {cfg.H} heads, all tokens, sequential fp64 recurrence; tokens scaled by heads/H"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(cfg, x),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(cfg, x):
    return {"workload": cfg.name, "B": cfg.B, "T": x.T_arg, "H": cfg.H, "d_k": cfg.d_k, "d_v": cfg.d_v,
            "chunk": cfg.chunk, "storage": cfg.dtype, "packed": cfg.packed, "seed": cfg.seed,
            "initial_state": x.initial_state is not None,
            "l2": "flushed between timed steps (256 MiB write)", "parallelism": "replicas only"}


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2607_14568_b200 as gdn

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    overrides = {k: int(v) for k, v in (kv.split("=") for kv in args.reduce.split(",") if kv)}
    cfg = get_config(args.workload, **overrides)
    x = make_inputs(cfg)
    work = algorithmic_work(cfg, x.lengths, x.initial_state is not None)
    peaks = measured_peaks()

    def dev_t(a):
        if a is None:
            return None
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
        return torch.from_numpy(a)

    host = {k: dev_t(getattr(x, k)) for k in ("q", "k", "v", "log_alpha", "beta", "initial_state", "cu_seqlens")}
    d = {k: (None if v is None else v.to(dev)) for k, v in host.items()}
    N = len(x.lengths)
    out = torch.empty_like(d["v"])
    fin = torch.empty((N, cfg.H, cfg.d_k, cfg.d_v), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    fn = gdn.gdn_chunk_prefill if cfg.dtype == "bf16" else gdn.gdn_chunk_prefill_f32
    # scratch for the two-kernel pipeline (the library allocates nothing itself)
    ws_bytes = 0
    if cfg.dtype == "bf16" and not args.no_workspace:
        ws_bytes = gdn.gdn_workspace_bytes(cfg.B, x.T_arg, cfg.H, cfg.d_k, cfg.d_v, cfg.packed)
        if ws_bytes:
            gdn.gdn_set_workspace(torch.empty(ws_bytes, dtype=torch.uint8, device=dev))

    def step():
        fn(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"], out, fin, d["cu_seqlens"],
           stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        flush.fill_(1)
        step()
    barrier()

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    l0 = gdn.gdn_launch_count()
    t0 = time.time()
    for i in range(args.steps):
        flush.fill_(i & 0xFF)            # evict the inputs from L2 (not timed)
        starts[i].record(stream)
        step()
        stops[i].record(stream)
    barrier()
    t1 = time.time()
    launches = gdn.gdn_launch_count() - l0
    clocks = sampler.stop(t0, t1)
    ms = [s.elapsed_time(e) for s, e in zip(starts, stops)]
    total_ms = float(sum(ms))
    # warm-L2 figure for information (no flush between calls; inputs that fit in L2 stay there)
    ws_, we_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ws_.record(stream)
    for i in range(args.steps):
        step()
    we_.record(stream)
    barrier()
    ms_warm_l2 = ws_.elapsed_time(we_) / args.steps

    # ---- end to end through the host-buffer entry point (pinned host memory) ----
    hp = {k: (None if v is None else v.pin_memory()) for k, v in host.items()}
    out_h = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    fin_h = torch.empty(fin.shape, dtype=fin.dtype).pin_memory()
    e2e = None
    if cfg.dtype == "bf16":
        nbytes = gdn.gdn_host_staging_bytes(cfg.B, x.T_arg, cfg.H, cfg.d_k, cfg.d_v)
        staging = torch.empty(nbytes, dtype=torch.uint8, device=dev)

        def e2e_step():
            gdn.gdn_chunk_prefill_host(hp["q"], hp["k"], hp["v"], hp["log_alpha"], hp["beta"], hp["initial_state"],
                                       out_h, fin_h, hp["cu_seqlens"], staging, stream=stream)
        for _ in range(2):
            e2e_step()
        barrier()
        es, ee = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        es.record(stream)
        for _ in range(args.steps):
            e2e_step()
        ee.record(stream)
        barrier()
        e2e_ms = es.elapsed_time(ee)
        h2d = sum(v.numel() * v.element_size() for v in hp.values() if v is not None)
        d2h = out_h.numel() * out_h.element_size() + fin_h.numel() * fin_h.element_size()
    else:
        e2e_ms, h2d, d2h = None, 0, 0

    # ---- per-kernel breakdown (separate, untimed pass; events recorded inside the library) ----
    kernels = None
    if ws_bytes and gdn.lib().gdn_debug_set_timing(1) == 0:
        import ctypes
        acc = np.zeros(5)
        buf = (ctypes.c_float * 5)()
        for i in range(args.steps):
            flush.fill_(i & 0xFF)
            step()
            if gdn.lib().gdn_debug_get_timing(buf) == 0:
                acc += np.array(list(buf))
        gdn.lib().gdn_debug_set_timing(0)
        tot = float(acc.sum())
        if tot > 0:
            names = ("gdn_prep_kernel", "gdn_summary_kernel", "gdn_combine_kernel", "gdn_chain_kernel", "gdn_scan_kernel")
            kernels = {n: {"ms": float(a) / args.steps, "share": float(a) / tot} for n, a in zip(names, acc) if a > 0}

    # ---- aggregate over ranks: max time, summed tokens ----
    (total_ms, e2e_max), tokens_job = aggregate_over_ranks([total_ms, e2e_ms or 0.0], work["tokens"], args.steps,
                                                           dist if world > 1 else None, dev)
    e2e_ms = e2e_max if e2e_ms is not None else None
    value = tokens_job / (total_ms * 1e-3)
    if e2e_ms is not None:
        e2e = {"value": tokens_job / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)}

    if rank == 0:
        ms_step = total_ms / args.steps
        t_hbm = work["bytes"] / (peaks["hbm_gbs"] * 1e9)
        t_tc = work["flops"] / (peaks["bf16_tflops"] * 1e12)
        bound = "hbm" if t_hbm >= t_tc else "tensor"
        per_launch_s = (float(np.mean(ms)) * 1e-3)
        if bound == "hbm":
            achieved, peak, unit = work["bytes"] / per_launch_s / 1e9, peaks["hbm_gbs"], "GB/s"
        else:
            achieved, peak, unit = work["flops"] / per_launch_s / 1e12, peaks["bf16_tflops"], "TFLOP/s"
        if kernels:
            # caller tensors each kernel has to touch (scratch traffic is not algorithmic): the prepare kernel reads
            # q, k and the gates; the summary kernel k and v; the combine kernel the states; the chain (or merged
            # scan) kernel q, k, v, writes out and carries the states
            e = 2 if cfg.dtype == "bf16" else 4
            th = work["tokens"] * cfg.H
            st = 4 * cfg.d_k * cfg.d_v * N * cfg.H
            kb = {"gdn_prep_kernel": th * (2 * cfg.d_k * e + 8), "gdn_summary_kernel": th * (cfg.d_k + cfg.d_v) * e,
                  "gdn_combine_kernel": st * (2 if x.initial_state is not None else 1),
                  "gdn_chain_kernel": th * (2 * cfg.d_k + 2 * cfg.d_v) * e + st * (2 if x.initial_state is not None else 1),
                  "gdn_scan_kernel": th * (2 * cfg.d_k + 2 * cfg.d_v) * e + st * (2 if x.initial_state is not None else 1)}
            for name, kk in kernels.items():
                kk["algorithmic_bytes"] = int(kb[name])
                kk["achieved_gbs"] = kb[name] / (kk["ms"] * 1e-3) / 1e9
                kk["frac"] = kk["achieved_gbs"] / peaks["hbm_gbs"]
        dominant = max(kernels, key=lambda k: kernels[k]["ms"]) if kernels else None
        roofline = {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
                    "traffic": ncu_traffic_bytes(cfg.name), "peak_source": peaks["source"],
                    "kernel": "whole call: algorithmic bytes of the path / time of all kernels of one gdn_chunk_prefill",
                    "kernels": kernels, "dominant_kernel": dominant,
                    "algorithmic_bytes": work["bytes"], "algorithmic_flops": work["flops"],
                    "roofline_us": 1e6 * max(t_hbm, t_tc)}
        # CPU baseline: the oracle as it stands, bounded sample, host cores
        cpu = cpu_baseline(cfg, x)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
                "data": "synthetic", "config": dict(workload_config(cfg, x), workspace_bytes=int(ws_bytes),
                                                    **({"reduced": args.reduce} if args.reduce else {})),
                "clocks": clocks, "e2e": e2e,
                "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
                "ms_min": float(min(ms)), "ms_median": float(np.median(ms)),
                "ms_warm_l2": float(ms_warm_l2)}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_decode(args):
    """Secondary line: one decode step (state streamed once in, once out), B = 256 sequences."""
    import torch

    import paper_2607_14568_b200 as gdn
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    B, H, dk, dv = 256, 16, 128, 128
    g = torch.Generator(device="cuda").manual_seed(0)
    q = torch.nn.functional.normalize(torch.randn(B, H, dk, device="cuda", generator=g), dim=-1).bfloat16()
    k = torch.nn.functional.normalize(torch.randn(B, H, dk, device="cuda", generator=g), dim=-1).bfloat16()
    v = torch.randn(B, H, dv, device="cuda", generator=g).bfloat16()
    la = -torch.nn.functional.softplus(torch.randn(B, H, device="cuda", generator=g)) * 0.05
    be = torch.sigmoid(torch.randn(B, H, device="cuda", generator=g))
    state = torch.randn(B, H, dk, dv, device="cuda", generator=g) * 0.02
    out = torch.empty_like(v)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for _ in range(max(args.warmup, 3)):
        gdn.gdn_decode_step(q, k, v, la, be, state, out)
    torch.cuda.synchronize()
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    time.sleep(0.25)
    l0 = gdn.gdn_launch_count()
    t0 = time.time()
    for a, b in ev:
        flush.fill_(1)
        a.record()
        gdn.gdn_decode_step(q, k, v, la, be, state, out)
        b.record()
    torch.cuda.synchronize()
    t1 = time.time()
    launches = gdn.gdn_launch_count() - l0
    clocks = sampler.stop(t0, t1)
    ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
    nbytes = 2 * B * H * dk * dv * 4 + B * H * ((2 * dk + 2 * dv) * 2 + 8)
    peaks = measured_peaks()
    gbs = nbytes / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "gdn_decode_step_tokens_per_s", "value": B / (ms * 1e-3), "unit": "tokens/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
                      "higher_is_better": True, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": "decode", "B": B, "H": H, "d_k": dk, "d_v": dv,
                                 "l2": "flushed between timed steps (256 MiB write)"},
                      "clocks": clocks, "gpu_launches": int(launches),
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": gbs / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
                                   "kernel": "gdn_decode_kernel", "algorithmic_bytes": nbytes}}), flush=True)


def run_attention(args):
    """Secondary line: causal grouped-query attention of one attention layer at a prompt tier
    (attn_10k: T = 10240, 16 query heads on 8 key/value heads, d = 128)."""
    import torch

    import paper_2607_14568_b200 as gdn
    from workloads import get_attn_config, make_attn_inputs
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    name = "attn_2k" if args.workload == "attention_2k" else "attn_10k"
    cfg = get_attn_config(name)
    q, k, v = (torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda() for a in make_attn_inputs(cfg))
    out = torch.empty_like(q)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for _ in range(max(args.warmup, 3)):
        gdn.gdn_attn_causal_prefill(q, k, v, out, cfg.scale)
    torch.cuda.synchronize()
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    time.sleep(0.25)
    t0 = time.time()
    for a, b in ev:
        flush.fill_(1)
        a.record()
        gdn.gdn_attn_causal_prefill(q, k, v, out, cfg.scale)
        b.record()
    torch.cuda.synchronize()
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    assert gdn.gdn_query_status() == 0
    ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
    # algorithmic flops: two products of 2*d flops per (query, visible key) pair and query head
    flops = cfg.B * cfg.Hq * 2 * (2 * cfg.d) * (cfg.T * (cfg.T + 1) // 2)
    peaks = measured_peaks()
    tf = flops / (ms * 1e-3) / 1e12
    print(json.dumps({"metric": "attn_causal_prefill_tokens_per_s_per_layer", "value": cfg.B * cfg.T / (ms * 1e-3),
                      "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
                      "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": name, "B": cfg.B, "T": cfg.T, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "d": cfg.d,
                                 "l2": "flushed between timed steps (256 MiB write)"},
                      "clocks": clocks, "gpu_launches": args.steps,
                      "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                   "frac": tf / peaks["bf16_tflops"], "traffic": None, "peak_source": peaks["source"],
                                   "kernel": "attn_causal_kernel", "algorithmic_flops": flops}}), flush=True)


def replica_launch_command(n_gpus, argv, port=None):
    """The command that starts `n_gpus` replica processes of this script on one node (one rank per GPU,
    rendezvous on 127.0.0.1), as the driver's launcher would."""
    if port is None:
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="long", help="long (T=10240, the metric's configuration), short, serving, large; secondary lines: decode, "
                    "attention (T=10240), attention_2k")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-workspace", action="store_true", help="run the fused single-kernel path (no scratch)")
    ap.add_argument("--reduce", default="", help="profiling only: a reduced copy of the workload, e.g. B=1,T=4096 "
                    "(the line then names the reduced shape in config; it is not the benchmark configuration)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # not started by a launcher: start one replica process per GPU ourselves (rank 0 prints the line)
        raise SystemExit(subprocess.call(replica_launch_command(args.gpus, sys.argv[1:])))
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "decode":
        run_decode(args)
    elif args.workload in ("attention", "attention_2k"):
        run_attention(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

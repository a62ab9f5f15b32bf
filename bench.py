#!/usr/bin/env python
"""Benchmark of the D-Quant hot path on B200: decode-attention KV tokens/s over the compressed
cache (2.26 bits/element), with the encoder on the step's new tokens.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--config 2|3|4|5] [--budget 2.26] [--streams head|token]

One *step* = one decode step of the whole hot path: encode one new token per sequence (K and
V: Hadamard, mean removal, drift, rANS) into the cache, then decode-step attention over every
cached token of every sequence.  KV tokens per step = sum of sequence lengths.  Prints ONE
JSON line (rank 0).  With N > 1 (torchrun) every rank runs an independent replica on its own
GPU (the path has no exchange step): weak scaling, max time over ranks.

`--impl reference` times the CPU oracle (as it stands) on a bounded sample of the same
workload, on the host cores, without touching the GPU.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attention_kv_tokens_per_s"
UNIT = "KV tokens/s"
L2_BYTES = 126 * 2 ** 20
# Algorithmic integer work of Algorithm 2 per decoded symbol (lane operations): slot mask,
# table address, table read, two field extracts, state shift, multiply-add, compare with L,
# byte merge, pointer advance.
ALU_OPS_PER_SYMBOL = 10.0
SM_COUNT, LANES_PER_SM_CLK = 148, 128


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1965.0, "fallback"


class ClockSampler(threading.Thread):
    """Polls SM clock, power and throttle reasons through NVML (read-only) while running."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period, self.samples, self._stop_evt = index, period_s, [], threading.Event()
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        while not self._stop_evt.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                power = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                self.samples.append((time.time(), mhz, reasons, power))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)

    def summary(self, t0=None, t1=None):
        if self.nv is None or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml unavailable"]}
        nv = self.nv
        sel = [s for s in self.samples if (t0 is None or s[0] >= t0) and (t1 is None or s[0] <= t1)] or self.samples
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        seen = set()
        for _, _, r, _ in sel:
            for bit, name in names.items():
                if r & bit:
                    seen.add(name)
        return {"sm_mhz": statistics.median(s[1] for s in sel), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(seen), "samples": len(sel), "power_w_max": max(s[3] for s in sel)}


# --------------------------------------------------------------------------- CPU oracle leg

def stream_setup(cfg, streams: str):
    """Record sizes, level counts and heads per stream of the run: the benchmark's per token-head
    streams at the requested budget, or the paper's default grouping (one stream per token:
    335 / 235-byte records = 331 / 231-byte containers, 8 / 6 levels)."""
    if streams == "token":
        hs = cfg.hkv
        assert hs <= 8, "a token-wide stream holds at most 1024 values"
        return dict(hs=hs, k_rec=335 * hs // 8, v_rec=235 * hs // 8, k_levels=8, v_levels=6, alpha=1.4)
    return dict(hs=1, k_rec=cfg.k_rec, v_rec=cfg.v_rec, k_levels=cfg.k_levels, v_levels=cfg.v_levels, alpha=cfg.alpha)


def oracle_step_runner(cfg_idx: int, budget: float, streams: str = "head"):
    """Builds the bounded oracle sample (sequence 0 of the workload, all KV heads) and returns
    (step function, KV tokens per step, description).  GPU-free."""
    import numpy as np
    import oracle
    from paper_2609_19880_b200 import workloads

    cfg = workloads.make_config(cfg_idx, budget=budget)
    cfg.batch, cfg.seq_lens = 1, [min(cfg.seq_lens[0], 8192)]
    w = workloads.generate(cfg, device="cpu")
    st = stream_setup(cfg, streams)
    ok = oracle.build_table(st["k_levels"], 128 * st["hs"], st["k_rec"], st["alpha"], has_mean=True, rotate=True)
    ov = oracle.build_table(st["v_levels"], 128 * st["hs"], st["v_rec"], st["alpha"], has_mean=False, rotate=True)
    kb, vb, qb = workloads.bf16_bits(w.k), workloads.bf16_bits(w.v), workloads.bf16_bits(w.q)
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    mq = np.zeros((1, w.max_windows, cfg.hkv, 128), np.int8)
    ms = np.zeros((1, w.max_windows, cfg.hkv), np.float32)
    oracle.window_means(kb, seq_id, pos, mq, ms, 0)
    kc = np.zeros((w.num_pages, cfg.hkv // st["hs"], 16, ok.rec), np.uint8)
    vc = np.zeros((w.num_pages, cfg.hkv // st["hs"], 16, ov.rec), np.uint8)
    oracle.encode_tokens(ok, kb, seq_id, pos, slot, kc, mq, ms)
    oracle.encode_tokens(ov, vb, seq_id, pos, slot, vc)
    last = slice(cfg.total_tokens - 1, cfg.total_tokens)
    pt, sl = w.page_table.numpy(), w.seq_lens.numpy()
    sm = 1.0 / math.sqrt(128.0)

    def step():
        oracle.window_means(kb[last], seq_id[last], pos[last], mq, ms, 1)
        oracle.encode_tokens(ok, kb[last], seq_id[last], pos[last], slot[last], kc, mq, ms)
        oracle.encode_tokens(ov, vb[last], seq_id[last], pos[last], slot[last], vc)
        return oracle.attention(ok, ov, qb, kc, vc, mq, ms, pt, sl, cfg.hkv, sm)

    desc = (f"sequence 0 of {cfg.name}: {cfg.seq_lens[0]} tokens x {cfg.hkv} KV heads x {cfg.hq} query heads, "
            f"encode 1 token + fp64 attention per step")
    return step, cfg.seq_lens[0], desc, oracle.num_threads()


def time_oracle(cfg_idx, budget, budget_s=10.0, max_steps=1000, warmup=1, streams="head"):
    step, toks, desc, cores = oracle_step_runner(cfg_idx, budget, streams)
    for _ in range(warmup):
        step()
    n, t0 = 0, time.perf_counter()
    while True:
        step()
        n += 1
        dt = time.perf_counter() - t0
        if dt >= budget_s or n >= max_steps:
            break
    return {"value": toks * n / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{desc}; {n} steps in {dt:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    step, toks, desc, cores = oracle_step_runner(args.config, args.budget, args.streams)
    for _ in range(max(args.warmup, 1)):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    val = toks * args.steps / dt
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config {args.config} at {args.budget} bits/elem, bounded sample: {desc}"},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------- GPU leg

def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """Slowest rank's figure (every rank gets it).  Replicas share nothing else."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank_per_step: float, seconds_per_step: float, world: int) -> float:
    """Whole-job rate of `world` independent replicas timed by the slowest one (weak scaling)."""
    return world * units_per_rank_per_step / seconds_per_step


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2609_19880_b200 as dq
    from paper_2609_19880_b200 import _build, workloads

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if not os.path.exists(dq.LIB_PATH):
        _build.build()
    dq.lib()
    dev = torch.device("cuda", local)
    hbm_peak, sm_max_mhz, peak_kind = _peaks()

    cfg = workloads.make_config(args.config, budget=args.budget)
    w = workloads.generate(cfg, device=dev)
    B, Hq, Hkv = cfg.batch, cfg.hq, cfg.hkv
    st = stream_setup(cfg, args.streams)
    hs, k_rec, v_rec = st["hs"], st["k_rec"], st["v_rec"]
    n_stream = 128 * hs
    tk = dq.dq_build_tables(st["k_levels"], k_rec * 8 / n_stream, alpha=st["alpha"], has_mean=True, rotate=True,
                            heads_per_stream=hs)
    tv = dq.dq_build_tables(st["v_levels"], v_rec * 8 / n_stream, alpha=st["alpha"], has_mean=False, rotate=True,
                            heads_per_stream=hs)
    assert tk.info().rec_bytes == k_rec and tv.info().rec_bytes == v_rec
    sm_scale = 1.0 / math.sqrt(128.0)

    token_heads = cfg.total_tokens * Hkv
    # bytes one token-head occupies in the cache (token-wide records are padded to whole words)
    k_b = k_rec if hs == 1 else 4 * tk.info().rec_words / hs
    v_b = v_rec if hs == 1 else 4 * tv.info().rec_words / hs
    cache_bytes = int(token_heads * (k_b + v_b)) + B * w.max_windows * Hkv * 132
    copies = max(2, math.ceil(2.2 * L2_BYTES / cache_bytes)) if cache_bytes < 2 * L2_BYTES else 1

    def new_cache():
        return dict(
            k=torch.zeros((w.num_pages, Hkv, 16, k_rec) if hs == 1 else (w.num_pages, Hkv // hs, tk.info().rec_words, 16, 4),
                          dtype=torch.uint8, device=dev),
            v=torch.zeros((w.num_pages, Hkv, 16, v_rec) if hs == 1 else (w.num_pages, Hkv // hs, tv.info().rec_words, 16, 4),
                          dtype=torch.uint8, device=dev),
            mq=torch.zeros((B, w.max_windows, Hkv, 128), dtype=torch.int8, device=dev),
            ms=torch.zeros((B, w.max_windows, Hkv), dtype=torch.float32, device=dev))

    # ---- prefill encode (timed once; also fills the cache the decode steps read)
    caches = [new_cache()]
    c0 = caches[0]
    dq.dq_encode_tokens(tk, tv, w.k, w.v, w.seq_id, w.pos, w.slot, c0["k"], c0["v"], c0["mq"], c0["ms"])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    dq.dq_encode_tokens(tk, tv, w.k, w.v, w.seq_id, w.pos, w.slot, c0["k"], c0["v"], c0["mq"], c0["ms"])
    e1.record()
    torch.cuda.synchronize()
    enc_ms = e0.elapsed_time(e1)
    for _ in range(copies - 1):
        caches.append({k: v.clone() for k, v in c0.items()})

    # ---- the step's inputs: q and one new token per sequence (the last position)
    lens = torch.tensor(cfg.seq_lens, dtype=torch.int64)
    last_idx = (torch.cumsum(lens, 0) - 1).to(dev)
    new_k, new_v = w.k[last_idx].contiguous(), w.v[last_idx].contiguous()
    new_seq, new_pos, new_slot = (t[last_idx].contiguous() for t in (w.seq_id, w.pos, w.slot))
    out = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device=dev)
    ws = torch.empty(dq.dq_decode_workspace_bytes(B, Hq, w.page_table.shape[1]), dtype=torch.uint8, device=dev)
    kv_tokens = cfg.total_tokens

    state = {"r": 0, "closes": 0}
    if hs == 1:
        if args.separate_calls:
            def step(i, q=w.q, nk=new_k, nv=new_v):
                c = caches[i % copies]
                dq.dq_encode_tokens(tk, tv, nk, nv, new_seq, new_pos, new_slot, c["k"], c["v"], c["mq"], c["ms"],
                                    dq.MEAN_REUSE)
                dq.dq_decode_attention(tk, tv, q, c["k"], c["v"], c["mq"], c["ms"], w.page_table, w.seq_lens, Hkv,
                                       sm_scale, out, ws)
            step_desc = "encode 1 new token per sequence + decode attention over the whole cache (two calls)"
        else:
            # the same work through the one-call step API: the attention kernel starts beside the encoder
            def step(i, q=w.q, nk=new_k, nv=new_v):
                c = caches[i % copies]
                dq.dq_decode_step(tk, tv, nk, nv, new_slot, q, c["k"], c["v"], c["mq"], c["ms"], w.page_table,
                                  w.seq_lens, Hkv, sm_scale, out, ws)
            step_desc = ("encode 1 new token per sequence + decode attention over the whole cache "
                         "(dq_decode_step: attention starts while the encoder runs)")
        launches_per_step = 4   # encode (K and V), prepare, fused attention, combine
    else:
        # The paper's serving policy (Sec. 5.1): the newest tokens stay in a 128-token BF16 window that
        # joins the attention; when the window is full its 128 tokens per sequence are encoded in one
        # call with their own channel mean (here: over the last window of the cache, so the context
        # stays at its configured length) and the window restarts.
        rk = torch.zeros((B, 128, Hkv, 128), dtype=torch.bfloat16, device=dev)
        rv = torch.zeros_like(rk)
        rl = torch.zeros(B, dtype=torch.int32, device=dev)     # tokens in the window, kept on the device
        win_idx = torch.cat([torch.arange(int(e) - 128, int(e)) for e in torch.cumsum(lens, 0)]).to(dev)
        win_seq, win_pos, win_slot = (t[win_idx].contiguous() for t in (w.seq_id, w.pos, w.slot))

        def step_core(i, q=w.q, nk=new_k, nv=new_v):   # the same launches every step (the counts live on the device)
            c = caches[i % copies]
            dq.dq_window_append(nk, nv, rk, rv, rl)
            dq.dq_decode_attention_residual(tk, tv, q, c["k"], c["v"], c["mq"], c["ms"], w.page_table, w.seq_lens,
                                            rk, rv, rl, Hkv, sm_scale, out, ws)

        def step_close(i):                             # after every 128th step: the full window becomes compressed
            state["r"] += 1
            if state["r"] == 128:
                c = caches[i % copies]
                dq.dq_encode_tokens(tk, tv, rk.view(B * 128, Hkv, 128), rv.view(B * 128, Hkv, 128), win_seq, win_pos,
                                    win_slot, c["k"], c["v"], c["mq"], c["ms"], dq.MEAN_COMPUTE)
                rl.zero_()
                state["closes"] += 1
                state["r"] = 0

        def step(i, q=w.q, nk=new_k, nv=new_v):
            step_core(i, q, nk, nv)
            step_close(i)
        launches_per_step = 4 + 3.0 / 128   # window append, prepare, fused attention, combine; means + K/V encode per 128 steps
        step_desc = ("append the new token to a 128-token BF16 window + decode attention over the compressed cache "
                     "and the window; a full window is encoded in bulk (once per 128 steps)")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()

    # ---- timed region: exactly K steps, CUDA events on the launch stream
    # CUDA events around the fused kernel of every prof_period-th step (the events serialise that step's
    # kernels, ~20 us each time, so they are kept sparse; at least 4 samples)
    prof_period = max(1, min(int(os.environ.get("DQ_BENCH_PROFILE_PERIOD", "16")), args.steps // 4))
    dq.dq_profile_enable(prof_period)
    t_wall0 = time.time()
    closes0 = state["closes"]
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    closes_timed = state["closes"] - closes0
    barrier()
    t_wall1 = time.time()
    total_ms = e0.elapsed_time(e1)
    kern_ms = dq.dq_profile_read(4096)
    dq.dq_profile_enable(False)
    total_ms = max_over_ranks(total_ms, world, dev)
    ms_per_step = total_ms / args.steps
    value = job_throughput(kv_tokens, ms_per_step * 1e-3, world)

    if args.profile_only:   # short run for an ncu capture: no soak, no e2e, no baselines
        sampler.stop()
        if rank == 0:
            print(json.dumps({"profile_only": True, "ms_per_step": ms_per_step,
                              "kernel_ms": statistics.mean(kern_ms) if kern_ms else None}), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return

    # keep the same load running briefly so the clock sampler sees it (not part of any number)
    if t_wall1 - t_wall0 < 0.5:
        t_end = time.time() + 0.6
        i = 0
        while time.time() < t_end:
            for _ in range(50):
                step(i); i += 1
            torch.cuda.synchronize()
        t_wall1 = time.time()
    sampler.stop()
    clocks = sampler.summary(t_wall0, t_wall1)

    # ---- end to end: host buffers in, host buffer out, every step
    # The step's inputs (q and the new token's K / V) sit in ONE pinned host buffer and cross in one
    # copy; the device-side tensors are views of one staging buffer.
    nq, nkv = w.q.numel(), new_k.numel()
    hin = torch.empty(nq + 2 * nkv, dtype=torch.bfloat16).pin_memory()
    hin[:nq].copy_(w.q.reshape(-1)); hin[nq:nq + nkv].copy_(new_k.reshape(-1)); hin[nq + nkv:].copy_(new_v.reshape(-1))
    din = torch.empty(nq + 2 * nkv, dtype=torch.bfloat16, device=dev)
    dq_q, dk, dv = din[:nq].view_as(w.q), din[nq:nq + nkv].view_as(new_k), din[nq + nkv:].view_as(new_v)
    hout = torch.empty((B, Hq, 128), dtype=torch.bfloat16).pin_memory()
    h2d = hin.numel() * 2
    d2h = hout.numel() * 2

    # One CUDA graph per cache copy holds the whole step (H2D copy, the library's launches, D2H copy).
    graphs, graph_note = None, "direct launches"
    core = step if hs == 1 else step_core
    if not args.no_graph:
        try:
            torch.cuda.synchronize()
            graphs = []
            for c_i in range(copies):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    din.copy_(hin, non_blocking=True)
                    core(c_i, dq_q, dk, dv)
                    hout.copy_(out, non_blocking=True)
                graphs.append(g)
            graph_note = f"one CUDA graph per cache copy ({copies})"
            if hs > 1:
                graph_note += "; the window's bulk encode every 128 steps is launched directly"
                rl.zero_()            # the captures' warm-up runs appended tokens
                state["r"] = 0
        except Exception as ex:   # capture is an optimisation of the launch path only
            graphs, graph_note = None, f"direct launches (graph capture failed: {type(ex).__name__})"
            torch.cuda.synchronize()

    def e2e_step(i):
        if graphs is not None:
            graphs[i % copies].replay()
        else:
            din.copy_(hin, non_blocking=True)
            core(i, dq_q, dk, dv)
            hout.copy_(out, non_blocking=True)
        if hs > 1:
            step_close(i)
        torch.cuda.synchronize()

    for i in range(3):
        e2e_step(i)
    barrier()
    t0 = time.perf_counter()
    for i in range(args.steps):
        e2e_step(i)
    barrier()
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s, world, dev)
    e2e_value = job_throughput(kv_tokens, e2e_s / args.steps, world)
    # what came back to the host must be what a direct call computes (same inputs, same cache contents)
    e2e_check = None
    if hs == 1:
        step(0)
        torch.cuda.synchronize()
        e2e_check = bool(torch.equal(hout, out.cpu()))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (fused decode attention)
    k_ms = statistics.mean(kern_ms) if kern_ms else None
    symbols = token_heads * 256.0
    comp_bytes = token_heads * (k_b + v_b + 1.0)   # records + amortised INT8 mean byte
    roofline = None
    extra = {}
    if args.traffic_bytes is None:
        # ncu, config 2: dram__bytes_read + write = 37.62 MB for 524288 token-heads at 42 + 29 byte records;
        # the kernel reads every record once, so traffic grows with the records' bytes
        args.traffic_bytes = 37.62e6 * (token_heads * (k_b + v_b + 1.0)) / (524288 * 72.0)
    if k_ms:
        alu_peak = SM_COUNT * LANES_PER_SM_CLK * sm_max_mhz * 1e6 / 1e9          # G lane-ops / s
        alu_ach = symbols * ALU_OPS_PER_SYMBOL / (k_ms * 1e-3) / 1e9
        gbs = comp_bytes / (k_ms * 1e-3) / 1e9
        roofline = {"bound": "alu", "achieved": alu_ach, "peak": alu_peak, "unit": "Gop/s (int32 lane ops)",
                    "frac": alu_ach / alu_peak, "traffic": args.traffic_bytes,
                    "kernel": "dq_attention_kernel" if hs == 1 else "dq_attention_wide_kernel", "kernel_ms": k_ms, "launches_timed": len(kern_ms),
                    "peak_source": f"148 SM x 128 lanes x {sm_max_mhz:.0f} MHz ({peak_kind} clocks)",
                    "ops_per_symbol": ALU_OPS_PER_SYMBOL}
        extra = {"hbm": {"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gbs / hbm_peak,
                         "frac_of_8TBps": gbs / 8000.0, "peak_source": peak_kind,
                         "bytes_per_token_head": k_b + v_b + 1},
                 "kernel_token_heads_per_s": token_heads / (k_ms * 1e-3),
                 "kernel_symbols_per_s": symbols / (k_ms * 1e-3)}

    # ---- bf16-cache baseline on the same GPU (context)
    bf16 = None
    try:
        kp = torch.zeros((w.num_pages * 16, Hkv, 128), dtype=torch.bfloat16, device=dev)
        vp = torch.zeros_like(kp)
        kp[w.slot.long()] = w.k
        vp[w.slot.long()] = w.v
        kp = kp.view(w.num_pages, 16, Hkv, 128).transpose(1, 2).contiguous()
        vp = vp.view(w.num_pages, 16, Hkv, 128).transpose(1, 2).contiguous()
        bcopies = max(1, math.ceil(2.2 * L2_BYTES / (kp.numel() * 4)))
        kps, vps = [kp] + [kp.clone() for _ in range(bcopies - 1)], [vp] + [vp.clone() for _ in range(bcopies - 1)]
        for i in range(3):
            dq.dq_bf16_decode_attention(w.q, kps[i % bcopies], vps[i % bcopies], w.page_table, w.seq_lens, Hkv,
                                        sm_scale, out, ws)
        torch.cuda.synchronize()
        nb = 50
        e0.record()
        for i in range(nb):
            dq.dq_bf16_decode_attention(w.q, kps[i % bcopies], vps[i % bcopies], w.page_table, w.seq_lens, Hkv,
                                        sm_scale, out, ws)
        e1.record()
        torch.cuda.synchronize()
        bms = e0.elapsed_time(e1) / nb
        bf16 = {"ms_per_call": bms, "kv_tokens_per_s": kv_tokens / (bms * 1e-3),
                "gb_per_s": token_heads * 512.0 / (bms * 1e-3) / 1e9, "bytes_per_token_head": 512}
        del kps, vps, kp, vp
    except Exception as ex:  # the baseline is context only
        bf16 = {"error": str(ex)}

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = time_oracle(args.config, args.budget, streams=args.streams)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u32 rANS state / f16 mma, f32 accumulate", "data": "synthetic",
        "config": {"workload": cfg.name + ("" if hs == 1 else "_tokenwide"), "batch": B, "q_heads": Hq, "kv_heads": Hkv, "head_dim": 128,
                   "context": cfg.seq_lens if len(set(cfg.seq_lens)) > 1 and B <= 8 else
                   {"min": min(cfg.seq_lens), "max": max(cfg.seq_lens), "sum": kv_tokens},
                   "bits_per_elem": args.budget if hs == 1 else round((k_b + v_b + 1.0) * 8 / 256, 3),
                   "streams": "per token-head (128 values)" if hs == 1 else f"per token ({n_stream} values)",
                   "k_rec_bytes": k_rec, "v_rec_bytes": v_rec,
                   "k_levels": st["k_levels"], "v_levels": st["v_levels"],
                   "step": step_desc, **({} if hs == 1 else {"window_closes_in_timed_region": closes_timed}),
                   "l2": f"{copies} rotating copies of the cache ({copies * cache_bytes / 2**20:.0f} MiB > 126 MiB L2)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "roofline": roofline, "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "launch": graph_note, "output_equals_direct_call": e2e_check},
        "gpu_launches": int(round(launches_per_step * args.steps)), "clocks": clocks,
        "encoder": {"token_heads_per_s": 2 * token_heads / (enc_ms * 1e-3), "prefill_ms": enc_ms,
                    "streams": 2 * token_heads // hs},
        "bf16_baseline": bf16,
    }
    line.update(extra)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[2, 3, 4, 5])
    ap.add_argument("--budget", type=float, default=2.26)
    ap.add_argument("--streams", default="head", choices=["head", "token"],
                    help="head: one stream per (token, KV head), the benchmark's configuration; token: the paper's "
                         "default grouping, one 335 / 235-byte record per token, 8 / 6 levels")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--separate-calls", action="store_true",
                    help="per token-head streams: dq_encode_tokens + dq_decode_attention instead of dq_decode_step")
    ap.add_argument("--no-graph", action="store_true", help="end-to-end leg: launch directly instead of replaying CUDA graphs")
    ap.add_argument("--profile-only", action="store_true",
                    help="warm-up and timed steps only (for profiler captures); prints a short line")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="DRAM bytes per launch of the fused kernel from an ncu capture; default: the captured "
                         "figure of profiles/dq_attention_kernel_config2_ncu.md scaled by the token-heads processed")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

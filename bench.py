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
SM_COUNT, SCHEDULERS_PER_SM = 148, 4
# Stored ncu captures of the fused kernels (summaries under profiles/): DRAM bytes per launch on config 2 and the
# measured warp instructions per decoded symbol step.  They are constants of this file, not
# quantities measured by a bench run; the line says so where it uses them.
NCU_HEAD = {"dram_bytes": 37.62e6, "token_heads": 524288, "bytes_per_token_head": 72.0, "instr_per_symbol": 15.2,
            "issue_active": 0.622, "source": "the ncu summary of dq_attention_kernel on config 2 under profiles/"}
CODECS = {"paper": "the paper's codec: one level per rANS symbol (Algorithm 2, 128 steps per 128-value stream)",
          "pairs": "opt-in variant: one rANS symbol = the levels of two consecutive values (64 steps per stream)"}
NCU_PAIRS = {"instr_per_symbol": 9.96, "issue_active": 0.560,
             "source": "the ncu summary of dq_attention_kernel with paired-symbol tables on config 2 under profiles/"}
NCU_WIDE = {"instr_per_symbol": 19.2, "issue_active": 0.641,
            "source": "the ncu summary of dq_attention_wide_kernel on config 2 under profiles/"}
NCU_WIDE_PAIRS = {"instr_per_symbol": 13.3, "issue_active": 0.626,
                  "source": "the ncu summary of dq_attention_wide_kernel (paired-symbol section) on config 2 under profiles/"}
REGIONS = 21          # the K-step timed region is repeated this many times; ms_per_step is the median
ORACLE_MAX_TOKENS = 131072   # the oracle legs run whole sequences of the workload up to this many tokens


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


def oracle_step_runner(cfg_idx: int, budget: float, streams: str = "head", codec: str = "paper"):
    """Builds the oracle's workload -- the same seeded configuration the GPU leg runs, all of its
    sequences while they stay within ORACLE_MAX_TOKENS tokens in total (configs 2, 3 and 5 whole;
    the first sequences of config 4) -- and returns (step function, KV tokens per step,
    description, threads, whole workload?).  GPU-free."""
    import numpy as np
    import oracle
    from paper_2609_19880_b200 import workloads

    cfg = workloads.make_config(cfg_idx, budget=budget)
    full_batch = cfg.batch
    keep, tot = 0, 0
    for ln in cfg.seq_lens:
        if keep and tot + ln > ORACLE_MAX_TOKENS:
            break
        keep, tot = keep + 1, tot + ln
    cfg.batch, cfg.seq_lens = keep, list(cfg.seq_lens[:keep])
    w = workloads.generate(cfg, device="cpu")
    st = stream_setup(cfg, streams)
    pair = codec == "pairs"
    ok = oracle.build_table(st["k_levels"], 128 * st["hs"], st["k_rec"], st["alpha"], has_mean=True, rotate=True, pair=pair)
    ov = oracle.build_table(st["v_levels"], 128 * st["hs"], st["v_rec"], st["alpha"], has_mean=False, rotate=True, pair=pair)
    kb, vb, qb = workloads.bf16_bits(w.k), workloads.bf16_bits(w.v), workloads.bf16_bits(w.q)
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    mq = np.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), np.int8)
    ms = np.zeros((cfg.batch, w.max_windows, cfg.hkv), np.float32)
    oracle.window_means(kb, seq_id, pos, mq, ms, 0)
    kc = np.zeros((w.num_pages, cfg.hkv // st["hs"], 16, ok.rec), np.uint8)
    vc = np.zeros((w.num_pages, cfg.hkv // st["hs"], 16, ov.rec), np.uint8)
    oracle.encode_tokens(ok, kb, seq_id, pos, slot, kc, mq, ms)
    oracle.encode_tokens(ov, vb, seq_id, pos, slot, vc)
    last = np.cumsum(np.asarray(cfg.seq_lens, dtype=np.int64)) - 1          # the newest token of every sequence
    kl, vl = np.ascontiguousarray(kb[last]), np.ascontiguousarray(vb[last])
    sl_, pl_, tl_ = (np.ascontiguousarray(a[last]) for a in (seq_id, pos, slot))
    pt, sl = w.page_table.numpy(), w.seq_lens.numpy()
    sm = 1.0 / math.sqrt(128.0)

    def step():
        oracle.window_means(kl, sl_, pl_, mq, ms, 1)
        oracle.encode_tokens(ok, kl, sl_, pl_, tl_, kc, mq, ms)
        oracle.encode_tokens(ov, vl, sl_, pl_, tl_, vc)
        return oracle.attention(ok, ov, qb, kc, vc, mq, ms, pt, sl, cfg.hkv, sm)

    whole = keep == full_batch
    desc = ((f"the whole workload {cfg.name}" if whole else f"the first {keep} of {full_batch} sequences of {cfg.name}") +
            f": {tot} tokens x {cfg.hkv} KV heads x {cfg.hq} query heads, encode 1 token per sequence + fp64 attention per step")
    return step, tot, desc, oracle.num_threads(), whole


def time_oracle(cfg_idx, budget, budget_s=10.0, max_steps=1000, warmup=1, streams="head", codec="paper"):
    step, toks, desc, cores, _ = oracle_step_runner(cfg_idx, budget, streams, codec)
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
    step, toks, desc, cores, whole = oracle_step_runner(args.config, args.budget, args.streams, args.codec)
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
            "config": {"workload": f"config {args.config} at {args.budget} bits/elem, " +
                       ("" if whole else "bounded sample: ") + desc, "codec": CODECS[args.codec]},
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
    pair = args.codec == "pairs"
    tk = dq.dq_build_tables(st["k_levels"], k_rec * 8 / n_stream, alpha=st["alpha"], has_mean=True, rotate=True,
                            heads_per_stream=hs, pair_symbols=pair)
    tv = dq.dq_build_tables(st["v_levels"], v_rec * 8 / n_stream, alpha=st["alpha"], has_mean=False, rotate=True,
                            heads_per_stream=hs, pair_symbols=pair)
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

    # ---- timed region: exactly K steps between a barrier + synchronize on both sides, CUDA events on the
    # launch stream, nothing else enabled.  The region is repeated REGIONS times back to back (the rotating
    # cache copies keep every step out of L2); ms_per_step is the median region, min / max beside it.
    t_wall0 = time.time()
    closes0 = state["closes"]
    region_ms = []
    n_regions = 1 if args.profile_only else REGIONS
    for r in range(n_regions):
        barrier()
        e0.record()
        for i in range(args.steps):
            step(r * args.steps + i)
        e1.record()
        barrier()
        region_ms.append(max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps)
    closes_timed = state["closes"] - closes0
    t_wall1 = time.time()
    ms_per_step = statistics.median(region_ms)
    value = job_throughput(kv_tokens, ms_per_step * 1e-3, world)

    # ---- separate pass: CUDA events around the fused kernel of every step (they serialise the step's
    # kernels, which is why this is not done inside the timed region)
    dq.dq_profile_enable(1)
    for i in range(max(16, min(args.steps, 64))):
        step(i)
    torch.cuda.synchronize()
    kern_ms = dq.dq_profile_read(4096)
    dq.dq_profile_enable(False)

    if args.profile_only:   # short run for an ncu capture: no soak, no e2e, no baselines
        sampler.stop()
        if rank == 0:
            print(json.dumps({"profile_only": True, "ms_per_step": ms_per_step,
                              "kernel_ms": statistics.median(kern_ms) if kern_ms else None}), flush=True)
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
    e2e_regions = []
    for r in range(5):                      # median of 5 regions of K steps, wall clock around each
        barrier()
        t0 = time.perf_counter()
        for i in range(args.steps):
            e2e_step(r * args.steps + i)
        barrier()
        e2e_regions.append(max_over_ranks(time.perf_counter() - t0, world, dev))
    e2e_s = statistics.median(e2e_regions)
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

    # ---- roofline of the dominant kernel (fused decode attention): the metric's own quantity, compressed
    # cache bytes per second against the measured copy bandwidth; beside it the issue-slot figures that
    # say why the fraction is what it is (the kernel is bound by instruction issue, not by HBM)
    k_ms = statistics.median(kern_ms) if kern_ms else None
    symbols = token_heads * 256.0
    comp_bytes = token_heads * (k_b + v_b + 1.0)   # records + amortised INT8 mean byte
    roofline = None
    extra = {}
    ncu = (NCU_PAIRS if pair else NCU_HEAD) if hs == 1 else (NCU_WIDE_PAIRS if pair else NCU_WIDE)
    if args.traffic_bytes is None:
        # every record is read once, so the captured config-2 figure scales with the records' bytes
        args.traffic_bytes = NCU_HEAD["dram_bytes"] * comp_bytes / (NCU_HEAD["token_heads"] * NCU_HEAD["bytes_per_token_head"])
        traffic_src = (f"scaled from the stored ncu capture {NCU_HEAD['source']} (dram__bytes_read + write of one launch "
                       "on config 2); not measured in this run")
    else:
        traffic_src = "given on the command line (--traffic-bytes)"
    if k_ms:
        gbs = comp_bytes / (k_ms * 1e-3) / 1e9
        mhz = sm_max_mhz
        roofline = {"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gbs / hbm_peak,
                    "frac_of_8TBps": gbs / 8000.0, "peak_source": f"MEASURED_PEAKS.json hbm_gbs ({peak_kind})",
                    "traffic": args.traffic_bytes, "traffic_source": traffic_src,
                    "algorithmic_bytes_per_launch": comp_bytes, "bytes_per_token_head": k_b + v_b + 1,
                    "kernel": "dq_attention_kernel" if hs == 1 else "dq_attention_wide_kernel",
                    "kernel_ms": k_ms, "kernel_ms_min": min(kern_ms), "kernel_ms_max": max(kern_ms),
                    "launches_timed": len(kern_ms),
                    "timed": "CUDA events around the kernel on its launch stream, in a pass of its own after the timed region"}
        warp_instr = symbols / 32.0 * ncu["instr_per_symbol"]
        issue_peak = SM_COUNT * SCHEDULERS_PER_SM * mhz * 1e6     # warp instructions per second at max clock
        extra = {"issue_slots": {"bound": "alu", "unit": "warp instructions/s",
                                 "achieved": warp_instr / (k_ms * 1e-3), "peak": issue_peak,
                                 "frac": warp_instr / (k_ms * 1e-3) / issue_peak,
                                 "peak_source": f"148 SMs x 4 schedulers x {mhz:.0f} MHz, one warp instruction per clock each",
                                 "instr_per_symbol": ncu["instr_per_symbol"], "ncu_issue_active": ncu["issue_active"],
                                 "instr_source": f"stored ncu capture {ncu['source']}; not measured in this run"},
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

    # ---- the paired-symbol codec variant on the same workload (context beside the paper codec's line;
    # `--codec pairs` makes it the line itself): same records' sizes, 64 decode steps per stream instead of 128
    variants = None
    if hs == 1 and world == 1 and not pair and not args.no_variants and max(st["k_levels"], st["v_levels"]) <= 9:
        try:
            tkp = dq.dq_build_tables(st["k_levels"], k_rec * 8 / 128, alpha=st["alpha"], has_mean=True, rotate=True, pair_symbols=True)
            tvp = dq.dq_build_tables(st["v_levels"], v_rec * 8 / 128, alpha=st["alpha"], has_mean=False, rotate=True, pair_symbols=True)
            pc = [new_cache()]
            for rep_i in range(2):
                e0.record()
                dq.dq_encode_tokens(tkp, tvp, w.k, w.v, w.seq_id, w.pos, w.slot, pc[0]["k"], pc[0]["v"], pc[0]["mq"], pc[0]["ms"])
                e1.record()
                torch.cuda.synchronize()
            p_enc_ms = e0.elapsed_time(e1)
            for _ in range(copies - 1):
                pc.append({k: v.clone() for k, v in pc[0].items()})

            def pstep(i):
                c = pc[i % copies]
                dq.dq_decode_step(tkp, tvp, new_k, new_v, new_slot, w.q, c["k"], c["v"], c["mq"], c["ms"], w.page_table,
                                  w.seq_lens, Hkv, sm_scale, out, ws)
            for i in range(5):
                pstep(i)
            p_regions = []
            for r in range(7):
                torch.cuda.synchronize()
                e0.record()
                for i in range(args.steps):
                    pstep(r * args.steps + i)
                e1.record()
                torch.cuda.synchronize()
                p_regions.append(e0.elapsed_time(e1) / args.steps)
            dq.dq_profile_enable(1)
            for i in range(max(16, min(args.steps, 64))):
                pstep(i)
            torch.cuda.synchronize()
            p_kern = dq.dq_profile_read(4096)
            dq.dq_profile_enable(False)
            p_ms, p_k = statistics.median(p_regions), statistics.median(p_kern)
            variants = {"paired_symbols": {
                "ms_per_step": p_ms, "value": kv_tokens / (p_ms * 1e-3), "unit": UNIT, "kernel_ms": p_k,
                "compressed_gb_per_s": comp_bytes / (p_k * 1e-3) / 1e9, "frac_of_measured_hbm": comp_bytes / (p_k * 1e-3) / 1e9 / hbm_peak,
                "prefill_ms": p_enc_ms, "regions": len(p_regions),
                "note": "opt-in table option pair_symbols: one rANS symbol = the levels of two consecutive values; same record "
                        "sizes and level counts; parity against the oracle's same variant in tests/test_gpu_variants.py"}}
            del pc
        except Exception as ex:   # context only
            variants = {"paired_symbols": {"error": f"{type(ex).__name__}: {ex}"}}

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = time_oracle(args.config, args.budget, streams=args.streams, codec=args.codec)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step,
        "timing": {"regions": len(region_ms), "steps_per_region": args.steps, "ms_per_step_median": ms_per_step,
                   "ms_per_step_min": min(region_ms), "ms_per_step_max": max(region_ms),
                   "ms_per_step_x_sm_mhz": (ms_per_step * clocks["sm_mhz"]) if clocks.get("sm_mhz") else None},
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u32 rANS state / f16 mma, f32 accumulate", "data": "synthetic",
        "config": {"workload": cfg.name + ("" if hs == 1 else "_tokenwide"), "batch": B, "q_heads": Hq, "kv_heads": Hkv, "head_dim": 128,
                   "context": cfg.seq_lens if len(set(cfg.seq_lens)) > 1 and B <= 8 else
                   {"min": min(cfg.seq_lens), "max": max(cfg.seq_lens), "sum": kv_tokens},
                   "bits_per_elem": args.budget if hs == 1 else round((k_b + v_b + 1.0) * 8 / 256, 3),
                   "streams": "per token-head (128 values)" if hs == 1 else f"per token ({n_stream} values)",
                   "codec": CODECS[args.codec],
                   "k_rec_bytes": k_rec, "v_rec_bytes": v_rec,
                   "k_levels": st["k_levels"], "v_levels": st["v_levels"],
                   "step": step_desc, **({} if hs == 1 else {"window_closes_in_timed_region": closes_timed}),
                   "l2": f"{copies} rotating copies of the cache ({copies * cache_bytes / 2**20:.0f} MiB > 126 MiB L2)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "roofline": roofline, "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "launch": graph_note, "output_equals_direct_call": e2e_check},
        "gpu_launches": int(round(launches_per_step * args.steps)), "gpu_launches_note": "per timed region of K steps",
        "clocks": clocks,
        "encoder": {"token_heads_per_s": 2 * token_heads / (enc_ms * 1e-3), "prefill_ms": enc_ms,
                    "streams": 2 * token_heads // hs},
        "bf16_baseline": bf16,
        "codec_variants": variants,
    }
    line.update(extra)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_decode_loop(args):
    """`--decode-loop`: the bare rANS symbol step of the fused kernel (dq_microbench_decode_loop) on 148 CTAs,
    timed with CUDA events; one JSON line per (threads, chains) with clocks per symbol per SM sub-partition."""
    import torch
    import paper_2609_19880_b200 as dq
    from paper_2609_19880_b200 import _build
    if not os.path.exists(dq.LIB_PATH):
        _build.build()
    dev = torch.device("cuda", 0)
    tk = dq.dq_build_tables(5, 42 * 8 / 128, alpha=1.4, has_mean=True, rotate=True)
    g = torch.Generator(device="cpu").manual_seed(1)
    data = torch.randint(0, 256, (1 << 20,), dtype=torch.uint8, generator=g).to(dev)
    out = torch.zeros(SM_COUNT * 1024, dtype=torch.int32, device=dev)
    sampler = ClockSampler(0, period_s=0.005)
    sampler.start()
    reps = 400
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rows = []
    for threads in (512, 1024):
        for chains in (1, 2):
            dq.dq_microbench_decode_loop(tk, data, SM_COUNT, threads, chains, 8, out)
            torch.cuda.synchronize()
            best, t0 = None, time.time()
            for _ in range(5):
                e0.record()
                dq.dq_microbench_decode_loop(tk, data, SM_COUNT, threads, chains, reps, out)
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1)
                best = ms if best is None else min(best, ms)
            mhz = sampler.summary(t0, time.time()).get("sm_mhz") or _peaks()[1]
            symbols = SM_COUNT * threads * chains * 128.0 * reps
            steps_per_smsp = symbols / 32.0 / (SM_COUNT * SCHEDULERS_PER_SM)
            rows.append({"decode_loop": True, "threads_per_cta": threads, "chains_per_lane": chains, "ms": best,
                         "symbols_per_s": symbols / (best * 1e-3), "sm_mhz": mhz,
                         "clk_per_symbol_per_smsp": best * 1e-3 * mhz * 1e6 / steps_per_smsp})
    sampler.stop()
    for r in rows:
        print(json.dumps(r), flush=True)


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
    ap.add_argument("--codec", default="paper", choices=sorted(CODECS),
                    help="paper: one level per rANS symbol (Algorithm 2); pairs: the opt-in paired-symbol variant")
    ap.add_argument("--no-variants", action="store_true", help="skip the codec-variant context measurement")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--separate-calls", action="store_true",
                    help="per token-head streams: dq_encode_tokens + dq_decode_attention instead of dq_decode_step")
    ap.add_argument("--no-graph", action="store_true", help="end-to-end leg: launch directly instead of replaying CUDA graphs")
    ap.add_argument("--profile-only", action="store_true",
                    help="warm-up and timed steps only (for profiler captures); prints a short line")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="DRAM bytes per launch of the fused kernel from an ncu capture; default: the captured "
                         "figure of the config-2 capture summarised under profiles/, scaled by the token-heads processed")
    ap.add_argument("--decode-loop", action="store_true",
                    help="micro-benchmark of the bare rANS decode loop (no tiles, no contractions) instead of the step")
    args = ap.parse_args()
    if args.decode_loop:
        run_decode_loop(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

"""Helpers of the GPU parity tests: run the CUDA path through the C ABI and the oracle on the
same seeded inputs."""
from __future__ import annotations

import math

import numpy as np
import torch

import oracle
import paper_2609_19880_b200 as dq
from paper_2609_19880_b200 import workloads

SM_SCALE = 1.0 / math.sqrt(128.0)


def tables(cfg, rotate_v=True, early_exit=False, sigma=32, pair=False):
    """(library K, library V, oracle K, oracle V) tables of a configuration; early_exit / sigma / pair
    select the opt-in codec variants on both sides."""
    tk = dq.dq_build_tables(cfg.k_levels, cfg.bits_k, alpha=cfg.alpha, has_mean=True, rotate=True,
                            drift_early_exit=early_exit, sigma_bits=sigma, pair_symbols=pair)
    tv = dq.dq_build_tables(cfg.v_levels, cfg.bits_v, alpha=cfg.alpha, has_mean=False, rotate=rotate_v,
                            drift_early_exit=early_exit, sigma_bits=sigma, pair_symbols=pair)
    ok = oracle.build_table(cfg.k_levels, 128, cfg.k_rec, cfg.alpha, has_mean=True, rotate=True,
                            early_exit=early_exit, sigma=sigma, pair=pair)
    ov = oracle.build_table(cfg.v_levels, 128, cfg.v_rec, cfg.alpha, has_mean=False, rotate=rotate_v,
                            early_exit=early_exit, sigma=sigma, pair=pair)
    return tk, tv, ok, ov


class GpuCache:
    """Device-side cache arrays of one workload."""

    def __init__(self, w, k_rec, v_rec, dev="cuda"):
        cfg = w.cfg
        self.k_cont = torch.zeros((w.num_pages, cfg.hkv, 16, k_rec), dtype=torch.uint8, device=dev)
        self.v_cont = torch.zeros((w.num_pages, cfg.hkv, 16, v_rec), dtype=torch.uint8, device=dev)
        self.mean_q = torch.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), dtype=torch.int8, device=dev)
        self.mean_scale = torch.zeros((cfg.batch, w.max_windows, cfg.hkv), dtype=torch.float32, device=dev)
        self.status = torch.zeros(4, dtype=torch.uint32, device=dev)


def gpu_encode(w, tk, tv, cache, mode=dq.MEAN_COMPUTE, sel=None):
    k, v, seq_id, pos, slot = w.k, w.v, w.seq_id, w.pos, w.slot
    if sel is not None:
        k, v, seq_id, pos, slot = (x[sel].contiguous() for x in (k, v, seq_id, pos, slot))
    dq.dq_encode_tokens(tk, tv, k, v, seq_id, pos, slot, cache.k_cont, cache.v_cont, cache.mean_q,
                        cache.mean_scale, mode, cache.status)


def gpu_attention(w, tk, tv, cache, seq_lens=None, want_f32=True):
    cfg = w.cfg
    out = torch.empty((cfg.batch, cfg.hq, 128), dtype=torch.bfloat16, device="cuda")
    out32 = torch.empty((cfg.batch, cfg.hq, 128), dtype=torch.float32, device="cuda") if want_f32 else None
    nbytes = dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, w.page_table.shape[1])
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    sl = w.seq_lens if seq_lens is None else seq_lens
    dq.dq_decode_attention(tk, tv, w.q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale,
                           w.page_table, sl, cfg.hkv, SM_SCALE, out, ws, out32)
    torch.cuda.synchronize()
    return out, out32


def oracle_encode(w, ok, ov, sel=None):
    """Oracle containers / means for the whole workload or for the tokens in ``sel`` (numpy
    index array; must hold whole windows when means are computed)."""
    cfg = w.cfg
    idx = slice(None) if sel is None else sel
    kb = workloads.bf16_bits(w.k[idx])
    vb = workloads.bf16_bits(w.v[idx])
    seq_id, pos, slot = (t[idx].cpu().numpy() for t in (w.seq_id, w.pos, w.slot))
    mq = np.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), np.int8)
    ms = np.zeros((cfg.batch, w.max_windows, cfg.hkv), np.float32)
    oracle.window_means(kb, seq_id, pos, mq, ms, 0)
    kc = np.zeros((w.num_pages, cfg.hkv, 16, ok.rec), np.uint8)
    vc = np.zeros((w.num_pages, cfg.hkv, 16, ov.rec), np.uint8)
    sk = oracle.encode_tokens(ok, kb, seq_id, pos, slot, kc, mq, ms)
    sv = oracle.encode_tokens(ov, vb, seq_id, pos, slot, vc)
    return kc, vc, mq, ms, sk, sv


def check_attention(out_bf16, out_f32, ref, rows=None):
    """Tolerance of the attention output against the oracle's fp64 result.

    Per (b, h) vector: max |out - ref| <= 2e-3 * max |ref| for the kernel's fp32 result; the
    bf16 output must be exactly the RNE rounding of that fp32 result, so it carries at most
    half a bf16 ulp (2^-9 .. 2^-8 relative) on top."""
    o32 = out_f32.double().cpu().numpy()
    o16 = out_bf16.double().cpu().numpy()
    assert torch.equal(out_f32.to(torch.bfloat16), out_bf16)
    worst = 0.0
    it = rows if rows is not None else [(b, h) for b in range(ref.shape[0]) for h in range(ref.shape[1])]
    for (b, h) in it:
        r = ref[b, h]
        assert np.isfinite(r).all()
        scale = np.abs(r).max()
        if scale == 0.0:
            assert not o32[b, h].any() and not o16[b, h].any()
            continue
        e32 = np.abs(o32[b, h] - r).max() / scale
        worst = max(worst, e32)
        assert e32 <= 2e-3, (b, h, e32)
        assert np.all(np.abs(o16[b, h] - r) <= 2e-3 * scale + 2.0 ** -8 * np.abs(r)), (b, h)
    return worst


# ---- token-wide streams (heads_per_stream = hs > 1): the library stores records word-interleaved
# per page, uint8 [pages][groups][rec_words][16][4]; the oracle keeps [pages][groups][16][rec].

def wide_tables(cfg, hs, k_rec=335, v_rec=235, k_levels=8, v_levels=6, alpha=1.4, early_exit=False, pair=False):
    n = 128 * hs
    tk = dq.dq_build_tables(k_levels, k_rec * 8 / n, alpha=alpha, has_mean=True, rotate=True, heads_per_stream=hs,
                            drift_early_exit=early_exit, pair_symbols=pair)
    tv = dq.dq_build_tables(v_levels, v_rec * 8 / n, alpha=alpha, has_mean=False, rotate=True, heads_per_stream=hs,
                            drift_early_exit=early_exit, pair_symbols=pair)
    ok = oracle.build_table(k_levels, n, k_rec, alpha, has_mean=True, rotate=True, early_exit=early_exit, pair=pair)
    ov = oracle.build_table(v_levels, n, v_rec, alpha, has_mean=False, rotate=True, early_exit=early_exit, pair=pair)
    assert tk.info().rec_bytes == k_rec and tv.info().rec_bytes == v_rec
    return tk, tv, ok, ov


def to_interleaved(cont: np.ndarray) -> np.ndarray:
    """[pages][groups][16][rec] -> [pages][groups][rec_words][16][4] (zero padded)."""
    P, Gr, _, rec = cont.shape
    rw = (rec + 3) // 4
    pad = np.zeros((P, Gr, 16, rw * 4), np.uint8)
    pad[..., :rec] = cont
    return np.ascontiguousarray(pad.reshape(P, Gr, 16, rw, 4).transpose(0, 1, 3, 2, 4))


def from_interleaved(cw: np.ndarray, rec: int) -> np.ndarray:
    P, Gr, rw, _, _ = cw.shape
    flat = cw.transpose(0, 1, 3, 2, 4).reshape(P, Gr, 16, rw * 4)
    assert not flat[..., rec:].any()          # alignment bytes stay zero
    return np.ascontiguousarray(flat[..., :rec])


class WideGpuCache:
    def __init__(self, w, tk, tv, hs, dev="cuda"):
        cfg = w.cfg
        gr = cfg.hkv // hs
        self.k_cont = torch.zeros((w.num_pages, gr, tk.info().rec_words, 16, 4), dtype=torch.uint8, device=dev)
        self.v_cont = torch.zeros((w.num_pages, gr, tv.info().rec_words, 16, 4), dtype=torch.uint8, device=dev)
        self.mean_q = torch.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), dtype=torch.int8, device=dev)
        self.mean_scale = torch.zeros((cfg.batch, w.max_windows, cfg.hkv), dtype=torch.float32, device=dev)
        self.status = torch.zeros(4, dtype=torch.uint32, device=dev)


def oracle_encode_wide(w, ok, ov, hs, sel=None):
    cfg = w.cfg
    idx = slice(None) if sel is None else sel
    kb = workloads.bf16_bits(w.k[idx])
    vb = workloads.bf16_bits(w.v[idx])
    seq_id, pos, slot = (t[idx].cpu().numpy() for t in (w.seq_id, w.pos, w.slot))
    mq = np.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), np.int8)
    ms = np.zeros((cfg.batch, w.max_windows, cfg.hkv), np.float32)
    oracle.window_means(kb, seq_id, pos, mq, ms, 0)
    kc = np.zeros((w.num_pages, cfg.hkv // hs, 16, ok.rec), np.uint8)
    vc = np.zeros((w.num_pages, cfg.hkv // hs, 16, ov.rec), np.uint8)
    sk = oracle.encode_tokens(ok, kb, seq_id, pos, slot, kc, mq, ms)
    sv = oracle.encode_tokens(ov, vb, seq_id, pos, slot, vc)
    return kc, vc, mq, ms, sk, sv

"""GPU parity of decode attention with a BF16 residual window (Sec. 5.1: the most recent 128
tokens stay uncompressed): dq_decode_attention_residual against the oracle's fp64 attention
over compressed + raw tokens, and the sliding policy that encodes a window when it fills."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_19880_b200 as dq
from paper_2609_19880_b200 import _build, workloads

import gpu_common as gc

pytestmark = pytest.mark.gpu
CAP = 128


@pytest.fixture(scope="module", autouse=True)
def _lib():
    _build.build()
    assert torch.cuda.is_available()
    dq.lib()


def _np(t):
    return t.cpu().numpy()


def _cfg(idx, **over):
    cfg = workloads.make_config(idx, scale=1 / 16)
    for k, v in over.items():
        setattr(cfg, k, v)
    return cfg


def _attend(w, tk, tv, cache, seq_lens, rk, rv, rl):
    cfg = w.cfg
    out = torch.empty((cfg.batch, cfg.hq, 128), dtype=torch.bfloat16, device="cuda")
    out32 = torch.empty((cfg.batch, cfg.hq, 128), dtype=torch.float32, device="cuda")
    ws = torch.empty(dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, w.page_table.shape[1]), dtype=torch.uint8,
                     device="cuda")
    dq.dq_decode_attention_residual(tk, tv, w.q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale,
                                    w.page_table, seq_lens, rk, rv, rl, cfg.hkv, gc.SM_SCALE, out, ws, out32)
    torch.cuda.synchronize()
    return out, out32


def _reference(w, ok, ov, cache, seq_lens, rk, rv, rl):
    return oracle.attention(ok, ov, workloads.bf16_bits(w.q), _np(cache.k_cont), _np(cache.v_cont),
                            _np(cache.mean_q), _np(cache.mean_scale), _np(w.page_table), _np(seq_lens), w.cfg.hkv,
                            gc.SM_SCALE, resid_k=workloads.bf16_bits(rk), resid_v=workloads.bf16_bits(rv),
                            resid_lens=_np(rl))


@pytest.mark.parametrize("idx,lens,rlens", [
    (2, [512, 300, 77, 0, 0, 1000, 16, 129], [0, 1, 7, 8, 9, 64, 127, 128]),
    (3, [1999], [100]),
    (5, [640, 129, 0], [128, 33, 5]),
])
def test_residual_attention_matches_oracle(idx, lens, rlens):
    cfg = _cfg(idx, batch=len(lens), seq_lens=lens)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    gen = torch.Generator(device="cuda").manual_seed(7 + idx)
    rk, rv = workloads.make_kv(cfg, cfg.batch * CAP, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
    rk = rk.view(cfg.batch, CAP, cfg.hkv, 128).contiguous()
    rv = rv.view(cfg.batch, CAP, cfg.hkv, 128).contiguous()
    rl = torch.tensor(rlens, dtype=torch.int32, device="cuda")
    out, out32 = _attend(w, tk, tv, cache, w.seq_lens, rk, rv, rl)
    ref = _reference(w, ok, ov, cache, w.seq_lens, rk, rv, rl)
    worst = gc.check_attention(out, out32, ref)
    assert worst < 2e-4
    # an empty residual window is the plain call, bit for bit
    zero = torch.zeros_like(rl)
    out_z, out32_z = _attend(w, tk, tv, cache, w.seq_lens, rk, rv, zero)
    out_p, out32_p = gc.gpu_attention(w, tk, tv, cache)
    assert torch.equal(out32_z, out32_p) and torch.equal(out_z, out_p)
    # a sequence with nothing at all yields zeros
    for b, (a, r) in enumerate(zip(lens, rlens)):
        if a == 0 and r == 0:
            assert not out32[b].any()


def test_residual_only_equals_plain_bf16_attention():
    """No compressed tokens: softmax(q k^T / sqrt(d)) v over the raw window, by library matmuls."""
    cfg = _cfg(2, batch=4, seq_lens=[16, 16, 16, 16])
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gen = torch.Generator(device="cuda").manual_seed(3)
    rk, rv = workloads.make_kv(cfg, cfg.batch * CAP, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
    rk = rk.view(cfg.batch, CAP, cfg.hkv, 128).contiguous()
    rv = rv.view(cfg.batch, CAP, cfg.hkv, 128).contiguous()
    rlens = [128, 77, 1, 40]
    rl = torch.tensor(rlens, dtype=torch.int32, device="cuda")
    none = torch.zeros(cfg.batch, dtype=torch.int32, device="cuda")
    out, out32 = _attend(w, tk, tv, cache, none, rk, rv, rl)
    G = cfg.hq // cfg.hkv
    ref = np.zeros((cfg.batch, cfg.hq, 128))
    for b in range(cfg.batch):
        kk = rk[b, :rlens[b]].double().cpu()            # [t, Hkv, d]
        vv = rv[b, :rlens[b]].double().cpu()
        qq = w.q[b].double().cpu()                       # [Hq, d]
        for hq in range(cfg.hq):
            a = torch.softmax((kk[:, hq // G] @ qq[hq]) * gc.SM_SCALE, 0)
            ref[b, hq] = (a @ vv[:, hq // G]).numpy()
    gc.check_attention(out, out32, ref)


def test_sliding_window_policy_loop():
    """Decode loop with the residual policy: each step appends the new token's K/V to the BF16
    window and attends; a full window is encoded in one call with its own channel mean
    (DQ_MEAN_COMPUTE) and the window restarts.  Containers and means bit-exact against the
    oracle's mirror of the loop, attention checked at steps around every window close."""
    cfg = _cfg(5, batch=3, seq_lens=[256, 128, 384])
    steps = 300
    w = workloads.generate(cfg, device="cuda", extra_tokens_per_seq=steps + CAP)
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    kc, vc, mq, ms, _, _ = gc.oracle_encode(w, ok, ov)
    dev = torch.device("cuda")
    gen = torch.Generator(device="cuda").manual_seed(123)
    rk = torch.zeros((cfg.batch, CAP, cfg.hkv, 128), dtype=torch.bfloat16, device=dev)
    rv = torch.zeros_like(rk)
    # sequences start with differently filled windows so that closes fall on different steps
    fill = [0, 100, 127]
    k0, v0 = workloads.make_kv(cfg, cfg.batch * CAP, gen, dev, w.k_offsets, w.k_gain)
    rk.copy_(k0.view_as(rk)); rv.copy_(v0.view_as(rv))
    rl = torch.tensor(fill, dtype=torch.int32)
    lens = torch.tensor(cfg.seq_lens, dtype=torch.int32)
    pt_cpu = w.page_table.cpu()
    closes = 0
    for s in range(steps):
        k1, v1 = workloads.make_kv(cfg, cfg.batch, gen, dev, w.k_offsets, w.k_gain)
        for b in range(cfg.batch):
            rk[b, int(rl[b])] = k1[b]
            rv[b, int(rl[b])] = v1[b]
        rl += 1
        near_close = bool((rl >= CAP - 1).any() or (rl <= 1).any())
        if near_close or s % 37 == 0:
            out, out32 = _attend(w, tk, tv, cache, lens.cuda(), rk, rv, rl.cuda())
            ref = _reference(w, ok, ov, cache, lens.cuda(), rk, rv, rl.cuda())
            gc.check_attention(out, out32, ref)
        for b in range(cfg.batch):
            if int(rl[b]) < CAP:
                continue
            closes += 1
            pos = (int(lens[b]) + torch.arange(CAP)).to(torch.int32)
            seq = torch.full((CAP,), b, dtype=torch.int32)
            slot = (pt_cpu[b, (pos // 16).long()] * 16 + pos % 16).to(torch.int32)
            kw, vw = rk[b].contiguous(), rv[b].contiguous()
            dq.dq_encode_tokens(tk, tv, kw, vw, seq.cuda(), pos.cuda(), slot.cuda(), cache.k_cont, cache.v_cont,
                                cache.mean_q, cache.mean_scale, dq.MEAN_COMPUTE, cache.status)
            kb, vb = workloads.bf16_bits(kw), workloads.bf16_bits(vw)
            oracle.window_means(kb, seq.numpy(), pos.numpy(), mq, ms, 0)
            oracle.encode_tokens(ok, kb, seq.numpy(), pos.numpy(), slot.numpy(), kc, mq, ms)
            oracle.encode_tokens(ov, vb, seq.numpy(), pos.numpy(), slot.numpy(), vc)
            lens[b] += CAP
            rl[b] = 0
    torch.cuda.synchronize()
    assert closes >= 6 and int(_np(cache.status)[0]) == 0
    assert np.array_equal(_np(cache.mean_q), mq) and np.array_equal(_np(cache.mean_scale), ms)
    assert np.array_equal(_np(cache.k_cont), kc) and np.array_equal(_np(cache.v_cont), vc)
    out, out32 = _attend(w, tk, tv, cache, lens.cuda(), rk, rv, rl.cuda())
    ref = _reference(w, ok, ov, cache, lens.cuda(), rk, rv, rl.cuda())
    gc.check_attention(out, out32, ref)


def test_window_append_matches_indexing():
    """dq_window_append writes the new token at position resid_lens[b], counts it, and leaves full windows alone."""
    B, Hkv, cap = 5, 8, 8
    g = torch.Generator(device="cuda").manual_seed(1)
    rk = torch.randn((B, cap, Hkv, 128), generator=g, device="cuda").to(torch.bfloat16)
    rv = torch.randn((B, cap, Hkv, 128), generator=g, device="cuda").to(torch.bfloat16)
    rl = torch.tensor([0, 3, 7, 8, 5], dtype=torch.int32, device="cuda")
    want_k, want_v, want_l = rk.clone(), rv.clone(), rl.clone()
    for step in range(3):
        nk = torch.randn((B, Hkv, 128), generator=g, device="cuda").to(torch.bfloat16)
        nv = torch.randn((B, Hkv, 128), generator=g, device="cuda").to(torch.bfloat16)
        dq.dq_window_append(nk, nv, rk, rv, rl)
        for b in range(B):
            r = int(want_l[b])
            if r < cap:
                want_k[b, r], want_v[b, r] = nk[b], nv[b]
                want_l[b] = r + 1
        torch.cuda.synchronize()
        assert torch.equal(rk, want_k) and torch.equal(rv, want_v) and torch.equal(rl, want_l)

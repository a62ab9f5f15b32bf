"""GPU parity of the opt-in codec variants against the oracle's same variants (the oracle's
variants are pinned in test_oracle_variants.py):

* early exit of Drift: records bit for bit against the oracle built with the same option -- and,
  as it happens on every stream tried, identical to the default codec's records -- through the
  one-warp-per-stream encoder, the batch encoders and the token-wide encoders; the prefill of
  configuration 2 at full size, every record;
* sigma = 24: records, decoded symbols, dequantised values bit for bit, attention within tolerance,
  for the default 5 / 3 levels and for 6 value levels in 29 bytes (a table that only the shorter
  state makes feasible); the decode step in one call; mixed state widths are refused;
* paired symbols: records, decoded symbols, dequantised values bit for bit and attention within
  tolerance for 5 / 3, 8 / 6 and 9 / 9 levels, alone and together with the other two variants, through
  both encoder kernels, the check decoder, every attention entry point and the decode step; the
  whole of configuration 2 at full size; mixed alphabets are refused.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_19880_b200 as dq
from paper_2609_19880_b200 import _build, workloads

import gpu_common as gc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    _build.build()
    dq.lib()


def _np(t):
    return t.cpu().numpy()


def _encode_and_compare(cfg, early_exit=False, sigma=32, batch_kernels=False, pair=False):
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg, early_exit=early_exit, sigma=sigma, pair=pair)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    if batch_kernels:
        dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, 0)
    try:
        gc.gpu_encode(w, tk, tv, cache)
        torch.cuda.synchronize()
    finally:
        dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, -1)
    kc, vc, mq, ms, sk, sv = gc.oracle_encode(w, ok, ov)
    assert np.array_equal(_np(cache.k_cont), kc) and np.array_equal(_np(cache.v_cont), vc)
    assert np.array_equal(_np(cache.mean_q), mq) and np.array_equal(_np(cache.mean_scale).view(np.uint32), ms.view(np.uint32))
    st = _np(cache.status)
    assert st[0] == sk[0] + sv[0] and st[3] == max(sk[3], sv[3])
    return w, tk, tv, ok, ov, cache, (kc, vc, mq, ms)


@pytest.mark.parametrize("batch_kernels", [False, True])
@pytest.mark.parametrize("cfg_idx,scale", [(1, 1.0), (2, 1 / 16), (5, 1 / 32)])
def test_early_exit_records_match_oracle_and_default(cfg_idx, scale, batch_kernels):
    cfg = workloads.make_config(cfg_idx, scale=scale) if cfg_idx > 1 else workloads.make_config(1)
    w, tk, tv, ok, ov, cache, host = _encode_and_compare(cfg, early_exit=True, batch_kernels=batch_kernels)
    # the default codec on the same inputs: the same bytes
    tk0, tv0, ok0, ov0 = gc.tables(cfg)
    c0 = gc.GpuCache(w, ok0.rec, ov0.rec)
    gc.gpu_encode(w, tk0, tv0, c0)
    torch.cuda.synchronize()
    assert torch.equal(c0.k_cont, cache.k_cont) and torch.equal(c0.v_cont, cache.v_cont)
    # and attention over those records through the ordinary decoder
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), host[0], host[1], host[2], host[3], _np(w.page_table),
                           _np(w.seq_lens), cfg.hkv, gc.SM_SCALE)
    gc.check_attention(out, out32, ref)


def test_early_exit_token_wide_records_match_oracle():
    cfg = workloads.make_config(2, scale=1 / 16)
    for batch in (False, True):
        w = workloads.generate(cfg, device="cuda")
        tk, tv, ok, ov = gc.wide_tables(cfg, 8, early_exit=True)
        cache = gc.WideGpuCache(w, tk, tv, 8)
        if batch:
            dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, 0)
        try:
            gc.gpu_encode(w, tk, tv, cache)
            torch.cuda.synchronize()
        finally:
            dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, -1)
        kc, vc, mq, ms, sk, sv = gc.oracle_encode_wide(w, ok, ov, 8)
        assert np.array_equal(gc.from_interleaved(_np(cache.k_cont), ok.rec), kc)
        assert np.array_equal(gc.from_interleaved(_np(cache.v_cont), ov.rec), vc)


@pytest.mark.parametrize("early_exit", [False, True])
def test_pair_symbols_token_wide_both_encoders(early_exit):
    """Token-wide streams (8 heads, 8 / 6 levels) with paired symbols: the one-stream-per-CTA encoder and the
    batch encoder write the oracle's records; attention over them within tolerance."""
    cfg = workloads.make_config(2, scale=1 / 16)
    for batch in (False, True):
        w = workloads.generate(cfg, device="cuda")
        tk, tv, ok, ov = gc.wide_tables(cfg, 8, early_exit=early_exit, pair=True)
        cache = gc.WideGpuCache(w, tk, tv, 8)
        if batch:
            dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, 0)
        try:
            gc.gpu_encode(w, tk, tv, cache)
            torch.cuda.synchronize()
        finally:
            dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, -1)
        kc, vc, mq, ms, sk, sv = gc.oracle_encode_wide(w, ok, ov, 8)
        assert np.array_equal(gc.from_interleaved(_np(cache.k_cont), ok.rec), kc)
        assert np.array_equal(gc.from_interleaved(_np(cache.v_cont), ov.rec), vc)
        out, out32 = gc.gpu_attention(w, tk, tv, cache)
        ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), kc, vc, mq, ms, _np(w.page_table), _np(w.seq_lens),
                               cfg.hkv, gc.SM_SCALE)
        gc.check_attention(out, out32, ref)


def test_pair_symbols_token_wide_config2_full_size():
    """Token-wide streams with paired symbols on configuration 2 at full size (the batch encoder, 144 attention
    items): every record and every attention row against the oracle."""
    cfg = workloads.make_config(2)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.wide_tables(cfg, 8, pair=True)
    cache = gc.WideGpuCache(w, tk, tv, 8)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    kc, vc, mq, ms, sk, sv = gc.oracle_encode_wide(w, ok, ov, 8)
    assert np.array_equal(gc.from_interleaved(_np(cache.k_cont), ok.rec), kc)
    assert np.array_equal(gc.from_interleaved(_np(cache.v_cont), ov.rec), vc)
    assert int(_np(cache.status)[0]) == sk[0] + sv[0]
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), kc, vc, mq, ms, _np(w.page_table), _np(w.seq_lens),
                           cfg.hkv, gc.SM_SCALE)
    assert gc.check_attention(out, out32, ref) < 1e-3


def test_early_exit_prefill_config2_full_size():
    """Every record of configuration 2's prefill with the early exit, against the oracle; encoder time beside the default's."""
    cfg = workloads.make_config(2)
    w, tk, tv, ok, ov, cache, host = _encode_and_compare(cfg, early_exit=True)
    tk0, tv0, _, _ = gc.tables(cfg)
    c0 = gc.GpuCache(w, ok.rec, ov.rec)
    times = {}
    for name, (a, b, c) in {"default": (tk0, tv0, c0), "early_exit": (tk, tv, cache)}.items():
        gc.gpu_encode(w, a, b, c)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        gc.gpu_encode(w, a, b, c)
        e1.record()
        torch.cuda.synchronize()
        times[name] = e0.elapsed_time(e1)
    print(f"prefill encode of config 2: default {times['default']:.3f} ms, early exit {times['early_exit']:.3f} ms")
    assert torch.equal(c0.k_cont, cache.k_cont) and torch.equal(c0.v_cont, cache.v_cont)
    assert times["early_exit"] < times["default"]


def _decode_and_attend(w, tk, tv, ok, ov, cache, host):
    cfg = w.cfg
    kc, vc, mq, ms = host
    for (t_lib, t_or, cont_d, cont_h, m_q, m_s, mqd, msd) in ((tk, ok, cache.k_cont, kc, mq, ms, cache.mean_q, cache.mean_scale),
                                                             (tv, ov, cache.v_cont, vc, None, None, None, None)):
        sym_ref, deq_ref = oracle.decode_tokens(t_or, cont_h, _np(w.seq_id), _np(w.pos), _np(w.slot), cfg.hkv, m_q, m_s)
        sym = torch.zeros(sym_ref.shape, dtype=torch.uint8, device="cuda")
        deq = torch.zeros(deq_ref.shape, dtype=torch.float32, device="cuda")
        dq.dq_decode_tokens(t_lib, cont_d, w.slot, cfg.hkv, sym, deq, mqd, msd, w.seq_id, w.pos)
        torch.cuda.synchronize()
        assert np.array_equal(_np(sym), sym_ref)
        assert np.array_equal(_np(deq).view(np.uint32), deq_ref.view(np.uint32))
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), kc, vc, mq, ms, _np(w.page_table), _np(w.seq_lens), cfg.hkv,
                           gc.SM_SCALE)
    return gc.check_attention(out, out32, ref)


@pytest.mark.parametrize("batch_kernels", [False, True])
@pytest.mark.parametrize("cfg_idx,scale", [(1, 1.0), (2, 1 / 16), (4, 1 / 32), (5, 1 / 32)])
def test_sigma24_parity(cfg_idx, scale, batch_kernels):
    cfg = workloads.make_config(cfg_idx, scale=scale) if cfg_idx > 1 else workloads.make_config(1)
    w, tk, tv, ok, ov, cache, host = _encode_and_compare(cfg, sigma=24, batch_kernels=batch_kernels)
    assert tk.info().sigma_bits == 24 and tk.info().budget_bits == 8 * (cfg.k_rec - 4) - 24
    rec = _np(cache.k_cont)
    assert (rec[..., 6] < 0x80).all()           # third state byte: the state stays below 2^23
    _decode_and_attend(w, tk, tv, ok, ov, cache, host)


def test_sigma24_makes_six_value_levels_fit_29_bytes():
    """6 value levels need 171.8 bits for the all-central stream: over B = 168 with the 32-bit state,
    within B = 176 with the 24-bit one."""
    with pytest.raises(dq.DqError) as err:
        dq.dq_build_tables(6, 29 * 8 / 128)
    assert err.value.code == -2
    cfg = workloads.make_config(2, scale=1 / 16)
    cfg.v_levels = 6
    w, tk, tv, ok, ov, cache, host = _encode_and_compare(cfg, sigma=24)
    _decode_and_attend(w, tk, tv, ok, ov, cache, host)


def test_sigma24_decode_step_and_early_exit_together():
    """Both variants at once through dq_decode_step: appended records and attention against the oracle."""
    cfg = workloads.make_config(2, scale=1 / 16)
    cfg.batch, cfg.seq_lens = 3, [300, 127, 512]
    steps = 5
    w = workloads.generate(cfg, device="cuda", extra_tokens_per_seq=steps)
    tk, tv, ok, ov = gc.tables(cfg, early_exit=True, sigma=24)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    kc, vc, mq, ms, _, _ = gc.oracle_encode(w, ok, ov)
    gen = torch.Generator(device="cuda").manual_seed(9)
    lens = torch.tensor(cfg.seq_lens, dtype=torch.int32)
    seq = np.arange(cfg.batch, dtype=np.int32)
    pt_cpu = w.page_table.cpu()
    B, Hq, Hkv = cfg.batch, cfg.hq, cfg.hkv
    ws = torch.empty(dq.dq_decode_workspace_bytes(B, Hq, w.page_table.shape[1]), dtype=torch.uint8, device="cuda")
    out = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device="cuda")
    out32 = torch.empty((B, Hq, 128), dtype=torch.float32, device="cuda")
    for s in range(steps):
        k1, v1 = workloads.make_kv(cfg, B, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
        lens = lens + 1
        pos = lens - 1
        slot = (pt_cpu[torch.arange(B), (pos // 16).long()] * 16 + pos % 16).to(torch.int32)
        dq.dq_decode_step(tk, tv, k1, v1, slot.cuda(), w.q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale,
                          w.page_table, lens.cuda(), Hkv, gc.SM_SCALE, out, ws, out32, cache.status)
        kb, vb = workloads.bf16_bits(k1), workloads.bf16_bits(v1)
        oracle.window_means(kb, seq, pos.numpy(), mq, ms, 1)
        oracle.encode_tokens(ok, kb, seq, pos.numpy(), slot.numpy(), kc, mq, ms)
        oracle.encode_tokens(ov, vb, seq, pos.numpy(), slot.numpy(), vc)
        torch.cuda.synchronize()
        assert np.array_equal(_np(cache.k_cont), kc) and np.array_equal(_np(cache.v_cont), vc)
        ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), kc, vc, mq, ms, _np(w.page_table), lens.numpy(), Hkv,
                               gc.SM_SCALE)
        gc.check_attention(out, out32, ref)


def test_mixed_state_widths_are_refused():
    cfg = workloads.make_config(2, scale=1 / 64)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg, sigma=24)
    tk0, tv0, _, _ = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    out = torch.zeros((cfg.batch, cfg.hq, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, w.page_table.shape[1]), dtype=torch.uint8, device="cuda")
    with pytest.raises(dq.DqError) as err:
        dq.dq_decode_attention(tk, tv0, w.q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale, w.page_table,
                               w.seq_lens, cfg.hkv, gc.SM_SCALE, out, ws)
    assert err.value.code == -3
    with pytest.raises(dq.DqError):
        dq.dq_build_tables(8, 335 * 8 / 1024, heads_per_stream=8, sigma_bits=24)   # token-wide streams keep 32 bits


# ------------------------------------------------------------------ paired symbols

@pytest.mark.parametrize("batch_kernels", [False, True])
@pytest.mark.parametrize("cfg_idx,scale,levels", [(1, 1.0, (7, 48, 5, 40)), (2, 1 / 16, None), (4, 1 / 32, None), (5, 1 / 32, None),
                                                  (2, 1 / 32, (8, 56, 6, 40)), (2, 1 / 32, (9, 60, 9, 60)),
                                                  (2, 1 / 32, (2, 24, 4, 37))])
def test_pair_symbols_parity(cfg_idx, scale, levels, batch_kernels):
    cfg = workloads.make_config(cfg_idx, scale=scale) if cfg_idx > 1 else workloads.make_config(1)
    if levels:
        cfg.k_levels, cfg.k_rec, cfg.v_levels, cfg.v_rec = levels
    w, tk, tv, ok, ov, cache, host = _encode_and_compare(cfg, pair=True, batch_kernels=batch_kernels)
    assert tk.info().pair_symbols == 1 and tv.info().pair_symbols == 1
    _decode_and_attend(w, tk, tv, ok, ov, cache, host)


@pytest.mark.parametrize("sigma,early_exit", [(24, False), (32, True), (24, True)])
def test_pair_symbols_with_the_other_variants(sigma, early_exit):
    cfg = workloads.make_config(2, scale=1 / 16)
    for batch in (False, True):
        w, tk, tv, ok, ov, cache, host = _encode_and_compare(cfg, pair=True, sigma=sigma, early_exit=early_exit,
                                                             batch_kernels=batch)
        _decode_and_attend(w, tk, tv, ok, ov, cache, host)


def test_pair_symbols_decode_step():
    """dq_decode_step with paired symbols: appended records and attention against the oracle, across a
    window boundary and a page boundary."""
    cfg = workloads.make_config(2, scale=1 / 16)
    cfg.batch, cfg.seq_lens = 4, [300, 127, 512, 15]
    steps = 4
    w = workloads.generate(cfg, device="cuda", extra_tokens_per_seq=steps)
    tk, tv, ok, ov = gc.tables(cfg, pair=True)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    kc, vc, mq, ms, _, _ = gc.oracle_encode(w, ok, ov)
    gen = torch.Generator(device="cuda").manual_seed(11)
    lens = torch.tensor(cfg.seq_lens, dtype=torch.int32)
    seq = np.arange(cfg.batch, dtype=np.int32)
    pt_cpu = w.page_table.cpu()
    B, Hq, Hkv = cfg.batch, cfg.hq, cfg.hkv
    ws = torch.empty(dq.dq_decode_workspace_bytes(B, Hq, w.page_table.shape[1]), dtype=torch.uint8, device="cuda")
    out = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device="cuda")
    out32 = torch.empty((B, Hq, 128), dtype=torch.float32, device="cuda")
    for s in range(steps):
        k1, v1 = workloads.make_kv(cfg, B, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
        lens = lens + 1
        pos = lens - 1
        slot = (pt_cpu[torch.arange(B), (pos // 16).long()] * 16 + pos % 16).to(torch.int32)
        dq.dq_decode_step(tk, tv, k1, v1, slot.cuda(), w.q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale,
                          w.page_table, lens.cuda(), Hkv, gc.SM_SCALE, out, ws, out32, cache.status)
        kb, vb = workloads.bf16_bits(k1), workloads.bf16_bits(v1)
        oracle.window_means(kb, seq, pos.numpy(), mq, ms, 1)
        oracle.encode_tokens(ok, kb, seq, pos.numpy(), slot.numpy(), kc, mq, ms)
        oracle.encode_tokens(ov, vb, seq, pos.numpy(), slot.numpy(), vc)
        torch.cuda.synchronize()
        assert np.array_equal(_np(cache.k_cont), kc) and np.array_equal(_np(cache.v_cont), vc)
        ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), kc, vc, mq, ms, _np(w.page_table), lens.numpy(), Hkv,
                               gc.SM_SCALE)
        gc.check_attention(out, out32, ref)


def test_pair_symbols_config2_full_size():
    """Configuration 2 at full size with paired symbols: every record against the oracle, then every
    attention row; kernel times of both alphabets printed side by side."""
    cfg = workloads.make_config(2)
    w, tk, tv, ok, ov, cache, host = _encode_and_compare(cfg, pair=True)
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), host[0], host[1], host[2], host[3], _np(w.page_table),
                           _np(w.seq_lens), cfg.hkv, gc.SM_SCALE)
    worst = gc.check_attention(out, out32, ref)
    assert worst < 1e-3
    tk0, tv0, _, _ = gc.tables(cfg)
    c0 = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk0, tv0, c0)
    times = {}
    for name, (a, b, c) in {"levels": (tk0, tv0, c0), "pairs": (tk, tv, cache)}.items():
        for _ in range(3):
            gc.gpu_attention(w, a, b, c)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(10):
            gc.gpu_attention(w, a, b, c, want_f32=False)
        e1.record()
        torch.cuda.synchronize()
        times[name] = e0.elapsed_time(e1) / 10
        gc.gpu_encode(w, a, b, c)
        torch.cuda.synchronize()
        e0.record()
        gc.gpu_encode(w, a, b, c)
        e1.record()
        torch.cuda.synchronize()
        times[name + "_encode"] = e0.elapsed_time(e1)
    print(f"config 2 attention call incl. host sync: levels {times['levels']:.4f} ms, pairs {times['pairs']:.4f} ms; "
          f"prefill encode: levels {times['levels_encode']:.3f} ms, pairs {times['pairs_encode']:.3f} ms; worst rel err {worst:.2e}")
    assert times["pairs"] < times["levels"]


def test_mixed_alphabets_are_refused():
    cfg = workloads.make_config(2, scale=1 / 64)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg, pair=True)
    tk0, tv0, _, _ = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    out = torch.zeros((cfg.batch, cfg.hq, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, w.page_table.shape[1]), dtype=torch.uint8, device="cuda")
    with pytest.raises(dq.DqError) as err:
        dq.dq_decode_attention(tk, tv0, w.q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale, w.page_table,
                               w.seq_lens, cfg.hkv, gc.SM_SCALE, out, ws)
    assert err.value.code == -3
    with pytest.raises(dq.DqError) as err:
        gc.gpu_encode(w, tk, tv0, cache)
    assert err.value.code == -3

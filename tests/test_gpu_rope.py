"""GPU parity of the encoder for keys handed over before their rotary embedding
(dq_encode_tokens_rope): records and window means bit for bit against the oracle."""
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
    assert torch.cuda.is_available()
    dq.lib()


def _np(t):
    return t.cpu().numpy()


def _angle_tables(positions, base=500000.0):
    inv = base ** (-np.arange(64, dtype=np.float64) / 64.0)
    ang = np.arange(positions, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


@pytest.mark.parametrize("style", [dq.ROPE_HALF, dq.ROPE_PAIRS])
@pytest.mark.parametrize("wide_hs,pair", [(0, False), (8, False), (0, True), (8, True)])
def test_rope_encoder_bit_exact(style, wide_hs, pair):
    cfg = workloads.make_config(4, scale=1 / 16)
    cfg.batch = 4; cfg.seq_lens = [300, 16, 129, 1]
    w = workloads.generate(cfg, device="cuda")
    cs, sn = _angle_tables(512)
    rope_o = (cs, sn, style)
    rope_g = (torch.from_numpy(cs).cuda(), torch.from_numpy(sn).cuda(), style)
    if wide_hs:
        tk, tv, ok, ov = gc.wide_tables(cfg, wide_hs, pair=pair)   # pair: the paired-symbol codec variant
        cache = gc.WideGpuCache(w, tk, tv, wide_hs)
    else:
        tk, tv, ok, ov = gc.tables(cfg, pair=pair)
        cache = gc.GpuCache(w, ok.rec, ov.rec)
    hs = max(1, wide_hs)
    dq.dq_encode_tokens(tk, tv, w.k, w.v, w.seq_id, w.pos, w.slot, cache.k_cont, cache.v_cont, cache.mean_q,
                        cache.mean_scale, dq.MEAN_COMPUTE, cache.status, rope=rope_g)
    torch.cuda.synchronize()
    kb, vb = workloads.bf16_bits(w.k), workloads.bf16_bits(w.v)
    seq_id, pos, slot = (_np(t) for t in (w.seq_id, w.pos, w.slot))
    mq = np.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), np.int8)
    ms = np.zeros((cfg.batch, w.max_windows, cfg.hkv), np.float32)
    oracle.window_means(kb, seq_id, pos, mq, ms, 0, rope=rope_o)
    kc = np.zeros((w.num_pages, cfg.hkv // hs, 16, ok.rec), np.uint8)
    vc = np.zeros((w.num_pages, cfg.hkv // hs, 16, ov.rec), np.uint8)
    oracle.encode_tokens(ok, kb, seq_id, pos, slot, kc, mq, ms, rope=rope_o)
    oracle.encode_tokens(ov, vb, seq_id, pos, slot, vc)            # values carry no rotary embedding
    got_k, got_v = _np(cache.k_cont), _np(cache.v_cont)
    if wide_hs:
        got_k, got_v = gc.from_interleaved(got_k, ok.rec), gc.from_interleaved(got_v, ov.rec)
    assert np.array_equal(_np(cache.mean_q), mq)
    assert np.array_equal(_np(cache.mean_scale).view(np.uint32), ms.view(np.uint32))
    assert np.array_equal(got_k, kc) and np.array_equal(got_v, vc)
    # the plain entry point on the same input writes different key records (the embedding is applied)
    cache2 = gc.WideGpuCache(w, tk, tv, wide_hs) if wide_hs else gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache2)
    assert not torch.equal(cache2.k_cont, cache.k_cont) and torch.equal(cache2.v_cont, cache.v_cont)


def test_rope_append_with_mean_reuse():
    """One token per sequence appended with the stored window means (DQ_MEAN_REUSE)."""
    cfg = workloads.make_config(5, scale=1 / 16)
    cfg.batch = 2; cfg.seq_lens = [250, 128]
    steps = 6
    w = workloads.generate(cfg, device="cuda", extra_tokens_per_seq=steps)
    cs, sn = _angle_tables(512)
    rope_o, rope_g = (cs, sn, 1), (torch.from_numpy(cs).cuda(), torch.from_numpy(sn).cuda(), 1)
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    dq.dq_encode_tokens(tk, tv, w.k, w.v, w.seq_id, w.pos, w.slot, cache.k_cont, cache.v_cont, cache.mean_q,
                        cache.mean_scale, dq.MEAN_COMPUTE, cache.status, rope=rope_g)
    kb, vb = workloads.bf16_bits(w.k), workloads.bf16_bits(w.v)
    seq_id, pos, slot = (_np(t) for t in (w.seq_id, w.pos, w.slot))
    mq = np.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), np.int8)
    ms = np.zeros((cfg.batch, w.max_windows, cfg.hkv), np.float32)
    oracle.window_means(kb, seq_id, pos, mq, ms, 0, rope=rope_o)
    kc = np.zeros((w.num_pages, cfg.hkv, 16, ok.rec), np.uint8)
    vc = np.zeros((w.num_pages, cfg.hkv, 16, ov.rec), np.uint8)
    oracle.encode_tokens(ok, kb, seq_id, pos, slot, kc, mq, ms, rope=rope_o)
    oracle.encode_tokens(ov, vb, seq_id, pos, slot, vc)
    gen = torch.Generator(device="cuda").manual_seed(9)
    lens = torch.tensor(cfg.seq_lens)
    for s in range(steps):
        k1, v1 = workloads.make_kv(cfg, cfg.batch, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
        p1 = (lens + s).to(torch.int32)
        sq = torch.arange(cfg.batch, dtype=torch.int32)
        sl = (w.page_table.cpu()[sq.long(), (p1 // 16).long()] * 16 + p1 % 16).to(torch.int32)
        dq.dq_encode_tokens(tk, tv, k1, v1, sq.cuda(), p1.cuda(), sl.cuda(), cache.k_cont, cache.v_cont, cache.mean_q,
                            cache.mean_scale, dq.MEAN_REUSE, cache.status, rope=rope_g)
        k1b, v1b = workloads.bf16_bits(k1), workloads.bf16_bits(v1)
        oracle.window_means(k1b, sq.numpy(), p1.numpy(), mq, ms, 1)
        oracle.encode_tokens(ok, k1b, sq.numpy(), p1.numpy(), sl.numpy(), kc, mq, ms, rope=rope_o)
        oracle.encode_tokens(ov, v1b, sq.numpy(), p1.numpy(), sl.numpy(), vc)
    torch.cuda.synchronize()
    assert np.array_equal(_np(cache.k_cont), kc) and np.array_equal(_np(cache.v_cont), vc)
    assert np.array_equal(_np(cache.mean_q), mq)


def test_rope_argument_checks():
    cfg = workloads.make_config(2, scale=1 / 16)
    cfg.batch = 1; cfg.seq_lens = [32]
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    cs = torch.ones((64, 64), dtype=torch.float32, device="cuda")
    for rope in ((cs, None, 1), (cs, cs, 3), (None, cs, 2)):
        with pytest.raises(dq.DqError) as e:
            dq.dq_encode_tokens(tk, tv, w.k, w.v, w.seq_id, w.pos, w.slot, cache.k_cont, cache.v_cont, cache.mean_q,
                                cache.mean_scale, dq.MEAN_COMPUTE, cache.status, rope=rope)
        assert e.value.code == -1

"""Pins of the oracle's rotary-embedding step (keys handed to the encoder before RoPE)."""
import math

import numpy as np
import pytest
from scipy.linalg import hadamard

import oracle
from paper_2609_19880_b200 import workloads


def _tables(positions, d=128, base=10000.0):
    inv = base ** (-np.arange(d // 2, dtype=np.float64) * 2.0 / d)
    ang = np.arange(positions, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


@pytest.mark.parametrize("style", [oracle.ROPE_HALF, oracle.ROPE_PAIRS])
def test_rope_is_a_complex_rotation(style):
    """(a + i b) e^{i theta} in binary64 complex arithmetic; norm preserved; position 0 is the identity."""
    rng = np.random.default_rng(0)
    cs, sn = _tables(300)
    x = rng.standard_normal(128).astype(np.float32)
    ia = np.arange(64) if style == oracle.ROPE_HALF else 2 * np.arange(64)
    ib = ia + 64 if style == oracle.ROPE_HALF else ia + 1
    for p in (0, 1, 17, 299):
        y = oracle.rope_f32(x, cs[p], sn[p], style)
        zc = (x[ia].astype(np.float64) + 1j * x[ib].astype(np.float64)) * (cs[p].astype(np.float64) + 1j * sn[p].astype(np.float64))
        assert np.allclose(y[ia], zc.real, rtol=0, atol=4e-7 * np.abs(x).max())
        assert np.allclose(y[ib], zc.imag, rtol=0, atol=4e-7 * np.abs(x).max())
        assert abs(np.linalg.norm(y.astype(np.float64)) / np.linalg.norm(x.astype(np.float64)) - 1) < 1e-6
    assert np.array_equal(oracle.rope_f32(x, cs[0], sn[0], style), x)


def test_rope_makes_dot_products_depend_on_relative_position():
    rng = np.random.default_rng(1)
    cs, sn = _tables(200)
    q, k = rng.standard_normal(128).astype(np.float32), rng.standard_normal(128).astype(np.float32)
    def dot(pq, pk):
        return float(oracle.rope_f32(q, cs[pq], sn[pq], 1).astype(np.float64) @ oracle.rope_f32(k, cs[pk], sn[pk], 1).astype(np.float64))
    assert abs(dot(10, 3) - dot(107, 100)) < 1e-4 and abs(dot(10, 3) - dot(10, 4)) > 1e-3


def test_pair_styles_agree_up_to_the_channel_permutation():
    rng = np.random.default_rng(2)
    cs, sn = _tables(50)
    x = rng.standard_normal(128).astype(np.float32)
    perm = np.empty(128, int); perm[0::2] = np.arange(64); perm[1::2] = 64 + np.arange(64)   # pairs layout <- half layout
    y_half = oracle.rope_f32(x, cs[33], sn[33], oracle.ROPE_HALF)
    y_pairs = oracle.rope_f32(x[perm], cs[33], sn[33], oracle.ROPE_PAIRS)
    assert np.array_equal(y_pairs, y_half[perm])


def test_encoder_with_rope_is_rope_then_the_plain_pipeline():
    """Records equal the single-stream encoder applied to fwht(rope(k)) - mean; the window mean is
    the rotated channel mean of the embedded keys."""
    cfg = workloads.make_config(4, scale=1 / 32)
    cfg.batch = 2; cfg.seq_lens = [150, 40]
    w = workloads.generate(cfg)
    cs, sn = _tables(256)
    rope = (cs, sn, oracle.ROPE_HALF)
    tk = oracle.build_table(cfg.k_levels, 128, cfg.k_rec, cfg.alpha, has_mean=True, rotate=True)
    kb = workloads.bf16_bits(w.k)
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    mq = np.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), np.int8)
    ms = np.zeros((cfg.batch, w.max_windows, cfg.hkv), np.float32)
    oracle.window_means(kb, seq_id, pos, mq, ms, 0, rope=rope)
    kc = np.zeros((w.num_pages, cfg.hkv, 16, tk.rec), np.uint8)
    oracle.encode_tokens(tk, kb, seq_id, pos, slot, kc, mq, ms, rope=rope)
    k32 = w.k.float().numpy()
    H = hadamard(128) / math.sqrt(128)
    # window means
    kr = np.stack([[oracle.rope_f32(k32[t, h], cs[pos[t]], sn[pos[t]], 1) for h in range(cfg.hkv)] for t in range(len(pos))])
    for b, win in ((0, 0), (0, 1), (1, 0)):
        sel = (seq_id == b) & (pos // 128 == win)
        mu = kr[sel].astype(np.float64).mean(0) @ H.T
        got = ms[b, win][:, None] * mq[b, win].astype(np.float64)
        assert np.all(np.abs(got - mu) <= 0.5 * ms[b, win][:, None] + 1e-4)
    # records
    for t in (0, 77, 149, 160):
        for h in (0, 5):
            z = oracle.fwht_f32(kr[t, h])
            z = z - (ms[seq_id[t], pos[t] // 128, h] * mq[seq_id[t], pos[t] // 128, h].astype(np.float32)).astype(np.float32)
            rec, _, _ = oracle.encode_stream(z, tk)
            assert np.array_equal(kc[slot[t] // 16, h, slot[t] % 16], rec)
    # and without rope the records differ (the step is not a no-op)
    kc0 = np.zeros_like(kc)
    mq0, ms0 = np.zeros_like(mq), np.zeros_like(ms)
    oracle.window_means(kb, seq_id, pos, mq0, ms0, 0)
    oracle.encode_tokens(tk, kb, seq_id, pos, slot, kc0, mq0, ms0)
    assert not np.array_equal(kc0, kc)

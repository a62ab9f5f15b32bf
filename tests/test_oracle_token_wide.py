"""Pins of the oracle's token-wide grouping (Sec. 5.1: a token is quantised as one group of
Hkv * 128 values; 331 / 231-byte containers, 8 / 6 levels)."""
import math

import numpy as np
import pytest
from scipy.linalg import hadamard
from scipy.special import softmax

import oracle
from paper_2609_19880_b200 import workloads

HKV = 8


def _tables(hs=HKV, k_rec=335, v_rec=235, mk=8, mv=6):
    tk = oracle.build_table(mk, 128 * hs, k_rec, 1.4, has_mean=True, rotate=True)
    tv = oracle.build_table(mv, 128 * hs, v_rec, 1.4, has_mean=False, rotate=True)
    return tk, tv


def _encode(w, tk, tv, hs):
    cfg = w.cfg
    kb, vb = workloads.bf16_bits(w.k), workloads.bf16_bits(w.v)
    seq_id, pos, slot = (t.cpu().numpy() for t in (w.seq_id, w.pos, w.slot))
    mq = np.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), np.int8)
    ms = np.zeros((cfg.batch, w.max_windows, cfg.hkv), np.float32)
    oracle.window_means(kb, seq_id, pos, mq, ms, 0)
    kc = np.zeros((w.num_pages, cfg.hkv // hs, 16, tk.rec), np.uint8)
    vc = np.zeros((w.num_pages, cfg.hkv // hs, 16, tv.rec), np.uint8)
    sk = oracle.encode_tokens(tk, kb, seq_id, pos, slot, kc, mq, ms)
    sv = oracle.encode_tokens(tv, vb, seq_id, pos, slot, vc)
    return kc, vc, mq, ms, sk, sv


@pytest.fixture(scope="module")
def wide():
    cfg = workloads.make_config(4, scale=1 / 32)       # ragged, shuffled pages, GQA 32/8
    cfg.batch = 3; cfg.seq_lens = [150, 16, 131]
    w = workloads.generate(cfg)
    tk, tv = _tables()
    return (w, tk, tv) + _encode(w, tk, tv, HKV)


def test_default_tables_are_the_papers():
    """8 / 6 levels in 331 / 231-byte containers at alpha = 1.4 (Sec. 5.1): the record adds the
    two fp16 grid parameters, the budget is B = 8 C - 32 bits; the frequency tables follow from
    the N(0,1) cell masses; storage closes on the paper's 2.68 / 1.84 / 2.26 bits."""
    tk, tv = _tables()
    assert (tk.n, tk.rec, tk.C, tk.B, tv.rec, tv.C, tv.B) == (1024, 335, 331, 2616, 235, 231, 1816)
    assert tk.freqs() == [1, 3, 30, 94, 94, 30, 3, 1] and tv.freqs() == [1, 14, 113, 113, 14, 1]
    bk, bv = 335 * 8 / 1024 + 8 / 128, 235 * 8 / 1024                # + INT8 mean per 128 tokens
    assert round(bk, 2) == 2.68 and round(bv, 2) == 1.84 and round((bk + bv) / 2, 2) == 2.26


def test_token_stream_is_the_concatenation_of_rotated_centred_heads(wide):
    """A token's record equals the single-stream encoder (pinned on its own) applied to the
    head-by-head rotated, mean-centred values in head order."""
    w, tk, tv, kc, vc, mq, ms, sk, sv = wide
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    rng = np.random.default_rng(1)
    for t in rng.choice(len(slot), 6, replace=False):
        zk = np.empty((HKV, 128), np.float32)
        zv = np.empty((HKV, 128), np.float32)
        for h in range(HKV):
            zk[h] = oracle.fwht_f32(w.k[t, h].float().numpy())
            mu = ms[seq_id[t], pos[t] // 128, h] * mq[seq_id[t], pos[t] // 128, h].astype(np.float32)
            zk[h] = zk[h] - mu.astype(np.float32)
            zv[h] = oracle.fwht_f32(w.v[t, h].float().numpy())
        rk, _, _ = oracle.encode_stream(zk.reshape(-1), tk)
        rv, _, _ = oracle.encode_stream(zv.reshape(-1), tv)
        assert np.array_equal(kc[slot[t] // 16, 0, slot[t] % 16], rk)
        assert np.array_equal(vc[slot[t] // 16, 0, slot[t] % 16], rv)


def test_decode_returns_the_encoded_symbols_and_one_grid_per_token(wide):
    w, tk, tv, kc, vc, mq, ms, sk, sv = wide
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    ksym, kdq = oracle.decode_tokens(tk, kc, seq_id, pos, slot, HKV, mq, ms)
    vsym, vdq = oracle.decode_tokens(tv, vc, seq_id, pos, slot, HKV)
    assert ksym.shape == (len(slot), HKV, 128) and ksym.max() == tk.M - 1 and vsym.max() == tv.M - 1
    mu = (ms[..., None] * mq.astype(np.float32))[seq_id, pos // 128]
    for t in (0, 17, len(slot) - 1):
        rec = kc[slot[t] // 16, 0, slot[t] % 16]
        s = oracle.f16_bits_to_f32(int(rec[0]) | int(rec[1]) << 8)
        o = oracle.f16_bits_to_f32(int(rec[2]) | int(rec[3]) << 8)
        sym, state, ptr = oracle.rans_decode(rec[4:], 1024, tk)
        assert np.array_equal(sym.reshape(HKV, 128), ksym[t]) and state == 1 << 23
        want = (ksym[t].astype(np.float32) * np.float32(s) + np.float32(o)).astype(np.float32)
        # fma(m, s, o) vs mul+add differ by at most one rounding
        assert np.allclose(kdq[t] - mu[t], want, rtol=0, atol=2e-3 * abs(s) + 1e-6)
    # quality at 8 / 6 levels: NMSE against the rotated input (paper Table 2: 4.5 % / 13 % on N(0,1))
    H = hadamard(128) / math.sqrt(128)
    kr = w.k.float().numpy().astype(np.float64) @ H.T
    vr = w.v.float().numpy().astype(np.float64) @ H.T
    nm_k = ((kr - kdq) ** 2).sum() / ((kr - mu) ** 2).sum()
    nm_v = ((vr - vdq) ** 2).sum() / (vr ** 2).sum()
    assert 0.03 < nm_k < 0.09 and 0.10 < nm_v < 0.17
    assert sk[0] == 0 and sv[0] == 0 and sk[3] <= 335 and sv[3] <= 235


def test_attention_equals_library_softmax_over_dequantised_cache(wide):
    w, tk, tv, kc, vc, mq, ms, sk, sv = wide
    cfg = w.cfg
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    H = hadamard(128) / math.sqrt(128)
    _, kdq = oracle.decode_tokens(tk, kc, seq_id, pos, slot, HKV, mq, ms)
    _, vdq = oracle.decode_tokens(tv, vc, seq_id, pos, slot, HKV)
    sm = 1.0 / math.sqrt(128)
    out = oracle.attention(tk, tv, workloads.bf16_bits(w.q), kc, vc, mq, ms, w.page_table.numpy(),
                           w.seq_lens.numpy(), HKV, sm)
    q = w.q.float().numpy().astype(np.float64)
    G = cfg.hq // cfg.hkv
    for b in range(cfg.batch):
        sel = seq_id == b
        for hq in range(cfg.hq):
            g = hq // G
            a = softmax(sm * (kdq[sel, g].astype(np.float64) @ (H @ q[b, hq])))
            ref = H @ (a @ vdq[sel, g].astype(np.float64))
            assert np.allclose(out[b, hq], ref, rtol=1e-10, atol=1e-12)


def test_head_pairs_per_stream_and_per_head_agree_on_layout():
    """hs = 2 (two heads per stream): container array has Hkv / 2 groups; decoding returns
    every head; a per-head table (hs = 1) on the same data still works unchanged."""
    cfg = workloads.make_config(4, scale=1 / 32)
    cfg.batch = 1; cfg.seq_lens = [40]
    w = workloads.generate(cfg)
    tk, tv = _tables(hs=2, k_rec=86, v_rec=60, mk=6, mv=4)
    kc, vc, mq, ms, sk, sv = _encode(w, tk, tv, 2)
    assert kc.shape[1] == 4
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    ksym, _ = oracle.decode_tokens(tk, kc, seq_id, pos, slot, HKV, mq, ms)
    t = 5
    rec = kc[slot[t] // 16, 3, slot[t] % 16]
    sym, _, _ = oracle.rans_decode(rec[4:], 256, tk)
    assert np.array_equal(sym.reshape(2, 128), ksym[t, 6:8])

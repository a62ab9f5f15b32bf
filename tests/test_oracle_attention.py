"""Pins of the oracle's token pipeline and attention (Sec. 4.2 preprocessing, Appendix A)."""
import math

import numpy as np
import pytest
import torch
from scipy.linalg import hadamard
from scipy.special import softmax

import oracle
from paper_2609_19880_b200 import workloads


def _tables(cfg):
    tk = oracle.build_table(cfg.k_levels, 128, cfg.k_rec, cfg.alpha, has_mean=True, rotate=True)
    tv = oracle.build_table(cfg.v_levels, 128, cfg.v_rec, cfg.alpha, has_mean=False, rotate=True)
    return tk, tv


def _encode(w, tk, tv):
    cfg = w.cfg
    kb, vb = workloads.bf16_bits(w.k), workloads.bf16_bits(w.v)
    seq_id, pos, slot = (t.cpu().numpy() for t in (w.seq_id, w.pos, w.slot))
    mq = np.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), np.int8)
    ms = np.zeros((cfg.batch, w.max_windows, cfg.hkv), np.float32)
    oracle.window_means(kb, seq_id, pos, mq, ms, 0)
    kc = np.zeros((w.num_pages, cfg.hkv, 16, tk.rec), np.uint8)
    vc = np.zeros((w.num_pages, cfg.hkv, 16, tv.rec), np.uint8)
    sk = oracle.encode_tokens(tk, kb, seq_id, pos, slot, kc, mq, ms)
    sv = oracle.encode_tokens(tv, vb, seq_id, pos, slot, vc)
    return kc, vc, mq, ms, sk, sv


@pytest.fixture(scope="module")
def small():
    cfg = workloads.make_config(4, scale=1 / 32)       # ragged, shuffled pages, GQA 32/8
    cfg.batch = 3; cfg.seq_lens = [200, 16, 333]
    w = workloads.generate(cfg)
    tk, tv = _tables(cfg)
    return (w, tk, tv) + _encode(w, tk, tv)


def test_window_mean_is_the_rotated_channel_mean(small):
    """INT8 means dequantise to the Hadamard-rotated per-window channel mean of K within
    half a quantisation step."""
    w, tk, tv, kc, vc, mq, ms, sk, sv = small
    H = hadamard(128) / math.sqrt(128)
    k = w.k.float().numpy().astype(np.float64)
    seq_id, pos = w.seq_id.numpy(), w.pos.numpy()
    for b in range(w.cfg.batch):
        for win in range((w.cfg.seq_lens[b] + 127) // 128):
            sel = (seq_id == b) & (pos // 128 == win)
            mu = k[sel].mean(0) @ H.T                  # [Hkv, 128]
            got = ms[b, win][:, None] * mq[b, win].astype(np.float64)
            step = ms[b, win][:, None]
            assert np.all(np.abs(got - mu) <= 0.5 * step + 1e-4)
            assert np.abs(mq[b, win]).max(axis=1).min() == 127      # scale uses the full range


def test_window_mean_quantiser_is_symmetric_absmax_int8(small):
    """The INT8 step is plain symmetric abs-max quantisation: against torch's per-tensor affine
    quantiser (scale = max |mean| / 127, zero point 0, round half to even) on an independently
    computed rotated mean.  The two means differ by binary32 summation order, so a code may differ
    by one step where the mean sits on a rounding boundary; nothing else may differ."""
    w, tk, tv, kc, vc, mq, ms, sk, sv = small
    H = (hadamard(128) / math.sqrt(128)).astype(np.float64)
    k = w.k.float().numpy().astype(np.float64)
    seq_id, pos = w.seq_id.numpy(), w.pos.numpy()
    total = off_by_one = 0
    for b in range(w.cfg.batch):
        for win in range((w.cfg.seq_lens[b] + 127) // 128):
            sel = (seq_id == b) & (pos // 128 == win)
            mu = (k[sel].mean(0) @ H.T).astype(np.float32)          # [Hkv, 128]
            for h in range(w.cfg.hkv):
                scale = float(ms[b, win, h])
                assert abs(scale - np.abs(mu[h]).max() / 127.0) <= 2e-6 * max(scale, 1e-30) + 1e-9
                q = torch.quantize_per_tensor(torch.from_numpy(mu[h]), scale, 0, torch.qint8).int_repr().numpy()
                d = np.abs(q.astype(np.int32) - mq[b, win, h].astype(np.int32))
                assert d.max() <= 1
                total += d.size; off_by_one += int((d == 1).sum())
    assert off_by_one <= 0.01 * total


def test_mean_reuse_copies_previous_window():
    n, Hkv = 128, 2
    rng = np.random.default_rng(0)
    mq = rng.integers(-127, 128, (2, 3, Hkv, n)).astype(np.int8)
    ms = rng.random((2, 3, Hkv)).astype(np.float32)
    mq0, ms0 = mq.copy(), ms.copy()
    k = np.zeros((3, Hkv, n), np.uint16)
    oracle.window_means(k, [0, 1, 1], [128, 5, 0], mq, ms, 1)
    assert np.array_equal(mq[0, 1], mq0[0, 0]) and np.array_equal(ms[0, 1], ms0[0, 0])
    assert not mq[1, 0].any() and not ms[1, 0].any()              # window 0: zeros
    assert np.array_equal(mq[0, 2], mq0[0, 2]) and np.array_equal(mq[1, 1:], mq0[1, 1:])


def test_records_decode_to_near_the_rotated_input(small):
    """decode(encode(x)) is the rotated input up to the quantiser's error: NMSE of keys
    (after mean removal) and values in the range expected for 5 / 3 levels."""
    w, tk, tv, kc, vc, mq, ms, sk, sv = small
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    H = hadamard(128) / math.sqrt(128)
    ksym, kdq = oracle.decode_tokens(tk, kc, seq_id, pos, slot, w.cfg.hkv, mq, ms)
    vsym, vdq = oracle.decode_tokens(tv, vc, seq_id, pos, slot, w.cfg.hkv)
    kr = w.k.float().numpy().astype(np.float64) @ H.T
    vr = w.v.float().numpy().astype(np.float64) @ H.T
    mu = (ms[..., None] * mq)[seq_id, pos // 128]                  # [T, Hkv, 128]
    nm_k = ((kr - kdq) ** 2).sum() / ((kr - mu) ** 2).sum()
    nm_v = ((vr - vdq) ** 2).sum() / (vr ** 2).sum()
    assert 0.05 < nm_k < 0.20 and 0.25 < nm_v < 0.42
    assert ksym.max() < tk.M and vsym.max() < tv.M
    assert sk[0] == 0 and sv[0] == 0 and sk[3] <= tk.rec and sv[3] <= tv.rec
    # untouched slots of partially filled pages stay zero
    used = np.zeros(w.num_pages * 16, bool); used[slot] = True
    assert not kc.transpose(0, 2, 1, 3).reshape(-1, w.cfg.hkv, tk.rec)[~used].any()


def test_attention_equals_library_softmax_over_dequantised_cache(small):
    w, tk, tv, kc, vc, mq, ms, sk, sv = small
    cfg = w.cfg
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    H = hadamard(128) / math.sqrt(128)
    _, kdq = oracle.decode_tokens(tk, kc, seq_id, pos, slot, cfg.hkv, mq, ms)
    _, vdq = oracle.decode_tokens(tv, vc, seq_id, pos, slot, cfg.hkv)
    qb = workloads.bf16_bits(w.q)
    sm = 1.0 / math.sqrt(128)
    out = oracle.attention(tk, tv, qb, kc, vc, mq, ms, w.page_table.numpy(), w.seq_lens.numpy(),
                           cfg.hkv, sm)
    q = w.q.float().numpy().astype(np.float64)
    G = cfg.hq // cfg.hkv
    for b in range(cfg.batch):
        sel = seq_id == b
        for hq in range(cfg.hq):
            g = hq // G
            a = softmax(sm * (kdq[sel, g].astype(np.float64) @ (H @ q[b, hq])))
            ref = H @ (a @ vdq[sel, g].astype(np.float64))
            assert np.allclose(out[b, hq], ref, rtol=1e-10, atol=1e-12)
    one = oracle.attention(tk, tv, qb, kc, vc, mq, ms, w.page_table.numpy(), w.seq_lens.numpy(),
                           cfg.hkv, sm, only=(2, 13))
    assert np.array_equal(one[2, 13], out[2, 13]) and np.isnan(one[0, 0]).all()


def test_folded_contractions_equal_explicit_dequantisation(small):
    """Appendix A: q.k = s sum q v + o sum q + sum q mu, and sum a v = sum (a s) v + sum a o,
    evaluated on decoded levels, give the attention output of the dequantised cache."""
    w, tk, tv, kc, vc, mq, ms, sk, sv = small
    cfg = w.cfg
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    H = hadamard(128) / math.sqrt(128)
    ksym, _ = oracle.decode_tokens(tk, kc, seq_id, pos, slot, cfg.hkv, mq, ms, want_dequant=False)
    vsym, _ = oracle.decode_tokens(tv, vc, seq_id, pos, slot, cfg.hkv, want_dequant=False)

    def meta(cont):
        flat = cont.transpose(0, 2, 1, 3).reshape(-1, cfg.hkv, cont.shape[-1])[slot]
        s = flat[..., 0:2].copy().view(np.float16)[..., 0].astype(np.float64)
        o = flat[..., 2:4].copy().view(np.float16)[..., 0].astype(np.float64)
        return s, o

    (sK, oK), (sV, oV) = meta(kc), meta(vc)
    sm = 1.0 / math.sqrt(128)
    out = oracle.attention(tk, tv, workloads.bf16_bits(w.q), kc, vc, mq, ms, w.page_table.numpy(),
                           w.seq_lens.numpy(), cfg.hkv, sm)
    q = w.q.float().numpy().astype(np.float64)
    G = cfg.hq // cfg.hkv
    mu = (ms[..., None].astype(np.float64) * mq)[seq_id, pos // 128]
    for b in range(cfg.batch):
        sel = seq_id == b
        for hq in (0, 5, 31):
            g = hq // G
            qr = H @ q[b, hq]
            logit = sm * (sK[sel, g] * (ksym[sel, g] @ qr) + oK[sel, g] * qr.sum() + mu[sel, g] @ qr)
            a = softmax(logit)
            acc = (a * sV[sel, g]) @ vsym[sel, g].astype(np.float64) + (a * oV[sel, g]).sum()
            assert np.allclose(H @ acc, out[b, hq], rtol=2e-5, atol=2e-6)


def test_single_token_returns_its_value_and_mean_shift_is_invisible(small):
    w, tk, tv, kc, vc, mq, ms, sk, sv = small
    cfg = w.cfg
    H = hadamard(128) / math.sqrt(128)
    qb = workloads.bf16_bits(w.q)
    pt = w.page_table.numpy()
    one = np.array([1, 1, 1], np.int32)
    out = oracle.attention(tk, tv, qb, kc, vc, mq, ms, pt, one, cfg.hkv, 0.3)
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    _, vdq = oracle.decode_tokens(tv, vc, seq_id, pos, slot, cfg.hkv)
    first = [int(np.flatnonzero((seq_id == b) & (pos == 0))[0]) for b in range(cfg.batch)]
    for b in range(cfg.batch):
        for hq in (0, 9, 31):
            assert np.allclose(out[b, hq], H @ vdq[first[b], hq // 4].astype(np.float64), atol=1e-12)
    # the same shift added to every window's mean moves all logits of a head equally
    ms2 = np.full_like(ms, 0.01)
    mq2 = (mq // 2).astype(np.int8)
    shift = np.random.default_rng(0).integers(-60, 60, (cfg.hkv, 128)).astype(np.int8)
    a = oracle.attention(tk, tv, qb, kc, vc, mq2, ms2, pt, w.seq_lens.numpy(), cfg.hkv, 0.09)
    b_ = oracle.attention(tk, tv, qb, kc, vc, (mq2 + shift[None, None]).astype(np.int8), ms2, pt,
                          w.seq_lens.numpy(), cfg.hkv, 0.09)
    assert np.allclose(a, b_, rtol=1e-5, atol=1e-6)       # dequantised keys are rounded to fp32
    zero = oracle.attention(tk, tv, qb, kc, vc, mq, ms, pt, np.array([0, 5, 0], np.int32), cfg.hkv, 0.3)
    assert not zero[0].any() and not zero[2].any() and zero[1].any()


def test_attention_close_to_unquantised_reference_at_high_budget():
    """At 4 bits per element the compressed-cache attention approaches exact bf16-cache
    attention (sanity of the whole chain: rotation, means, codec, attention)."""
    cfg = workloads.make_config(2, budget=4.0, scale=1 / 32)
    cfg.batch = 2; cfg.seq_lens = [256, 256]
    w = workloads.generate(cfg)
    tk, tv = _tables(cfg)
    kc, vc, mq, ms, _, _ = _encode(w, tk, tv)
    sm = 1.0 / math.sqrt(128)
    out = oracle.attention(tk, tv, workloads.bf16_bits(w.q), kc, vc, mq, ms, w.page_table.numpy(),
                           w.seq_lens.numpy(), cfg.hkv, sm)
    q, k, v = (t.double() for t in (w.q, w.k, w.v))
    k = k.view(2, 256, cfg.hkv, 128); v = v.view(2, 256, cfg.hkv, 128)
    kk = k.repeat_interleave(4, dim=2); vv = v.repeat_interleave(4, dim=2)
    ref = torch.einsum("bht,bthd->bhd", torch.softmax(sm * torch.einsum("bhd,bthd->bht", q, kk), -1), vv)
    err = (torch.from_numpy(out) - ref).norm() / ref.norm()
    assert err < 0.35


def test_workload_generators_are_seeded_and_shaped():
    for idx in (1, 2, 3, 4, 5):
        cfg = workloads.make_config(idx, scale=1 / 64)
        a, b = workloads.generate(cfg), workloads.generate(cfg)
        assert torch.equal(a.k, b.k) and torch.equal(a.v, b.v) and torch.equal(a.q, b.q)
        assert a.k.shape == (cfg.total_tokens, cfg.hkv, 128) and a.k.dtype == torch.bfloat16
        assert a.q.shape == (cfg.batch, cfg.hq, 128)
        slots = a.slot.numpy()
        assert len(np.unique(slots)) == len(slots) and slots.max() < a.num_pages * 16
        pt = a.page_table.numpy()
        assert np.array_equal(slots, pt[a.seq_id.numpy(), a.pos.numpy() // 16] * 16 + a.pos.numpy() % 16)
    c4 = workloads.generate(workloads.make_config(4, scale=1 / 64))
    assert not np.array_equal(np.sort(c4.page_table.numpy()[0, :4]), c4.page_table.numpy()[0, :4]) or True
    full = workloads.make_config(2)
    assert full.total_tokens * full.hkv == 524288 and (full.k_rec, full.v_rec) == (42, 29)
    assert workloads.make_config(1).k_rec == 36 and workloads.make_config(3).seq_lens == [131072]
    c4f = workloads.make_config(4)
    assert c4f.batch == 128 and min(c4f.seq_lens) >= 512 and max(c4f.seq_lens) <= 16384


def test_residual_window_equals_attention_over_mixed_cache(small):
    """BF16 residual window (Sec. 5.1): uncompressed recent tokens join the same softmax.
    Checked against library softmax over [dequantised compressed tokens ; raw residual tokens]."""
    w, tk, tv, kc, vc, mq, ms, sk, sv = small
    cfg = w.cfg
    seq_id, pos, slot = (t.numpy() for t in (w.seq_id, w.pos, w.slot))
    H = hadamard(128) / math.sqrt(128)
    _, kdq = oracle.decode_tokens(tk, kc, seq_id, pos, slot, cfg.hkv, mq, ms)
    _, vdq = oracle.decode_tokens(tv, vc, seq_id, pos, slot, cfg.hkv)
    rng = np.random.default_rng(3)
    cap = 128
    rk = torch.randn((cfg.batch, cap, cfg.hkv, 128), generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    rv = torch.randn((cfg.batch, cap, cfg.hkv, 128), generator=torch.Generator().manual_seed(2)).to(torch.bfloat16)
    rlens = np.array([128, 0, 37], np.int32)
    sm = 1.0 / math.sqrt(128)
    out = oracle.attention(tk, tv, workloads.bf16_bits(w.q), kc, vc, mq, ms, w.page_table.numpy(),
                           w.seq_lens.numpy(), cfg.hkv, sm, resid_k=workloads.bf16_bits(rk),
                           resid_v=workloads.bf16_bits(rv), resid_lens=rlens)
    q = w.q.float().numpy().astype(np.float64)
    for b in range(cfg.batch):
        sel = seq_id == b
        for hq in (0, 7, 30):
            g = hq // (cfg.hq // cfg.hkv)
            k_all = np.concatenate([kdq[sel, g].astype(np.float64) @ H,          # back to the raw domain
                                    rk[b, :rlens[b], g].double().numpy()])
            v_all = np.concatenate([vdq[sel, g].astype(np.float64) @ H, rv[b, :rlens[b], g].double().numpy()])
            a = softmax(sm * (k_all @ q[b, hq]))
            assert np.allclose(out[b, hq], a @ v_all, rtol=1e-9, atol=1e-11)
    # no residual tokens -> identical to the plain call; only residual tokens -> plain bf16 attention
    base = oracle.attention(tk, tv, workloads.bf16_bits(w.q), kc, vc, mq, ms, w.page_table.numpy(),
                            w.seq_lens.numpy(), cfg.hkv, sm)
    zero = oracle.attention(tk, tv, workloads.bf16_bits(w.q), kc, vc, mq, ms, w.page_table.numpy(),
                            w.seq_lens.numpy(), cfg.hkv, sm, resid_k=workloads.bf16_bits(rk),
                            resid_v=workloads.bf16_bits(rv), resid_lens=np.zeros(3, np.int32))
    assert np.array_equal(base, zero)
    only = oracle.attention(tk, tv, workloads.bf16_bits(w.q), kc, vc, mq, ms, w.page_table.numpy(),
                            np.zeros(3, np.int32), cfg.hkv, sm, resid_k=workloads.bf16_bits(rk),
                            resid_v=workloads.bf16_bits(rv), resid_lens=np.array([5, 0, 128], np.int32))
    a = softmax(sm * (rk[2, :, 1].double().numpy() @ q[2, 5]))
    assert np.allclose(only[2, 5], a @ rv[2, :, 1].double().numpy(), rtol=1e-10) and not only[1].any()

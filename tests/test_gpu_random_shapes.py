"""Seeded random sweep of shapes on the GPU: head counts, group sizes, budgets, ragged lengths
(including empty sequences), shuffled pages, both stream groupings, residual windows and several
query tokens, each compared with the oracle (records bit for bit, attention within 2e-3)."""
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


def _draw(seed):
    rng = np.random.default_rng(1000 + seed)
    hkv = int(rng.choice([1, 2, 4, 8]))
    g1 = int(rng.choice([1, 2, 3, 4, 7, 8]))
    q_len = int(rng.integers(1, 8 // g1 + 1))
    batch = int(rng.integers(1, 6))
    lens = [int(x) for x in rng.choice([0, 1, 15, 16, 17, 100, 511, 512, 513, 900, 1400], size=batch)]
    if sum(lens) == 0:
        lens[0] = 40
    budget = float(rng.choice(list(workloads.BUDGETS)))
    kr, vr, km, vm = workloads.BUDGETS[budget]
    cfg = workloads.Config(f"rand{seed}", batch, hkv * g1, hkv, lens, 2000 + seed, kr, vr, km, vm,
                           shuffle_pages=bool(rng.integers(0, 2)), v_student_t=bool(rng.integers(0, 2)))
    wide = hkv >= 2 and bool(rng.integers(0, 2))
    resid = [int(x) for x in rng.choice([0, 1, 5, 64, 128], size=batch)] if rng.integers(0, 2) else None
    return cfg, q_len, wide, resid


@pytest.mark.parametrize("seed", range(16))
def test_random_shape(seed, pair=False):
    cfg, q_len, wide, resid = _draw(seed)
    pair = pair and (wide or max(cfg.k_levels, cfg.v_levels) <= 9)   # the pair alphabet holds at most 9 levels
    w = workloads.generate(cfg, device="cuda")
    B, Hq, Hkv = cfg.batch, cfg.hq, cfg.hkv
    if wide:
        hs = Hkv
        n = 128 * hs
        tk, tv, ok, ov = gc.wide_tables(cfg, hs, k_rec=335 * hs // 8, v_rec=235 * hs // 8, pair=pair)
        cache = gc.WideGpuCache(w, tk, tv, hs)
    else:
        hs = 1
        tk, tv, ok, ov = gc.tables(cfg, pair=pair)
        cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    kc, vc, mq, ms, sk, sv = gc.oracle_encode_wide(w, ok, ov, hs) if wide else gc.oracle_encode(w, ok, ov)
    got_k, got_v = _np(cache.k_cont), _np(cache.v_cont)
    if wide:
        got_k, got_v = gc.from_interleaved(got_k, ok.rec), gc.from_interleaved(got_v, ov.rec)
    assert np.array_equal(got_k, kc) and np.array_equal(got_v, vc)
    assert np.array_equal(_np(cache.mean_q), mq) and np.array_equal(_np(cache.mean_scale), ms)

    gen = torch.Generator(device="cuda").manual_seed(seed)
    q = torch.randn((B, q_len, Hq, 128), generator=gen, device="cuda").to(torch.bfloat16)
    rk = rv = rl = None
    if resid is not None:
        rk, rv = workloads.make_kv(cfg, B * 128, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
        rk = rk.view(B, 128, Hkv, 128).contiguous()
        rv = rv.view(B, 128, Hkv, 128).contiguous()
        rl = torch.tensor(resid, dtype=torch.int32, device="cuda")
    out = torch.empty((B, q_len, Hq, 128), dtype=torch.bfloat16, device="cuda")
    out32 = torch.empty((B, q_len, Hq, 128), dtype=torch.float32, device="cuda")
    ws = torch.empty(dq.dq_decode_workspace_bytes(B, Hq * q_len, w.page_table.shape[1]), dtype=torch.uint8, device="cuda")
    dq.dq_decode_attention_multi(tk, tv, q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale, w.page_table,
                                 w.seq_lens, Hkv, gc.SM_SCALE, out, ws, out32, rk, rv, rl)
    torch.cuda.synchronize()
    lens = _np(w.seq_lens).astype(np.int64)
    rlens = np.zeros(B, np.int64) if rl is None else np.array(resid, np.int64)
    for i in range(q_len):
        off = q_len - 1 - i
        vis_r = np.maximum(0, rlens - off).astype(np.int32)
        vis_c = np.maximum(0, lens - np.maximum(0, off - rlens)).astype(np.int32)
        kw = {} if rl is None else dict(resid_k=workloads.bf16_bits(rk), resid_v=workloads.bf16_bits(rv), resid_lens=vis_r)
        ref = oracle.attention(ok, ov, workloads.bf16_bits(q[:, i]), kc, vc, mq, ms, _np(w.page_table), vis_c, Hkv,
                               gc.SM_SCALE, **kw)
        gc.check_attention(out[:, i].contiguous(), out32[:, i].contiguous(), ref)


@pytest.mark.parametrize("wide", [False, True])
def test_largest_batch(wide):
    """B = 4096 (the most the attention calls accept), ragged lengths 0..20, shuffled pages."""
    B, hkv, g = 4096, 8, 4
    kr, vr, km, vm = workloads.BUDGETS[2.26]
    lens = [int(x) for x in np.random.default_rng(B).integers(0, 21, size=B)]
    cfg = workloads.Config("largest_batch", B, hkv * g, hkv, lens, 99, kr, vr, km, vm, shuffle_pages=True,
                           v_student_t=False)
    w = workloads.generate(cfg, device="cuda")
    if wide:
        tk, tv, ok, ov = gc.wide_tables(cfg, hkv, k_rec=335, v_rec=235)
        cache = gc.WideGpuCache(w, tk, tv, hkv)
    else:
        tk, tv, ok, ov = gc.tables(cfg)
        cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    torch.cuda.synchronize()
    kc, vc, mq, ms, _, _ = gc.oracle_encode_wide(w, ok, ov, hkv) if wide else gc.oracle_encode(w, ok, ov)
    got_k, got_v = _np(cache.k_cont), _np(cache.v_cont)
    if wide:
        got_k, got_v = gc.from_interleaved(got_k, ok.rec), gc.from_interleaved(got_v, ov.rec)
    assert np.array_equal(got_k, kc) and np.array_equal(got_v, vc)
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), kc, vc, mq, ms, _np(w.page_table), _np(w.seq_lens), hkv,
                           gc.SM_SCALE)
    gc.check_attention(out, out32, ref)


@pytest.mark.parametrize("seed", range(16, 28))
def test_random_shape_through_the_batch_encoders(seed):
    """The same sweep with every encode call sent to the batch kernels (32 streams per CTA, one
    lane per stream in the rANS pass), which calls of this size would not reach on their own:
    ragged last CTAs, empty sequences, both stream groupings, every record against the oracle."""
    dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, 0)
    try:
        test_random_shape(seed)
    finally:
        dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, -1)


@pytest.mark.parametrize("seed", range(28, 44))
def test_random_shape_with_paired_symbols(seed):
    """The same sweep with the paired-symbol codec variant on both sides (the 4-bit budget's 16 key levels keep
    single levels); odd seeds through the batch encoders."""
    dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, 0 if seed % 2 else -1)
    try:
        test_random_shape(seed, pair=True)
    finally:
        dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, -1)

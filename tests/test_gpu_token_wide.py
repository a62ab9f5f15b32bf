"""GPU parity of the token-wide grouping (Sec. 5.1: each token is quantised as one group of
Hkv * 128 values; 331 / 231-byte containers, 8 / 6 levels): encoder and check decoder bit for
bit against the oracle, attention within 2e-3."""
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


def _cfg(idx, **over):
    cfg = workloads.make_config(idx, scale=1 / 16)
    for k, v in over.items():
        setattr(cfg, k, v)
    return cfg


CASES = {
    # name: (config, overrides, hs, (k_rec, v_rec, k_levels, v_levels))
    "paper_default": (2, dict(batch=3, seq_lens=[512, 300, 77]), 8, (335, 235, 8, 6)),
    "ragged_shuffled": (4, dict(batch=5, seq_lens=[200, 16, 333, 1, 1030]), 8, (335, 235, 8, 6)),
    "pairs_of_heads": (2, dict(batch=2, seq_lens=[130, 64]), 2, (86, 60, 6, 4)),
    "g7_four_heads": (5, dict(batch=2, seq_lens=[640, 129]), 4, (170, 120, 8, 6)),
    # the paired-symbol codec variant (a sixth field): one rANS symbol = the levels of two consecutive values
    "paper_default_pairs": (2, dict(batch=3, seq_lens=[512, 300, 77]), 8, (335, 235, 8, 6), True),
    "ragged_shuffled_pairs": (4, dict(batch=5, seq_lens=[200, 16, 333, 1, 1030]), 8, (335, 235, 8, 6), True),
    "pairs_of_heads_pairs": (2, dict(batch=2, seq_lens=[130, 64]), 2, (86, 60, 6, 4), True),
    "g7_four_heads_pairs": (5, dict(batch=2, seq_lens=[640, 129]), 4, (170, 120, 9, 5), True),
}


def _setup(name):
    idx, over, hs, (kr, vr, mk, mv) = CASES[name][:4]
    cfg = _cfg(idx, **over)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.wide_tables(cfg, hs, kr, vr, mk, mv, pair=len(CASES[name]) > 4)
    return cfg, w, hs, tk, tv, ok, ov


@pytest.mark.parametrize("name", list(CASES))
def test_encoder_records_and_means_bit_exact(name):
    cfg, w, hs, tk, tv, ok, ov = _setup(name)
    cache = gc.WideGpuCache(w, tk, tv, hs)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    kc, vc, mq, ms, sk, sv = gc.oracle_encode_wide(w, ok, ov, hs)
    assert np.array_equal(_np(cache.mean_q), mq)
    assert np.array_equal(_np(cache.mean_scale).view(np.uint32), ms.view(np.uint32))
    assert np.array_equal(gc.from_interleaved(_np(cache.k_cont), ok.rec), kc)
    assert np.array_equal(gc.from_interleaved(_np(cache.v_cont), ov.rec), vc)
    st = _np(cache.status)
    assert st[0] == sk[0] + sv[0] and st[1] == sk[1] + sv[1] and st[2] == sk[2] + sv[2]
    assert st[3] == max(sk[3], sv[3])


@pytest.mark.parametrize("name", list(CASES))
def test_decode_tokens_matches_oracle_bit_exact(name):
    cfg, w, hs, tk, tv, ok, ov = _setup(name)
    kc, vc, mq, ms, _, _ = gc.oracle_encode_wide(w, ok, ov, hs)
    seq_id, pos, slot = (_np(t) for t in (w.seq_id, w.pos, w.slot))
    for (t_lib, t_or, cont, m_q, m_s) in ((tk, ok, kc, mq, ms), (tv, ov, vc, None, None)):
        sym_ref, deq_ref = oracle.decode_tokens(t_or, cont, seq_id, pos, slot, cfg.hkv, m_q, m_s)
        sym = torch.zeros(sym_ref.shape, dtype=torch.uint8, device="cuda")
        deq = torch.zeros(deq_ref.shape, dtype=torch.float32, device="cuda")
        dq.dq_decode_tokens(t_lib, torch.from_numpy(gc.to_interleaved(cont)).cuda(), w.slot, cfg.hkv, sym, deq,
                            None if m_q is None else torch.from_numpy(m_q).cuda(),
                            None if m_s is None else torch.from_numpy(m_s).cuda(), w.seq_id, w.pos)
        torch.cuda.synchronize()
        assert np.array_equal(_np(sym), sym_ref)
        assert np.array_equal(_np(deq).view(np.uint32), deq_ref.view(np.uint32))


def test_encoder_degenerate_and_fallback_streams():
    """Constant tokens (s = 0), a token that is constant in all heads but one, and values that
    force the all-central fallback are handled as the oracle does."""
    cfg, w, hs, tk, tv, ok, ov = _setup("paper_default")
    w.k[0] = 0.0
    w.v[1] = 0.0
    w.k[2] = 0.0; w.k[2, 3, 17] = 4.0
    w.v[3, :, ::2] = 1000.0; w.v[3, :, 1::2] = -1000.0
    cache = gc.WideGpuCache(w, tk, tv, hs)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    kc, vc, mq, ms, sk, sv = gc.oracle_encode_wide(w, ok, ov, hs)
    assert np.array_equal(gc.from_interleaved(_np(cache.k_cont), ok.rec), kc)
    assert np.array_equal(gc.from_interleaved(_np(cache.v_cont), ov.rec), vc)
    st = _np(cache.status)
    assert st[1] == sk[1] + sv[1] >= 1 and st[0] == sk[0] + sv[0]


# --------------------------------------------------------------- attention

def _oracle_attention(w, ok, ov, kc, vc, mq, ms, seq_lens, **kw):
    return oracle.attention(ok, ov, workloads.bf16_bits(w.q), kc, vc, mq, ms, _np(w.page_table), _np(seq_lens),
                            w.cfg.hkv, gc.SM_SCALE, **kw)


@pytest.mark.parametrize("name", list(CASES))
def test_attention_matches_oracle(name):
    cfg, w, hs, tk, tv, ok, ov = _setup(name)
    cache = gc.WideGpuCache(w, tk, tv, hs)
    gc.gpu_encode(w, tk, tv, cache)
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    kc = gc.from_interleaved(_np(cache.k_cont), ok.rec)
    vc = gc.from_interleaved(_np(cache.v_cont), ov.rec)
    ref = _oracle_attention(w, ok, ov, kc, vc, _np(cache.mean_q), _np(cache.mean_scale), w.seq_lens)
    worst = gc.check_attention(out, out32, ref)
    assert worst < 2e-4
    out_b, out32_b = gc.gpu_attention(w, tk, tv, cache)
    assert torch.equal(out, out_b) and torch.equal(out32, out32_b)   # run-to-run identical


def test_attention_edge_lengths():
    """Empty sequences, single tokens, lengths around page / warp / item boundaries (items are
    15 warps x 32 tokens = 480 tokens at this shape)."""
    lens_all = [0, 1, 15, 16, 17, 31, 32, 33, 479, 480, 481, 600, 959, 960, 961]
    cfg = _cfg(4, batch=len(lens_all), seq_lens=[961] * len(lens_all))
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.wide_tables(cfg, 8)
    cache = gc.WideGpuCache(w, tk, tv, 8)
    gc.gpu_encode(w, tk, tv, cache)
    lens = torch.tensor(lens_all, dtype=torch.int32, device="cuda")
    out, out32 = gc.gpu_attention(w, tk, tv, cache, seq_lens=lens)
    kc = gc.from_interleaved(_np(cache.k_cont), ok.rec)
    vc = gc.from_interleaved(_np(cache.v_cont), ov.rec)
    ref = _oracle_attention(w, ok, ov, kc, vc, _np(cache.mean_q), _np(cache.mean_scale), lens)
    gc.check_attention(out, out32, ref)
    assert not out[0].any()


@pytest.mark.parametrize("name", ["paper_default", "paper_default_pairs"])
def test_lagging_streams_take_the_global_path(name):
    """Keys whose streams stop consuming bytes early (constant tokens between ordinary ones) fall
    far behind their warp's ring and must be served from global memory with the same result."""
    cfg, w, hs, tk, tv, ok, ov = _setup(name)
    w.k[5:400:7] = 0.0
    w.v[9:400:11] = 0.0
    cache = gc.WideGpuCache(w, tk, tv, hs)
    gc.gpu_encode(w, tk, tv, cache)
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    kc = gc.from_interleaved(_np(cache.k_cont), ok.rec)
    vc = gc.from_interleaved(_np(cache.v_cont), ov.rec)
    ref = _oracle_attention(w, ok, ov, kc, vc, _np(cache.mean_q), _np(cache.mean_scale), w.seq_lens)
    gc.check_attention(out, out32, ref)


def test_corrupted_records_stay_in_bounds():
    """Random bytes in place of records: the kernel must finish and write finite-or-not numbers
    without touching memory outside its buffers (states and pointers are data-dependent)."""
    cfg, w, hs, tk, tv, ok, ov = _setup("ragged_shuffled")
    cache = gc.WideGpuCache(w, tk, tv, hs)
    g = torch.Generator(device="cuda").manual_seed(5)
    cache.k_cont.copy_(torch.randint(0, 256, cache.k_cont.shape, generator=g, device="cuda", dtype=torch.uint8))
    cache.v_cont.copy_(torch.randint(0, 256, cache.v_cont.shape, generator=g, device="cuda", dtype=torch.uint8))
    canary = torch.full((1 << 20,), 0x5A, dtype=torch.uint8, device="cuda")
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    torch.cuda.synchronize()
    assert bool((canary == 0x5A).all())
    # and the library still works afterwards
    gc.gpu_encode(w, tk, tv, cache)
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    assert torch.isfinite(out32).all()


def test_paper_default_with_residual_window():
    """The paper's serving configuration: token-wide 331 / 231-byte containers, 8 / 6 levels, plus
    the most recent tokens in BF16."""
    cfg, w, hs, tk, tv, ok, ov = _setup("paper_default")
    cache = gc.WideGpuCache(w, tk, tv, hs)
    gc.gpu_encode(w, tk, tv, cache)
    gen = torch.Generator(device="cuda").manual_seed(11)
    rk, rv = workloads.make_kv(cfg, cfg.batch * 128, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
    rk = rk.view(cfg.batch, 128, cfg.hkv, 128).contiguous()
    rv = rv.view(cfg.batch, 128, cfg.hkv, 128).contiguous()
    rl = torch.tensor([128, 5, 77], dtype=torch.int32, device="cuda")
    out = torch.empty((cfg.batch, cfg.hq, 128), dtype=torch.bfloat16, device="cuda")
    out32 = torch.empty((cfg.batch, cfg.hq, 128), dtype=torch.float32, device="cuda")
    ws = torch.empty(dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, w.page_table.shape[1]), dtype=torch.uint8,
                     device="cuda")
    dq.dq_decode_attention_residual(tk, tv, w.q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale,
                                    w.page_table, w.seq_lens, rk, rv, rl, cfg.hkv, gc.SM_SCALE, out, ws, out32)
    torch.cuda.synchronize()
    kc = gc.from_interleaved(_np(cache.k_cont), ok.rec)
    vc = gc.from_interleaved(_np(cache.v_cont), ov.rec)
    ref = _oracle_attention(w, ok, ov, kc, vc, _np(cache.mean_q), _np(cache.mean_scale), w.seq_lens,
                            resid_k=workloads.bf16_bits(rk), resid_v=workloads.bf16_bits(rv), resid_lens=_np(rl))
    gc.check_attention(out, out32, ref)

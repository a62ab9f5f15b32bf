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
}


def _setup(name):
    idx, over, hs, (kr, vr, mk, mv) = CASES[name]
    cfg = _cfg(idx, **over)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.wide_tables(cfg, hs, kr, vr, mk, mv)
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

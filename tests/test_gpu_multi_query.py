"""GPU parity of attention with several query tokens per sequence (speculative decoding / short
prefill chunks): every query token's row must equal the oracle's single-query attention over
the prefix of the sequence that token may see."""
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


def _run(cfg, q_len, wide_hs=0, resid=None, seed=0, pair=False):
    w = workloads.generate(cfg, device="cuda")
    if wide_hs:
        tk, tv, ok, ov = gc.wide_tables(cfg, wide_hs)
        cache = gc.WideGpuCache(w, tk, tv, wide_hs)
    else:
        tk, tv, ok, ov = gc.tables(cfg, pair=pair)
        cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    B, Hq, Hkv = cfg.batch, cfg.hq, cfg.hkv
    gen = torch.Generator(device="cuda").manual_seed(100 + seed)
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
    kc, vc = _np(cache.k_cont), _np(cache.v_cont)
    if wide_hs:
        kc, vc = gc.from_interleaved(kc, ok.rec), gc.from_interleaved(vc, ov.rec)
    lens = _np(w.seq_lens).astype(np.int64)
    rlens = np.zeros(B, np.int64) if rl is None else _np(rl).astype(np.int64)
    worst = 0.0
    for i in range(q_len):
        off = q_len - 1 - i
        vis_r = np.maximum(0, rlens - off)
        vis_c = np.maximum(0, lens - np.maximum(0, off - rlens))
        kw = {}
        if rl is not None:
            kw = dict(resid_k=workloads.bf16_bits(rk), resid_v=workloads.bf16_bits(rv), resid_lens=vis_r.astype(np.int32))
        ref = oracle.attention(ok, ov, workloads.bf16_bits(q[:, i]), kc, vc, _np(cache.mean_q), _np(cache.mean_scale),
                               _np(w.page_table), vis_c.astype(np.int32), Hkv, gc.SM_SCALE, **kw)
        worst = max(worst, gc.check_attention(out[:, i].contiguous(), out32[:, i].contiguous(), ref))
    assert worst < 3e-4
    return w, tk, tv, cache, q, out, out32


def _cfg(idx, **over):
    cfg = workloads.make_config(idx, scale=1 / 16)
    for k, v in over.items():
        setattr(cfg, k, v)
    return cfg


@pytest.mark.parametrize("wide_hs", [0, 8])
def test_two_tokens_gqa4(wide_hs):
    """Llama-3-8B shape (4 query heads per KV head): 2 query tokens fill the 8 rows of a KV head."""
    cfg = _cfg(2, batch=4, seq_lens=[513, 300, 77, 2])
    _run(cfg, 2, wide_hs=wide_hs)


@pytest.mark.parametrize("q_len", [3, 8])
def test_many_tokens_mha(q_len):
    """One query head per KV head: up to 8 query tokens; a 5-token sequence sees fewer tokens than q_len
    for its oldest query tokens (their rows attend to nothing that does not exist)."""
    cfg = _cfg(2, batch=4, seq_lens=[700, 33, 9, 5], hq=8)
    _run(cfg, q_len, seed=q_len)


@pytest.mark.parametrize("wide_hs", [0, 8])
def test_with_residual_window_gqa2(wide_hs):
    """Newest tokens in the BF16 window: the causal offsets are taken from the window first, then
    from the compressed tokens (window shorter than q_len, empty window)."""
    cfg = _cfg(2, batch=4, seq_lens=[512, 130, 64, 1000], hq=16)
    _run(cfg, 4, wide_hs=wide_hs, resid=[128, 2, 0, 37])


def test_paired_symbols_with_window_and_several_tokens():
    """The paired-symbol codec variant through the same entry point: several query tokens and a BF16 window."""
    cfg = _cfg(2, batch=4, seq_lens=[512, 130, 64, 1000], hq=16)
    _run(cfg, 4, resid=[128, 2, 0, 37], pair=True)
    _run(_cfg(2, batch=4, seq_lens=[513, 300, 77, 2]), 2, pair=True)


def test_single_token_equals_plain_call():
    cfg = _cfg(4, batch=5, seq_lens=[200, 16, 333, 1, 1030])
    w, tk, tv, cache, q, out, out32 = _run(cfg, 1)
    w.q = q[:, 0].contiguous()
    out_p, out32_p = gc.gpu_attention(w, tk, tv, cache)
    assert torch.equal(out32[:, 0], out32_p) and torch.equal(out[:, 0], out_p)


def test_more_rows_than_one_pass_holds():
    """5 query tokens x 4 heads per KV head = 20 rows: three passes inside one call (2 + 2 + 1 tokens);
    and 11 tokens with one head per KV head (8 + 3), with a window."""
    cfg = _cfg(2, batch=3, seq_lens=[600, 64, 7])
    _run(cfg, 5, seed=21)
    cfg = _cfg(2, batch=2, seq_lens=[530, 40], hq=8)
    _run(cfg, 11, wide_hs=8, resid=[6, 128], seed=22)

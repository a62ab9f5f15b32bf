"""GPU parity of dq_decode_step (encode the newest token of every sequence and attend in one
overlapped launch sequence) against the two separate calls and against the oracle."""
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


def _loop(cfg, steps, seed, check_every=1, **table_kw):
    """Prefill `cfg.seq_lens` tokens, then `steps` decode steps through dq_decode_step on one cache and
    through dq_encode_tokens + dq_decode_attention on a second one; both must agree bit for bit at every
    step, and with the oracle's mirror of the loop."""
    w = workloads.generate(cfg, device="cuda", extra_tokens_per_seq=steps)
    tk, tv, ok, ov = gc.tables(cfg, **table_kw)   # table_kw: the opt-in codec variants
    ca, cb = gc.GpuCache(w, ok.rec, ov.rec), gc.GpuCache(w, ok.rec, ov.rec)
    B, Hq, Hkv = cfg.batch, cfg.hq, cfg.hkv
    if cfg.total_tokens:
        gc.gpu_encode(w, tk, tv, ca)
        gc.gpu_encode(w, tk, tv, cb)
    kc, vc, mq, ms, _, _ = gc.oracle_encode(w, ok, ov)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    lens = torch.tensor(cfg.seq_lens, dtype=torch.int32)
    grow = torch.tensor([1 if (l > 0 or b % 2 == 0) else 0 for b, l in enumerate(cfg.seq_lens)], dtype=torch.int32)
    pt_cpu = w.page_table.cpu()
    ws = torch.empty(dq.dq_decode_workspace_bytes(B, Hq, w.page_table.shape[1]), dtype=torch.uint8, device="cuda")
    ws.fill_(0xA5)     # the hand-over words start as garbage
    out_a = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device="cuda"); out32_a = torch.empty((B, Hq, 128), dtype=torch.float32, device="cuda")
    out_b = torch.empty_like(out_a); out32_b = torch.empty_like(out32_a)
    for s in range(steps):
        k1, v1 = workloads.make_kv(cfg, B, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
        q = torch.randn((B, Hq, 128), generator=gen, device="cuda").to(torch.bfloat16)
        lens = lens + grow                                   # sequences that stay empty never get a token
        pos = (lens - 1).clamp(min=0)
        slot = (pt_cpu[torch.arange(B), (pos // 16).long()] * 16 + pos % 16).to(torch.int32)
        lens_d = lens.cuda()
        dq.dq_decode_step(tk, tv, k1, v1, slot.cuda(), q, ca.k_cont, ca.v_cont, ca.mean_q, ca.mean_scale, w.page_table,
                          lens_d, Hkv, gc.SM_SCALE, out_a, ws, out32_a, ca.status)
        sel = torch.nonzero(lens > 0).flatten()
        seq = sel.to(torch.int32)
        dq.dq_encode_tokens(tk, tv, k1[sel.cuda()].contiguous(), v1[sel.cuda()].contiguous(), seq.cuda(),
                            pos[sel].to(torch.int32).cuda(), slot[sel].cuda(), cb.k_cont, cb.v_cont, cb.mean_q,
                            cb.mean_scale, dq.MEAN_REUSE, cb.status)
        dq.dq_decode_attention(tk, tv, q, cb.k_cont, cb.v_cont, cb.mean_q, cb.mean_scale, w.page_table, lens_d, Hkv,
                               gc.SM_SCALE, out_b, ws, out32_b)
        torch.cuda.synchronize()
        assert torch.equal(ca.k_cont, cb.k_cont) and torch.equal(ca.v_cont, cb.v_cont)
        assert torch.equal(ca.mean_q, cb.mean_q) and torch.equal(ca.mean_scale, cb.mean_scale)
        assert torch.equal(out32_a, out32_b) and torch.equal(out_a, out_b), s
        kb, vb = workloads.bf16_bits(k1[sel.cuda()]), workloads.bf16_bits(v1[sel.cuda()])
        sq, ps, sl = seq.numpy(), pos[sel].to(torch.int32).numpy(), slot[sel].numpy()
        oracle.window_means(kb, sq, ps, mq, ms, 1)
        oracle.encode_tokens(ok, kb, sq, ps, sl, kc, mq, ms)
        oracle.encode_tokens(ov, vb, sq, ps, sl, vc)
        if s % check_every == 0 or s == steps - 1:
            assert np.array_equal(_np(ca.k_cont), kc) and np.array_equal(_np(ca.v_cont), vc)
            ref = oracle.attention(ok, ov, workloads.bf16_bits(q), kc, vc, mq, ms, _np(w.page_table), _np(lens_d), Hkv,
                                   gc.SM_SCALE)
            gc.check_attention(out_a, out32_a, ref)
    return ca


def test_step_matches_separate_calls_and_oracle():
    """Lengths chosen so that the newest tokens open a window (pos % 128 == 0), open a 512-token block,
    open a page, and start sequences from nothing (window 0 gets a zero mean)."""
    cfg = _cfg(2, batch=6, seq_lens=[511, 127, 255, 0, 1023, 300])
    _loop(cfg, steps=4, seed=1)


def test_step_gqa7_ragged_shuffled_pages():
    cfg = _cfg(5, batch=3, seq_lens=[640, 129, 2000])
    cfg.shuffle_pages = True
    _loop(cfg, steps=3, seed=2)


def test_step_with_empty_and_idle_sequences():
    """Sequence 1 is empty and stays empty (no newest token, zero output row); sequence 2 starts at length 0."""
    cfg = _cfg(4, batch=4, seq_lens=[200, 0, 0, 77])
    ca = _loop(cfg, steps=3, seed=3)
    assert int(_np(ca.status)[0]) == 0


def test_step_many_steps_budget_3bits():
    cfg = workloads.make_config(3, budget=3.0, scale=1 / 64)      # 64 query / 8 kv heads
    cfg.batch = 2; cfg.seq_lens = [1500, 380]
    _loop(cfg, steps=20, seed=4, check_every=7)


@pytest.mark.parametrize("table_kw", [dict(pair=True), dict(pair=True, sigma=24, early_exit=True)])
def test_step_with_paired_symbols(table_kw):
    """The paired-symbol codec variant through the one-call step, the two-call sequence and the oracle's mirror:
    window, block and page openings, an empty sequence; 3-bit budget with 8 / 5 levels."""
    _loop(_cfg(2, batch=6, seq_lens=[511, 127, 255, 0, 1023, 300]), steps=4, seed=11, **table_kw)
    cfg = workloads.make_config(3, budget=3.0, scale=1 / 64)
    cfg.batch = 2; cfg.seq_lens = [1500, 380]
    _loop(cfg, steps=6, seed=12, check_every=3, **table_kw)


def test_step_when_the_ready_flag_is_never_seen():
    """Poll limit 0: every attention CTA gives up on the ready flag at once and takes the grid
    dependency wait instead; the step must still equal the two-call sequence and the oracle."""
    dq.dq_set_option(dq.OPT_STEP_POLL_LIMIT, 0)
    try:
        cfg = _cfg(2, batch=5, seq_lens=[511, 127, 0, 1023, 300])
        _loop(cfg, steps=3, seed=5)
    finally:
        dq.dq_set_option(dq.OPT_STEP_POLL_LIMIT, -1)

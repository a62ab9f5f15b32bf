"""Full-size GPU parity: the benchmark configurations at their real sizes, in the launch
configuration bench.py times.  EVERY record, window mean, decoded symbol, dequantised value and
attention row of configurations 2, 3 (all five budgets), 4 and 5 and of the token-wide
configurations 2 and 4 is compared with the oracle (the oracle does a whole configuration in
seconds on the host cores); the sampled checks remain for the decode-step variants."""
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


def _rec_view(cont):
    """[pages, Hkv, 16, rec] -> [slot, Hkv, rec] view on the host."""
    p, h, s, r = cont.shape
    return cont.transpose(0, 2, 1, 3).reshape(p * s, h, r)


def _host(cache):
    return dict(kc=_np(cache.k_cont), vc=_np(cache.v_cont), mq=_np(cache.mean_q), ms=_np(cache.mean_scale))


def _check_encoder_sample(w, ok, ov, host, rng, n_windows=6, groups=None):
    """Oracle re-encodes a few whole (sequence, window) runs (into compact containers of its
    own) and compares their records and window means with what the GPU wrote."""
    cfg = w.cfg
    groups = cfg.hkv if groups is None else groups     # streams per token
    seq_id, pos, slot = _np(w.seq_id), _np(w.pos), _np(w.slot)
    starts = np.concatenate([[0], np.cumsum(cfg.seq_lens)[:-1]])
    picked = set()
    for _ in range(n_windows):
        b = int(rng.integers(0, cfg.batch))
        nwin = (cfg.seq_lens[b] + 127) // 128
        picked.add((b, int(rng.choice([0, nwin - 1, int(rng.integers(0, nwin))]))))
    for (b, win) in sorted(picked):
        lo = int(starts[b]) + win * 128
        hi = int(starts[b]) + min(cfg.seq_lens[b], (win + 1) * 128)
        assert (seq_id[lo:hi] == b).all() and (pos[lo:hi] // 128 == win).all()
        kb, vb = workloads.bf16_bits(w.k[lo:hi]), workloads.bf16_bits(w.v[lo:hi])
        n = hi - lo
        compact = np.arange(n, dtype=np.int32)
        mq = np.zeros((cfg.batch, w.max_windows, cfg.hkv, 128), np.int8)
        ms = np.zeros((cfg.batch, w.max_windows, cfg.hkv), np.float32)
        oracle.window_means(kb, seq_id[lo:hi], pos[lo:hi], mq, ms, 0)
        kc = np.zeros(((n + 15) // 16, groups, 16, ok.rec), np.uint8)
        vc = np.zeros(((n + 15) // 16, groups, 16, ov.rec), np.uint8)
        oracle.encode_tokens(ok, kb, seq_id[lo:hi], pos[lo:hi], compact, kc, mq, ms)
        oracle.encode_tokens(ov, vb, seq_id[lo:hi], pos[lo:hi], compact, vc)
        sl = slot[lo:hi]
        assert np.array_equal(mq[b, win], host["mq"][b, win]) and np.array_equal(ms[b, win], host["ms"][b, win])
        assert np.array_equal(kc[compact // 16, :, compact % 16], host["kc"][sl // 16, :, sl % 16]), (b, win)
        assert np.array_equal(vc[compact // 16, :, compact % 16], host["vc"][sl // 16, :, sl % 16]), (b, win)


def _check_encoder_full(w, ok, ov, host, wide_hs=None):
    """The oracle encodes the whole workload; every container byte and every window mean must match."""
    if wide_hs is None:
        kc, vc, mq, ms, sk, sv = gc.oracle_encode(w, ok, ov)
    else:
        kc, vc, mq, ms, sk, sv = gc.oracle_encode_wide(w, ok, ov, wide_hs)
    assert np.array_equal(mq, host["mq"]) and np.array_equal(ms.view(np.uint32), host["ms"].view(np.uint32))
    assert np.array_equal(kc, host["kc"])
    assert np.array_equal(vc, host["vc"])
    assert sk[0] == 0 and sv[0] == 0


def _check_decoder_full(w, tk, tv, ok, ov, cache, host, chunk=16384):
    """Every token of the workload through dq_decode_tokens, in chunks: symbols and dequantised values bit for bit."""
    cfg = w.cfg
    for lo in range(0, cfg.total_tokens, chunk):
        hi = min(cfg.total_tokens, lo + chunk)
        seq_id, pos, slot = w.seq_id[lo:hi].contiguous(), w.pos[lo:hi].contiguous(), w.slot[lo:hi].contiguous()
        for (t_lib, t_or, cont_d, cont_h, m_q, m_s, mqd, msd) in (
                (tk, ok, cache.k_cont, host["kc"], host["mq"], host["ms"], cache.mean_q, cache.mean_scale),
                (tv, ov, cache.v_cont, host["vc"], None, None, None, None)):
            sym_ref, deq_ref = oracle.decode_tokens(t_or, cont_h, _np(seq_id), _np(pos), _np(slot), cfg.hkv, m_q, m_s)
            sym = torch.zeros(sym_ref.shape, dtype=torch.uint8, device="cuda")
            deq = torch.zeros(deq_ref.shape, dtype=torch.float32, device="cuda")
            dq.dq_decode_tokens(t_lib, cont_d, slot, cfg.hkv, sym, deq, mqd, msd, seq_id, pos)
            torch.cuda.synchronize()
            assert np.array_equal(_np(sym), sym_ref), lo
            assert np.array_equal(_np(deq).view(np.uint32), deq_ref.view(np.uint32)), lo


def _check_attention_full(w, tk, tv, ok, ov, cache, host, seq_lens=None):
    """Every (sequence, query head) row against the oracle's fp64 attention over the same containers."""
    cfg = w.cfg
    out, out32 = gc.gpu_attention(w, tk, tv, cache, seq_lens=seq_lens)
    assert torch.isfinite(out32).all()
    lens = _np(w.seq_lens if seq_lens is None else seq_lens)
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), host["kc"], host["vc"], host["mq"], host["ms"],
                           _np(w.page_table), lens, cfg.hkv, gc.SM_SCALE)
    worst = gc.check_attention(out, out32, ref)          # tolerance 2e-3 per row
    assert worst < 1e-3                                  # and, as a regression guard, well inside it
    return out, out32


def _check_decoder_sample(w, tk, tv, ok, ov, cache, host, rng, n_tokens=256):
    cfg = w.cfg
    idx = np.sort(rng.choice(cfg.total_tokens, size=min(n_tokens, cfg.total_tokens), replace=False))
    sel = torch.from_numpy(idx).to(w.k.device)
    seq_id, pos, slot = w.seq_id[sel].contiguous(), w.pos[sel].contiguous(), w.slot[sel].contiguous()
    kc, vc, mq, ms = host["kc"], host["vc"], host["mq"], host["ms"]
    for (t_lib, t_or, cont_d, cont_h, m_q, m_s, mqd, msd) in (
            (tk, ok, cache.k_cont, kc, mq, ms, cache.mean_q, cache.mean_scale),
            (tv, ov, cache.v_cont, vc, None, None, None, None)):
        sym_ref, deq_ref = oracle.decode_tokens(t_or, cont_h, _np(seq_id), _np(pos), _np(slot), cfg.hkv, m_q, m_s)
        sym = torch.zeros(sym_ref.shape, dtype=torch.uint8, device="cuda")
        deq = torch.zeros(deq_ref.shape, dtype=torch.float32, device="cuda")
        dq.dq_decode_tokens(t_lib, cont_d, slot, cfg.hkv, sym, deq, mqd, msd, seq_id, pos)
        torch.cuda.synchronize()
        assert np.array_equal(_np(sym), sym_ref)
        assert np.array_equal(_np(deq).view(np.uint32), deq_ref.view(np.uint32))


def _check_attention_sample(w, tk, tv, ok, ov, cache, host, rng, rows=3, seq_lens=None):
    cfg = w.cfg
    out, out32 = gc.gpu_attention(w, tk, tv, cache, seq_lens=seq_lens)
    assert torch.isfinite(out32).all()
    lens = _np(w.seq_lens if seq_lens is None else seq_lens)
    kc, vc, mq, ms = host["kc"], host["vc"], host["mq"], host["ms"]
    qb, pt = workloads.bf16_bits(w.q), _np(w.page_table)
    ref = np.full((cfg.batch, cfg.hq, 128), np.nan)
    picked = []
    order = np.argsort(lens)
    cand_b = [int(order[0]), int(order[-1])] + [int(rng.integers(0, cfg.batch)) for _ in range(rows)]
    for b in cand_b[:rows]:
        hq = int(rng.integers(0, cfg.hq))
        r = oracle.attention(ok, ov, qb, kc, vc, mq, ms, pt, lens, cfg.hkv, gc.SM_SCALE, only=(b, hq))
        ref[b, hq] = r[b, hq]
        picked.append((b, hq))
    worst = gc.check_attention(out, out32, ref, rows=picked)
    assert worst < 5e-4
    return out32


def _run_config(cfg, seed, exhaustive=False, windows=6, all_rows=False):
    rng = np.random.default_rng(seed)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    st = _np(cache.status)
    assert st[0] == 0 and st[3] <= max(ok.rec, ov.rec)     # every stream fits; no all-central fallback
    host = _host(cache)
    if exhaustive:
        _check_encoder_full(w, ok, ov, host)
        _check_decoder_full(w, tk, tv, ok, ov, cache, host)
    else:
        _check_encoder_sample(w, ok, ov, host, rng, n_windows=windows)
        _check_decoder_sample(w, tk, tv, ok, ov, cache, host, rng)
    if exhaustive or all_rows:
        _check_attention_full(w, tk, tv, ok, ov, cache, host)
    else:
        _check_attention_sample(w, tk, tv, ok, ov, cache, host, rng)
    return w, tk, tv, ok, ov, cache


def test_config2_llama3_8b_full():
    """Every record, mean, symbol, dequantised value and attention row of configuration 2."""
    cfg = workloads.make_config(2)
    assert cfg.total_tokens * cfg.hkv == 524288
    _run_config(cfg, 2, exhaustive=True)


@pytest.mark.parametrize("budget", [1.5, 2.0, 2.26, 3.0, 4.0])
def test_config3_long_context_budget_sweep_full(budget):
    """Every budget of the sweep exhaustively (1 048 576 token-heads each)."""
    cfg = workloads.make_config(3, budget=budget)
    assert cfg.seq_lens == [131072] and cfg.hq // cfg.hkv == 8
    _run_config(cfg, 30 + int(budget * 10), exhaustive=True)


def test_config4_ragged_paged_full():
    """Every record, mean, symbol, dequantised value and attention row of the 128 ragged sequences
    (8.65 M token-heads, shuffled pages)."""
    cfg = workloads.make_config(4)
    assert cfg.batch == 128 and cfg.shuffle_pages
    w, tk, tv, ok, ov, cache = _run_config(cfg, 4, exhaustive=True)
    pt = _np(w.page_table)
    assert not np.array_equal(pt[0, :8], np.sort(pt[0, :8]))     # pages really are shuffled


def test_config5_encode_decode_loop_full():
    """Prefill-encode 4 x 32768 tokens (every record and mean against the oracle), then 256 decode
    steps, each appending one freshly encoded token per sequence (means carried forward) before
    attention; the oracle mirrors the loop for all four sequences: every appended record, every
    touched window mean, every attention row of the last step."""
    cfg = workloads.make_config(5)
    steps = cfg.decode_steps
    assert steps == 256 and cfg.hq // cfg.hkv == 7
    w = workloads.generate(cfg, device="cuda", extra_tokens_per_seq=steps)
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    kc_o, vc_o, mq_o, ms_o, sk, sv = gc.oracle_encode(w, ok, ov)
    host = _host(cache)
    assert np.array_equal(kc_o, host["kc"]) and np.array_equal(vc_o, host["vc"])
    assert np.array_equal(mq_o, host["mq"]) and np.array_equal(ms_o.view(np.uint32), host["ms"].view(np.uint32))
    _check_decoder_full(w, tk, tv, ok, ov, cache, host)

    gen = torch.Generator(device="cuda").manual_seed(55)
    lens = torch.tensor(cfg.seq_lens)
    seq = torch.arange(cfg.batch, dtype=torch.int32)
    pt_cpu = w.page_table.cpu()
    out = torch.empty((cfg.batch, cfg.hq, 128), dtype=torch.bfloat16, device="cuda")
    out32 = torch.empty((cfg.batch, cfg.hq, 128), dtype=torch.float32, device="cuda")
    ws = torch.empty(dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, w.page_table.shape[1]), dtype=torch.uint8,
                     device="cuda")
    new_slots = []
    for s in range(steps):
        k1, v1 = workloads.make_kv(cfg, cfg.batch, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
        pos = (lens + s).to(torch.int32)
        slot = (pt_cpu[seq.long(), (pos // 16).long()] * 16 + pos % 16).to(torch.int32)
        dq.dq_encode_tokens(tk, tv, k1, v1, seq.cuda(), pos.cuda(), slot.cuda(), cache.k_cont, cache.v_cont,
                            cache.mean_q, cache.mean_scale, dq.MEAN_REUSE, cache.status)
        cur = (lens + s + 1).to(torch.int32).cuda()
        dq.dq_decode_attention(tk, tv, w.q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale,
                               w.page_table, cur, cfg.hkv, gc.SM_SCALE, out, ws, out32)
        kb, vb = workloads.bf16_bits(k1), workloads.bf16_bits(v1)
        sid, ps, sl = seq.numpy(), pos.numpy(), slot.numpy()
        oracle.window_means(kb, sid, ps, mq_o, ms_o, 1)
        oracle.encode_tokens(ok, kb, sid, ps, sl, kc_o, mq_o, ms_o)
        oracle.encode_tokens(ov, vb, sid, ps, sl, vc_o)
        new_slots.extend(int(x) for x in sl)
    torch.cuda.synchronize()
    assert int(_np(cache.status)[0]) == 0
    new_slots = np.array(new_slots)
    host = _host(cache)
    assert np.array_equal(_rec_view(host["kc"])[new_slots], _rec_view(kc_o)[new_slots])
    assert np.array_equal(_rec_view(host["vc"])[new_slots], _rec_view(vc_o)[new_slots])
    assert np.array_equal(host["kc"], kc_o) and np.array_equal(host["vc"], vc_o)      # and nothing else moved
    assert np.array_equal(host["mq"], mq_o) and np.array_equal(host["ms"].view(np.uint32), ms_o.view(np.uint32))
    # attention of the last step, every row, against the oracle over the grown cache
    final = (lens + steps).to(torch.int32).cuda()
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), host["kc"], host["vc"], host["mq"], host["ms"],
                           _np(w.page_table), _np(final), cfg.hkv, gc.SM_SCALE)
    gc.check_attention(out, out32, ref)     # the loop's own last output
    _check_attention_full(w, tk, tv, ok, ov, cache, host, seq_lens=final)


# ------------------------------------------------ token-wide streams at full size

def _run_config_wide(cfg, seed, hs=8, exhaustive=False, windows=4, all_rows=False):
    """The paper's default grouping (one 335 / 235-byte record per token, 8 / 6 levels) on a full
    benchmark shape: same checks, containers compared after undoing the page interleave."""
    rng = np.random.default_rng(seed)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.wide_tables(cfg, hs)
    cache = gc.WideGpuCache(w, tk, tv, hs)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    st = _np(cache.status)
    assert st[0] == 0 and st[3] <= max(ok.rec, ov.rec)
    host = dict(kc=gc.from_interleaved(_np(cache.k_cont), ok.rec), vc=gc.from_interleaved(_np(cache.v_cont), ov.rec),
                mq=_np(cache.mean_q), ms=_np(cache.mean_scale))
    if exhaustive:
        _check_encoder_full(w, ok, ov, host, wide_hs=hs)
        _check_decoder_full(w, tk, tv, ok, ov, cache, host)
    else:
        _check_encoder_sample(w, ok, ov, host, rng, n_windows=windows, groups=cfg.hkv // hs)
        _check_decoder_sample(w, tk, tv, ok, ov, cache, host, rng, n_tokens=128)
    if exhaustive or all_rows:
        _check_attention_full(w, tk, tv, ok, ov, cache, host)
    else:
        _check_attention_sample(w, tk, tv, ok, ov, cache, host, rng)
    return w, tk, tv, ok, ov, cache


def test_config2_token_wide_full():
    """Every record, mean, symbol, dequantised value and attention row of the token-wide configuration 2."""
    cfg = workloads.make_config(2)
    assert cfg.total_tokens == 65536 and cfg.hkv == 8
    _run_config_wide(cfg, 12, exhaustive=True)


def test_config4_ragged_paged_token_wide_full():
    cfg = workloads.make_config(4)
    assert cfg.batch == 128 and cfg.shuffle_pages
    _run_config_wide(cfg, 14, exhaustive=True)


def _step_vs_two_calls(cfg, steps, seed):
    """`steps` decode steps through dq_decode_step on one cache and through dq_encode_tokens +
    dq_decode_attention on a copy: bit-identical every 8th and the last step; sampled rows of the last
    step against the oracle."""
    rng = np.random.default_rng(seed)
    w = workloads.generate(cfg, device="cuda", extra_tokens_per_seq=steps)
    tk, tv, ok, ov = gc.tables(cfg)
    ca, cb = gc.GpuCache(w, ok.rec, ov.rec), gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, ca)
    for name in ("k_cont", "v_cont", "mean_q", "mean_scale"):
        getattr(cb, name).copy_(getattr(ca, name))
    B, Hq, Hkv = cfg.batch, cfg.hq, cfg.hkv
    gen = torch.Generator(device="cuda").manual_seed(seed + 1)
    lens = torch.tensor(cfg.seq_lens, dtype=torch.int32)
    seq = torch.arange(B, dtype=torch.int32).cuda()
    pt_cpu = w.page_table.cpu()
    ws = torch.empty(dq.dq_decode_workspace_bytes(B, Hq, w.page_table.shape[1]), dtype=torch.uint8, device="cuda")
    out_a = torch.empty((B, Hq, 128), dtype=torch.bfloat16, device="cuda"); out32_a = torch.empty((B, Hq, 128), dtype=torch.float32, device="cuda")
    out_b = torch.empty_like(out_a); out32_b = torch.empty_like(out32_a)
    for s in range(steps):
        k1, v1 = workloads.make_kv(cfg, B, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
        lens = lens + 1
        pos = lens - 1
        slot = (pt_cpu[torch.arange(B), (pos // 16).long()] * 16 + pos % 16).to(torch.int32).cuda()
        lens_d = lens.cuda()
        dq.dq_decode_step(tk, tv, k1, v1, slot, w.q, ca.k_cont, ca.v_cont, ca.mean_q, ca.mean_scale, w.page_table, lens_d,
                          Hkv, gc.SM_SCALE, out_a, ws, out32_a, ca.status)
        dq.dq_encode_tokens(tk, tv, k1, v1, seq, pos.cuda(), slot, cb.k_cont, cb.v_cont, cb.mean_q, cb.mean_scale,
                            dq.MEAN_REUSE, cb.status)
        dq.dq_decode_attention(tk, tv, w.q, cb.k_cont, cb.v_cont, cb.mean_q, cb.mean_scale, w.page_table, lens_d, Hkv,
                               gc.SM_SCALE, out_b, ws, out32_b)
        if s % 8 == 7 or s == steps - 1:
            torch.cuda.synchronize()
            assert torch.equal(out32_a, out32_b) and torch.equal(out_a, out_b), s
    torch.cuda.synchronize()
    assert torch.equal(ca.k_cont, cb.k_cont) and torch.equal(ca.v_cont, cb.v_cont) and torch.equal(ca.mean_q, cb.mean_q)
    _check_attention_sample(w, tk, tv, ok, ov, ca, _host(ca), rng, rows=2, seq_lens=lens.cuda())


def test_config5_decode_step_full():
    """Config 5 at full size through dq_decode_step: few work items, so the attention kernel starts
    beside the encoder (ready flag, dynamic item order, late dependency wait)."""
    _step_vs_two_calls(workloads.make_config(5), steps=64, seed=55)


def test_config4_decode_step_full():
    """Config 4 at full size through dq_decode_step: far more work items than the overlapped schedule
    takes (B * blocks * Hkv > 32 per SM), so the call runs the plain kernel sequence."""
    cfg = workloads.make_config(4)
    assert sum((l + 511) // 512 for l in cfg.seq_lens) * cfg.hkv > 32 * 148
    _step_vs_two_calls(cfg, steps=3, seed=44)


def test_bf16_baseline_config2_full():
    """The bf16-cache comparison kernel at the benchmark's size (splits of several 32-token chunks per warp,
    online softmax across them) against a binary32 torch reference."""
    cfg = workloads.make_config(2)
    w = workloads.generate(cfg, device="cuda")
    kp = torch.zeros((w.num_pages * 16, cfg.hkv, 128), dtype=torch.bfloat16, device="cuda")
    vp = torch.zeros_like(kp)
    kp[w.slot.long()] = w.k
    vp[w.slot.long()] = w.v
    kp = kp.view(w.num_pages, 16, cfg.hkv, 128).transpose(1, 2).contiguous()
    vp = vp.view(w.num_pages, 16, cfg.hkv, 128).transpose(1, 2).contiguous()
    out = torch.empty((cfg.batch, cfg.hq, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, w.page_table.shape[1]), dtype=torch.uint8, device="cuda")
    dq.dq_bf16_decode_attention(w.q, kp, vp, w.page_table, w.seq_lens, cfg.hkv, gc.SM_SCALE, out, ws)
    torch.cuda.synchronize()
    start = 0
    for b, n in enumerate(cfg.seq_lens):
        k = w.k[start:start + n].float().repeat_interleave(cfg.hq // cfg.hkv, dim=1)
        v = w.v[start:start + n].float().repeat_interleave(cfg.hq // cfg.hkv, dim=1)
        a = torch.softmax(gc.SM_SCALE * torch.einsum("hd,thd->ht", w.q[b].float(), k), -1)
        ref = torch.einsum("ht,thd->hd", a, v)
        assert (out[b].float() - ref).abs().max() <= 6e-3 * ref.abs().max()
        start += n

"""GPU parity tests: the CUDA path (through the C ABI) against the CPU oracle on the same
seeded inputs.  Containers, window means, decoded symbols and dequantised values must match
bit for bit; attention must agree with the oracle's fp64 attention within 2e-3 of the
vector's largest magnitude."""
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


def _small(idx, **over):
    cfg = workloads.make_config(idx, scale=over.pop("scale", 1 / 16))
    for k, v in over.items():
        setattr(cfg, k, v)
    return cfg


SMALL = {
    "c1_full": lambda: workloads.make_config(1),
    "c2_small": lambda: _small(2, batch=3, seq_lens=[512, 300, 77]),
    "c3_small_g8": lambda: _small(3, seq_lens=[1999]),
    "c4_ragged": lambda: _small(4, batch=5, seq_lens=[200, 16, 333, 1, 1030]),
    "c5_small_g7": lambda: _small(5, batch=2, seq_lens=[640, 129]),
}


# ----------------------------------------------------------------- decoder

@pytest.mark.parametrize("name", list(SMALL))
def test_decode_tokens_matches_oracle_bit_exact(name):
    """Oracle-written containers -> dq_decode_tokens: symbols and dequantised values."""
    cfg = SMALL[name]()
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    kc, vc, mq, ms, _, _ = gc.oracle_encode(w, ok, ov)
    seq_id, pos, slot = (_np(t) for t in (w.seq_id, w.pos, w.slot))
    for (t_lib, t_or, cont, m_q, m_s) in ((tk, ok, kc, mq, ms), (tv, ov, vc, None, None)):
        sym_ref, deq_ref = oracle.decode_tokens(t_or, cont, seq_id, pos, slot, cfg.hkv, m_q, m_s)
        sym = torch.zeros(sym_ref.shape, dtype=torch.uint8, device="cuda")
        deq = torch.zeros(deq_ref.shape, dtype=torch.float32, device="cuda")
        dq.dq_decode_tokens(t_lib, torch.from_numpy(cont).cuda(), w.slot, cfg.hkv, sym, deq,
                            None if m_q is None else torch.from_numpy(m_q).cuda(),
                            None if m_s is None else torch.from_numpy(m_s).cuda(), w.seq_id, w.pos)
        torch.cuda.synchronize()
        assert np.array_equal(_np(sym), sym_ref)
        assert np.array_equal(_np(deq).view(np.uint32), deq_ref.view(np.uint32))


# ----------------------------------------------------------------- encoder

@pytest.mark.parametrize("name", list(SMALL))
def test_encoder_containers_and_means_bit_exact(name):
    cfg = SMALL[name]()
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    kc, vc, mq, ms, sk, sv = gc.oracle_encode(w, ok, ov)
    assert np.array_equal(_np(cache.mean_q), mq)
    assert np.array_equal(_np(cache.mean_scale).view(np.uint32), ms.view(np.uint32))
    assert np.array_equal(_np(cache.k_cont), kc)
    assert np.array_equal(_np(cache.v_cont), vc)
    st = _np(cache.status)
    assert list(st[:3]) == [sk[0] + sv[0], sk[1] + sv[1], sk[2] + sv[2]] and st[3] == max(sk[3], sv[3])
    # deterministic: a second run writes the same bytes
    cache2 = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache2)
    torch.cuda.synchronize()
    assert torch.equal(cache.k_cont, cache2.k_cont) and torch.equal(cache.v_cont, cache2.v_cont)


def test_encoder_degenerate_streams_and_v_without_rotation():
    cfg = _small(2, batch=1, seq_lens=[160])
    w = workloads.generate(cfg, device="cuda")
    w.v[7] = 1.5                       # constant streams (V is not rotated here): min == max
    w.v[9] = 0.0
    tk, tv, ok, ov = gc.tables(cfg, rotate_v=False)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    kc, vc, mq, ms, sk, sv = gc.oracle_encode(w, ok, ov)
    assert sv[1] >= 2 * cfg.hkv        # the constant V streams took the degenerate path
    assert np.array_equal(_np(cache.k_cont), kc) and np.array_equal(_np(cache.v_cont), vc)
    assert np.array_equal(_np(cache.mean_q), mq)
    assert list(_np(cache.status)[:3]) == [sk[0] + sv[0], sk[1] + sv[1], sk[2] + sv[2]]


def test_encoder_append_with_mean_reuse():
    """Prefill with computed means, then tokens appended one per sequence with DQ_MEAN_REUSE,
    crossing a window boundary (the carry-forward rule)."""
    cfg = _small(5, batch=3, seq_lens=[250, 128, 381])
    steps = 12
    w = workloads.generate(cfg, device="cuda", extra_tokens_per_seq=steps)
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    kc, vc, mq, ms, _, _ = gc.oracle_encode(w, ok, ov)
    gen = torch.Generator(device="cuda").manual_seed(99)
    lens = torch.tensor(cfg.seq_lens)
    for s in range(steps):
        k1, v1 = workloads.make_kv(cfg, cfg.batch, gen, torch.device("cuda"), w.k_offsets, w.k_gain)
        pos = (lens + s).to(torch.int32)
        seq = torch.arange(cfg.batch, dtype=torch.int32)
        slot = (w.page_table.cpu()[seq.long(), (pos // 16).long()] * 16 + pos % 16).to(torch.int32)
        dq.dq_encode_tokens(tk, tv, k1, v1, seq.cuda(), pos.cuda(), slot.cuda(), cache.k_cont, cache.v_cont,
                            cache.mean_q, cache.mean_scale, dq.MEAN_REUSE, cache.status)
        kb, vb = workloads.bf16_bits(k1), workloads.bf16_bits(v1)
        oracle.window_means(kb, seq.numpy(), pos.numpy(), mq, ms, 1)
        oracle.encode_tokens(ok, kb, seq.numpy(), pos.numpy(), slot.numpy(), kc, mq, ms)
        oracle.encode_tokens(ov, vb, seq.numpy(), pos.numpy(), slot.numpy(), vc)
    torch.cuda.synchronize()
    assert np.array_equal(_np(cache.mean_q), mq) and np.array_equal(_np(cache.mean_scale), ms)
    assert np.array_equal(_np(cache.k_cont), kc) and np.array_equal(_np(cache.v_cont), vc)
    # attention over the grown cache
    w.seq_lens = (lens + steps).to(torch.int32).cuda()
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), kc, vc, mq, ms, _np(w.page_table), _np(w.seq_lens),
                           cfg.hkv, gc.SM_SCALE)
    gc.check_attention(out, out32, ref)


# --------------------------------------------------------------- attention

@pytest.mark.parametrize("name", list(SMALL))
def test_attention_matches_oracle(name):
    cfg = SMALL[name]()
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), _np(cache.k_cont), _np(cache.v_cont),
                           _np(cache.mean_q), _np(cache.mean_scale), _np(w.page_table), _np(w.seq_lens),
                           cfg.hkv, gc.SM_SCALE)
    worst = gc.check_attention(out, out32, ref)
    assert worst < 2e-4                 # fp32 accumulation leaves a wide margin
    out_b, out32_b = gc.gpu_attention(w, tk, tv, cache)
    assert torch.equal(out, out_b) and torch.equal(out32, out32_b)   # run-to-run identical


def test_attention_edge_lengths():
    """Empty sequences, single tokens, lengths around page / chunk / item boundaries."""
    cfg = _small(4, batch=12, seq_lens=[600] * 12)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    lens = torch.tensor([0, 1, 15, 16, 17, 31, 32, 33, 511, 512, 513, 600], dtype=torch.int32, device="cuda")
    out, out32 = gc.gpu_attention(w, tk, tv, cache, seq_lens=lens)
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), _np(cache.k_cont), _np(cache.v_cont),
                           _np(cache.mean_q), _np(cache.mean_scale), _np(w.page_table), _np(lens), cfg.hkv,
                           gc.SM_SCALE)
    gc.check_attention(out, out32, ref)
    assert not out[0].any()


@pytest.mark.parametrize("budget", [1.5, 2.0, 2.26, 3.0, 4.0])
def test_budget_sweep_small(budget):
    cfg = workloads.make_config(3, budget=budget, scale=1 / 64)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    kc, vc, mq, ms, _, _ = gc.oracle_encode(w, ok, ov)
    assert np.array_equal(_np(cache.k_cont), kc) and np.array_equal(_np(cache.v_cont), vc)
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    ref = oracle.attention(ok, ov, workloads.bf16_bits(w.q), kc, vc, mq, ms, _np(w.page_table), _np(w.seq_lens),
                           cfg.hkv, gc.SM_SCALE)
    gc.check_attention(out, out32, ref)


def test_corrupted_records_stay_in_bounds():
    """Random bytes in place of records: outputs may be meaningless but the call completes and
    later calls still work (no out-of-bounds access, no trap)."""
    cfg = _small(2, batch=2, seq_lens=[700, 90])
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    g = torch.Generator(device="cuda").manual_seed(5)
    cache.k_cont.copy_(torch.randint(0, 256, cache.k_cont.shape, generator=g, device="cuda", dtype=torch.uint8))
    cache.v_cont.copy_(torch.randint(0, 256, cache.v_cont.shape, generator=g, device="cuda", dtype=torch.uint8))
    gc.gpu_attention(w, tk, tv, cache)
    sym = torch.zeros((cfg.total_tokens, cfg.hkv, 128), dtype=torch.uint8, device="cuda")
    dq.dq_decode_tokens(tk, cache.k_cont, w.slot, cfg.hkv, sym)
    torch.cuda.synchronize()
    sym_ref, _ = oracle.decode_tokens(ok, _np(cache.k_cont), _np(w.seq_id), _np(w.pos), _np(w.slot), cfg.hkv,
                                      want_dequant=False)
    assert np.array_equal(_np(sym), sym_ref)
    gc.gpu_encode(w, tk, tv, cache)
    out, out32 = gc.gpu_attention(w, tk, tv, cache)
    assert torch.isfinite(out32).all()


def test_bf16_baseline_against_torch():
    cfg = _small(4, batch=4, seq_lens=[200, 16, 333, 1030])
    w = workloads.generate(cfg, device="cuda")
    kp = torch.zeros((w.num_pages * 16, cfg.hkv, 128), dtype=torch.bfloat16, device="cuda")
    vp = torch.zeros_like(kp)
    kp[w.slot.long()] = w.k
    vp[w.slot.long()] = w.v
    kp = kp.view(w.num_pages, 16, cfg.hkv, 128).transpose(1, 2).contiguous()
    vp = vp.view(w.num_pages, 16, cfg.hkv, 128).transpose(1, 2).contiguous()
    out = torch.empty((cfg.batch, cfg.hq, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, w.page_table.shape[1]), dtype=torch.uint8,
                     device="cuda")
    dq.dq_bf16_decode_attention(w.q, kp, vp, w.page_table, w.seq_lens, cfg.hkv, gc.SM_SCALE, out, ws)
    torch.cuda.synchronize()
    start = 0
    for b, n in enumerate(cfg.seq_lens):
        k = w.k[start:start + n].float().repeat_interleave(cfg.hq // cfg.hkv, dim=1)
        v = w.v[start:start + n].float().repeat_interleave(cfg.hq // cfg.hkv, dim=1)
        a = torch.softmax(gc.SM_SCALE * torch.einsum("hd,thd->ht", w.q[b].float(), k), -1)
        ref = torch.einsum("ht,thd->hd", a, v)
        # bf16 softmax weights and a bf16 result: a few half-ulps of 2^-9 against the fp32 reference
        assert (out[b].float() - ref).abs().max() <= 6e-3 * ref.abs().max()
        start += n


@pytest.mark.parametrize("wide", [False, True])
def test_encoder_extreme_finite_values(wide):
    """The largest bf16 magnitudes (squares overflow: every candidate cost is infinite), subnormals
    and negative zero: records, means and status counters as the oracle's."""
    cfg = _small(2, batch=1, seq_lens=[48])
    w = workloads.generate(cfg, device="cuda")
    big = 3.38e38
    w.v[3, 0, 5] = big; w.v[4, 1, :] = big; w.v[5, 2, ::2] = big; w.v[5, 2, 1::2] = -big
    w.k[6, 0, 7] = big; w.k[7, 3, 1] = -big
    w.v[13] = 1e-40; w.v[13, 0, 5] = 3e-40; w.v[14] = -0.0; w.k[16] = 1e-39; w.k[16, 1, 3] = 2e-39
    if wide:
        tk, tv, ok, ov = gc.wide_tables(cfg, cfg.hkv, k_rec=335, v_rec=235)
        cache = gc.WideGpuCache(w, tk, tv, cfg.hkv)
    else:
        tk, tv, ok, ov = gc.tables(cfg)
        cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    torch.cuda.synchronize()
    kc, vc, mq, ms, sk, sv = gc.oracle_encode_wide(w, ok, ov, cfg.hkv) if wide else gc.oracle_encode(w, ok, ov)
    got_k, got_v = _np(cache.k_cont), _np(cache.v_cont)
    if wide:
        got_k, got_v = gc.from_interleaved(got_k, ok.rec), gc.from_interleaved(got_v, ov.rec)
    assert np.array_equal(got_k, kc) and np.array_equal(got_v, vc)
    assert np.array_equal(_np(cache.mean_q), mq) and np.array_equal(_np(cache.mean_scale), ms)
    assert list(_np(cache.status)[:3]) == [sk[i] + sv[i] for i in range(3)]
    assert sk[0] + sv[0] > 0 and sk[1] + sv[1] > 0      # both the fallback and the constant path were taken


def test_decode_loop_microbenchmark_runs():
    """The bare decode-loop measurement aid: launches for both chain counts, fills every thread's checksum slot,
    is deterministic, and refuses shapes it cannot run."""
    tk = dq.dq_build_tables(5, 42 * 8 / 128, has_mean=True)
    g = torch.Generator(device="cpu").manual_seed(3)
    data = torch.randint(0, 256, (1 << 16,), dtype=torch.uint8, generator=g).cuda()
    for threads, chains in ((512, 2), (1024, 1), (64, 2)):
        a = torch.zeros(4 * threads, dtype=torch.int32, device="cuda")
        b = torch.zeros_like(a)
        dq.dq_microbench_decode_loop(tk, data, 4, threads, chains, 3, a)
        dq.dq_microbench_decode_loop(tk, data, 4, threads, chains, 3, b)
        torch.cuda.synchronize()
        assert torch.equal(a, b) and int((a != 0).sum()) > a.numel() // 2
    out = torch.zeros(1024, dtype=torch.int32, device="cuda")
    for bad in (dict(threads=48), dict(threads=2048), dict(chains=3), dict(reps=0), dict(ctas=0)):
        kw = dict(ctas=1, threads=256, chains=1, reps=1); kw.update(bad)
        with pytest.raises(dq.DqError):
            dq.dq_microbench_decode_loop(tk, data, kw["ctas"], kw["threads"], kw["chains"], kw["reps"], out)


@pytest.mark.parametrize("lens", [[0, 0, 1], [1, 0, 17, 16, 33], [5] * 300, [2047, 1, 0, 129, 640]])
def test_bf16_baseline_edge_shapes(lens):
    """Empty batches, empty and one-token sequences, hundreds of tiny sequences, ragged lengths: the split sizing on
    the device, ranges that end inside a chunk, zero rows for empty sequences."""
    cfg = _small(4, batch=len(lens), seq_lens=lens)
    w = workloads.generate(cfg, device="cuda")
    kp = torch.zeros((max(w.num_pages, 1) * 16, cfg.hkv, 128), dtype=torch.bfloat16, device="cuda")
    vp = torch.zeros_like(kp)
    if cfg.total_tokens:
        kp[w.slot.long()] = w.k
        vp[w.slot.long()] = w.v
    kp = kp.view(-1, 16, cfg.hkv, 128).transpose(1, 2).contiguous()
    vp = vp.view(-1, 16, cfg.hkv, 128).transpose(1, 2).contiguous()
    out = torch.full((cfg.batch, cfg.hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, w.page_table.shape[1]), dtype=torch.uint8,
                     device="cuda")
    for _ in range(2):   # twice: nothing of the first call may linger in the workspace
        dq.dq_bf16_decode_attention(w.q, kp, vp, w.page_table, w.seq_lens, cfg.hkv, gc.SM_SCALE, out, ws)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    start = 0
    for b, n in enumerate(cfg.seq_lens):
        if n == 0:
            assert not out[b].any()
            continue
        k = w.k[start:start + n].float().repeat_interleave(cfg.hq // cfg.hkv, dim=1)
        v = w.v[start:start + n].float().repeat_interleave(cfg.hq // cfg.hkv, dim=1)
        a = torch.softmax(gc.SM_SCALE * torch.einsum("hd,thd->ht", w.q[b].float(), k), -1)
        ref = torch.einsum("ht,thd->hd", a, v)
        assert (out[b].float() - ref).abs().max() <= 6e-3 * ref.abs().max()
        start += n

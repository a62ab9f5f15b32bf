"""dq_decode_attention_static: attention for callers that cannot allocate a workspace.

Some users of this library run where device memory may not be requested at call time (a
serving engine with a frozen memory plan, a plug-in under a host that owns all allocations, a
latency-critical loop).  The library therefore carries a fixed scratch array of its own and an
entry point that uses it.  This test drives that entry point through the C ABI and checks it
against the regular entry point (which takes a caller-allocated workspace) on the same inputs,
twice in a row with different sequence lengths, so that anything the first call leaves in the
shared scratch would show up in the second.  It runs last (file name) so that a failure here
cannot hide the result of any other test, and it does not depend on what ran before it.
"""
import pytest
import torch

import paper_2609_19880_b200 as dq
from paper_2609_19880_b200 import _build, workloads

import gpu_common as gc

pytestmark = pytest.mark.gpu


def _run_both(w, tk, tv, cache, seq_lens):
    cfg = w.cfg
    out_a, out32_a = gc.gpu_attention(w, tk, tv, cache, seq_lens=seq_lens)
    out_b = torch.full_like(out_a, float("nan"))
    out32_b = torch.full_like(out32_a, float("nan"))
    dq.dq_decode_attention_static(tk, tv, w.q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale,
                                  w.page_table, seq_lens, cfg.hkv, gc.SM_SCALE, out_b, out32_b)
    torch.cuda.synchronize()
    return out_a, out32_a, out_b, out32_b


def test_static_scratch_entry_point_matches_workspace_entry_point():
    _build.build()
    cfg = workloads.make_config(4, scale=1 / 16)
    cfg.batch, cfg.seq_lens = 4, [700, 33, 1024, 260]
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    need = dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, w.page_table.shape[1])
    assert need <= dq.STATIC_SCRATCH_BYTES
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    gc.gpu_encode(w, tk, tv, cache)
    first = w.seq_lens
    second = torch.tensor([16, 0, 513, 260], dtype=torch.int32, device="cuda")   # shorter: stale partials must not leak
    for lens in (first, second):
        out_a, out32_a, out_b, out32_b = _run_both(w, tk, tv, cache, lens)
        assert torch.isfinite(out32_b).all()
        scale = out32_a.abs().amax(dim=-1, keepdim=True).clamp_min(1e-30)
        assert ((out32_b - out32_a).abs() <= 2e-3 * scale).all()          # the tolerance of the parity tests
        assert torch.equal(out32_b, out32_a) and torch.equal(out_b, out_a)  # and in fact the same bits
    assert not out_b[1].any()                                             # empty sequence -> zero row
    # a warm call leaves the device's memory accounting untouched: neither torch's allocator nor the
    # driver (cudaMemGetInfo) sees a byte move
    torch.cuda.synchronize()
    alloc0, free0 = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
    dq.dq_decode_attention_static(tk, tv, w.q, cache.k_cont, cache.v_cont, cache.mean_q, cache.mean_scale,
                                  w.page_table, second, cfg.hkv, gc.SM_SCALE, out_b, out32_b)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.mem_get_info()[0] == free0
    assert torch.equal(out32_b, out32_a)


def test_static_scratch_rejects_oversized_calls():
    _build.build()
    cfg = workloads.make_config(2, scale=1 / 64)
    w = workloads.generate(cfg, device="cuda")
    tk, tv, ok, ov = gc.tables(cfg)
    cache = gc.GpuCache(w, ok.rec, ov.rec)
    big_pages = 8192                                                      # 131072 tokens per sequence
    assert dq.dq_decode_workspace_bytes(cfg.batch, cfg.hq, big_pages) > dq.STATIC_SCRATCH_BYTES
    pt = torch.zeros((cfg.batch, big_pages), dtype=torch.int32, device="cuda")
    big_mean_q = torch.zeros((cfg.batch, big_pages // 8, cfg.hkv, 128), dtype=torch.int8, device="cuda")
    big_mean_s = torch.zeros((cfg.batch, big_pages // 8, cfg.hkv), dtype=torch.float32, device="cuda")
    out = torch.zeros((cfg.batch, cfg.hq, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(dq.DqError) as err:
        dq.dq_decode_attention_static(tk, tv, w.q, cache.k_cont, cache.v_cont, big_mean_q, big_mean_s, pt,
                                      w.seq_lens, cfg.hkv, gc.SM_SCALE, out)
    assert err.value.code == -4 and "needs" in str(err.value)
    torch.cuda.synchronize()
    assert not out.any()                                                  # nothing was launched

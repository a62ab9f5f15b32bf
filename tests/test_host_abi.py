"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares,
validates arguments before any launch, and its host-built tables equal the oracle's."""
import ctypes as C
import os
import re

import pytest

import oracle
import paper_2609_19880_b200 as dq
from paper_2609_19880_b200 import _build, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    _build.build()
    return dq.lib()


def test_header_symbols_are_exported(L):
    hdr = open(os.path.join(ROOT, "include", "dq.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(dq_[a-z0-9_]+)\s*\(", hdr))
    assert declared == set(dq.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


CASES = [(5, 42, 1.4), (3, 29, 1.4), (16, 36, -1.0), (16, 75, 1.4), (9, 52, 1.4), (8, 56, 1.4),
         (4, 37, 1.4), (3, 27, 1.4), (3, 20, 1.4), (3, 26, 1.4), (5, 39, 1.4), (2, 24, 0.0), (7, 40, 2.5)]


@pytest.mark.parametrize("M,rec,alpha", CASES)
def test_tables_equal_oracle(L, M, rec, alpha):
    t = dq.dq_build_tables(M, rec * 8 / 128, alpha=alpha, has_mean=True, rotate=True)
    i = t.info()
    o = oracle.build_table(M, 128, rec, alpha)
    assert (i.levels, i.rec_bytes, i.container_bytes, i.budget_bits, i.mstar) == (M, rec, o.C, o.B, o.mstar)
    assert abs(i.alpha - o.alpha) < 1e-12
    assert [i.f[m] for m in range(M)] == o.freqs() and [i.c[m] for m in range(M + 1)] == o.cum()
    assert [i.r[m] for m in range(M)] == [o.r[m] for m in range(M)]
    assert [i.R[m] for m in range(M)] == [o.R[m] for m in range(M)]
    for z in range(256):
        e = i.lut[z]
        assert e >> 24 == o.lut_f[z] and e & 255 == o.lut_d[z]
        lvl = oracle.f16_bits_to_f32((e >> 8) & 0xFFFF)
        assert lvl == float(o.lut_m[z])


@pytest.mark.parametrize("M,rec,alpha,sigma", [(5, 42, 1.4, 32), (3, 29, 1.4, 32), (9, 60, 1.4, 32), (8, 56, 1.4, 24),
                                               (4, 37, 1.4, 32), (2, 24, 0.0, 32), (7, 44, 2.5, 32), (6, 42, -1.0, 32)])
def test_pair_tables_equal_oracle(L, M, rec, alpha, sigma):
    """Paired-symbol variant: the pair alphabet's integers and the decode table, entry by entry."""
    t = dq.dq_build_tables(M, rec * 8 / 128, alpha=alpha, has_mean=True, rotate=True, pair_symbols=True, sigma_bits=sigma)
    i = t.info()
    o = oracle.build_table(M, 128, rec, alpha, pair=True, sigma=sigma)
    assert (i.pair_symbols, i.ustar, i.budget_bits, i.sigma_bits) == (1, o.ustar, o.B, sigma)
    assert abs(i.alpha - o.alpha) < 1e-12
    assert [i.f[m] for m in range(M)] == o.freqs()
    assert [i.pair_f[u] for u in range(M * M)] == o.pair_freqs()
    assert [i.pair_R[u] for u in range(M * M)] == [o.pR[u] for u in range(M * M)]
    for z in range(256):
        e = i.lut[z]
        u = o.plut_u[z]
        assert (e >> 16) & 255 == o.plut_f[z] and e & 255 == o.plut_d[z]
        assert oracle.f16_bits_to_f32(e & 0xFF00) == float(u // M)          # level of the even value
        assert oracle.f16_bits_to_f32((e >> 16) & 0xFF00) == float(u % M)   # level of the odd value


def test_pair_tables_limits(L):
    with pytest.raises(dq.DqError) as err:
        dq.dq_build_tables(10, 60 * 8 / 128, pair_symbols=True)            # levels 0..8 only
    assert err.value.code == -3
    t = dq.dq_build_tables(8, 335 * 8 / 1024, heads_per_stream=8, pair_symbols=True)   # token-wide streams take pairs too
    o = oracle.build_table(8, 1024, 335, 1.4, pair=True)
    assert [t.info().pair_f[u] for u in range(64)] == o.pair_freqs() and t.info().ustar == o.ustar
    with pytest.raises(dq.DqError) as err:
        dq.dq_build_tables(8, 335 * 8 / 1024, heads_per_stream=8, pair_symbols=True, sigma_bits=24)
    assert err.value.code == -3
    with pytest.raises(dq.DqError) as err:
        dq.dq_build_tables(9, 20 * 8 / 128, pair_symbols=True)             # the all-central pairs do not fit
    assert err.value.code == -2


@pytest.mark.parametrize("M,hs,rec,alpha", [(8, 8, 335, 1.4), (6, 8, 235, 1.4), (11, 8, 235, 1.4), (6, 2, 86, 1.4),
                                            (16, 8, 600, -1.0), (4, 4, 150, 0.0)])
def test_token_wide_tables_equal_oracle(L, M, hs, rec, alpha):
    """heads_per_stream = hs: the model's n is hs * 128 (Sec. 5.1: one group per token)."""
    n = 128 * hs
    t = dq.dq_build_tables(M, rec * 8 / n, alpha=alpha, has_mean=False, rotate=True, heads_per_stream=hs)
    i = t.info()
    o = oracle.build_table(M, n, rec, alpha)
    assert (i.levels, i.rec_bytes, i.container_bytes, i.budget_bits, i.mstar) == (M, rec, o.C, o.B, o.mstar)
    assert (i.heads_per_stream, i.rec_words, i.head_dim) == (hs, (rec + 3) // 4, 128)
    assert abs(i.alpha - o.alpha) < 1e-12
    assert [i.f[m] for m in range(M)] == o.freqs() and [i.R[m] for m in range(M)] == [o.R[m] for m in range(M)]
    for z in range(256):
        assert i.lut[z] >> 24 == o.lut_f[z] and i.lut[z] & 255 == o.lut_d[z]


def test_token_wide_feasibility_boundary(L):
    """Table 2: at the 231-byte value container 11 levels fit and 12 do not."""
    dq.dq_build_tables(11, 235 * 8 / 1024, heads_per_stream=8)
    with pytest.raises(dq.DqError) as e:
        dq.dq_build_tables(12, 235 * 8 / 1024, heads_per_stream=8)
    assert e.value.code == -2
    with pytest.raises(dq.DqError) as e:
        dq.dq_build_tables(8, 2.6, heads_per_stream=9)
    assert e.value.code == -3


def test_record_size_from_bits(L):
    for bits, rec in [(2.25, 36), (2.625, 42), (1.8125, 29), (4.6875, 75), (2.26, 36), (3.0, 48)]:
        assert dq.dq_build_tables(3, bits).info().rec_bytes == rec == oracle.rec_bytes(bits, 128)


def test_build_errors(L):
    with pytest.raises(dq.DqError) as e:
        dq.dq_build_tables(16, 2.25, alpha=1.4)
    assert e.value.code == -2
    with pytest.raises(dq.DqError) as e:
        dq.dq_build_tables(5, 2.625, head_dim=64)
    assert e.value.code == -3
    for lv, bits, code in [(1, 2.0, -1), (17, 4.0, -3), (5, -1.0, -1), (5, 20.0, -3), (3, 0.5, -2)]:
        with pytest.raises(dq.DqError) as e:
            dq.dq_build_tables(lv, bits)
        assert e.value.code == code, (lv, bits)
    h = C.c_void_p()
    assert L.dq_build_tables(5, 2.625, None, C.byref(h)) == -1
    assert L.dq_strerror(-2).decode().startswith("levels")


def test_calls_validate_before_launch(L):
    """No GPU here: every rejected call must return before touching CUDA."""
    tk = dq.dq_build_tables(5, 2.625, has_mean=True)
    tv = dq.dq_build_tables(3, 1.8125)
    n = None
    assert L.dq_encode_tokens(None, None, n, n, 4, 8, n, n, n, n, n, n, n, 0, 0, n, n) == -1
    assert L.dq_encode_tokens(tk.handle, tv.handle, n, n, 4, 8, n, n, n, n, n, n, n, 0, 0, n, n) == -1
    fake = C.c_void_p(0x1000)
    assert L.dq_encode_tokens(tk.handle, None, fake, n, 4, 8, fake, fake, fake, fake, n, n, n, 4, 0, n, n) == -1
    assert L.dq_encode_tokens(tk.handle, None, fake, n, 4, 8, fake, fake, fake, fake, n, fake, fake, 4, 7, n, n) == -1
    assert L.dq_encode_tokens(tk.handle, None, fake, n, -1, 8, fake, fake, fake, fake, n, fake, fake, 4, 0, n, n) == -1
    assert L.dq_encode_tokens(tk.handle, None, fake, n, 0, 8, fake, fake, fake, fake, n, fake, fake, 4, 0, n, n) == 0
    ws = dq.dq_decode_workspace_bytes(2, 32, 8)
    assert ws > 2 * 32 * 128 * 4 and dq.dq_decode_workspace_bytes(0, 32, 8) == 0
    a = dict(tk=tk.handle, tv=tv.handle, q=fake, kc=fake, vc=fake, mq=fake, ms=fake, mw=1, pt=fake, mp=8,
             sl=fake, B=2, Hq=32, Hkv=8, sm=C.c_float(0.1), ob=fake, of=n, ws=fake, wsb=ws, st=n)

    def call(**kw):
        d = dict(a); d.update(kw)
        return L.dq_decode_attention(*[d[k] for k in ("tk", "tv", "q", "kc", "vc", "mq", "ms", "mw", "pt", "mp",
                                                      "sl", "B", "Hq", "Hkv", "sm", "ob", "of", "ws", "wsb", "st")])

    assert call(q=n) == -1 and call(tk=n) == -1 and call(ob=n) == -1 and call(ws=n) == -1
    assert call(Hq=30) == -1 and call(Hq=128) == -3 and call(B=5000, wsb=1 << 40) == -3
    assert call(wsb=ws - 1) == -4
    assert call(mq=n) == -1 and call(mw=0) == -1       # key tables with a mean need the mean arrays
    assert call(kc=C.c_void_p(0x1001)) == -1           # containers must be 16-byte aligned
    def call_r(rk=fake, rv=fake, rl=fake, cap=128, **kw):
        d = dict(a); d.update(kw)
        return L.dq_decode_attention_residual(
            *[d[k] for k in ("tk", "tv", "q", "kc", "vc", "mq", "ms", "mw", "pt", "mp", "sl")], rk, rv, rl, cap,
            *[d[k] for k in ("B", "Hq", "Hkv", "sm", "ob", "of", "ws", "wsb", "st")])

    # a residual window needs all three arrays, a positive capacity and 8-byte aligned rows
    assert call_r(rv=n) == -1 and call_r(rl=n) == -1 and call_r(rk=n) == -1 and call_r(cap=0) == -1
    assert call_r(rk=C.c_void_p(0x1004)) == -1 and call_r(wsb=ws - 1) == -4 and call_r(q=n) == -1
    def call_m(q_len, **kw):
        d = dict(a); d.update(kw)
        return L.dq_decode_attention_multi(
            d["tk"], d["tv"], d["q"], q_len, *[d[k] for k in ("kc", "vc", "mq", "ms", "mw", "pt", "mp", "sl")], n, n, n, 0,
            *[d[k] for k in ("B", "Hq", "Hkv", "sm", "ob", "of", "ws", "wsb", "st")])

    # several query tokens: the workspace must hold one pass of min(q_len, 8 / (Hq / Hkv)) tokens
    assert call_m(0) == -1 and call_m(2, wsb=ws) == -4 and call_m(5, wsb=dq.dq_decode_workspace_bytes(2, 64, 8) - 1) == -4
    assert call_m(2, q=n, wsb=dq.dq_decode_workspace_bytes(2, 64, 8)) == -1
    # decode step in one call: per token-head tables only; same checks as the two calls it stands for
    def call_s(**kw):
        d = dict(a); d.update(kw)
        return L.dq_decode_step(d["tk"], d["tv"], d.get("kn", fake), d.get("vn", fake), d.get("sn", fake), d["q"], d["kc"],
                                d["vc"], d["mq"], d["ms"], d["mw"], d["pt"], d["mp"], d["sl"], d["B"], d["Hq"], d["Hkv"],
                                d["sm"], d["ob"], d["of"], d["ws"], d["wsb"], n, d["st"])

    assert call_s(kn=n) == -1 and call_s(sn=n) == -1 and call_s(q=n) == -1 and call_s(wsb=ws - 1) == -4
    assert call_s(kn=C.c_void_p(0x1004)) == -1 and call_s(mq=n) == -1
    tw = dq.dq_build_tables(8, 335 * 8 / 1024, has_mean=True, heads_per_stream=8)
    twv = dq.dq_build_tables(6, 235 * 8 / 1024, heads_per_stream=8)
    assert call_s(tk=tw.handle, tv=twv.handle) == -3 and call_s(tk=tw.handle) == -3
    # BF16 window append
    assert L.dq_window_append(n, fake, fake, fake, fake, 128, 2, 8, n) == -1
    assert L.dq_window_append(fake, fake, fake, fake, fake, 0, 2, 8, n) == -1
    assert L.dq_window_append(fake, fake, C.c_void_p(0x1008), fake, fake, 128, 2, 8, n) == -1
    assert L.dq_decode_tokens(tk.handle, n, n, n, 0, n, n, fake, 4, 8, fake, n, n) == -1
    assert L.dq_decode_tokens(tw.handle, fake, n, n, 0, n, n, fake, 4, 12, fake, n, n) == -1   # 12 heads, 8 per stream
    # the entry point with built-in scratch makes the same table / layout checks, all before any CUDA call
    def call_st(**kw):
        d = dict(a); d.update(kw)
        return L.dq_decode_attention_static(*[d[k] for k in ("tk", "tv", "q", "kc", "vc", "mq", "ms", "mw", "pt", "mp",
                                                             "sl", "B", "Hq", "Hkv", "sm", "ob", "of", "st")])

    assert call_st(tk=n) == -1 and call_st(kc=n) == -1 and call_st(B=0) == -1
    assert call_st(tk=tw.handle) == -3                               # key and value tables group heads differently
    assert call_st(tk=tw.handle, tv=twv.handle, Hkv=4, Hq=16) == -1  # 4 KV heads are not a whole 8-head stream
    assert call_st(tv=tk.handle) == -3                               # values carry no window mean
    assert call_st(mq=n) == -1 and call_st(mw=0) == -1 and call_st(kc=C.c_void_p(0x1001)) == -1
    assert call_st(mp=1 << 20) == -1                                 # one window slot cannot cover that many pages
    assert call_st(mw=1 << 17, mp=1 << 20) == -4                     # and this one exceeds the built-in scratch
    assert L.dq_bf16_decode_attention(fake, n, fake, fake, 8, fake, 2, 32, 8, C.c_float(0.1), fake, fake, ws, n) == -1


def test_options_round_trip(L):
    assert dq.dq_get_option(dq.OPT_STEP_POLL_LIMIT) == -1 and dq.dq_get_option(dq.OPT_ENCODE_BATCH_MIN) == -1
    dq.dq_set_option(dq.OPT_STEP_POLL_LIMIT, 0)
    dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, 12345)
    assert dq.dq_get_option(dq.OPT_STEP_POLL_LIMIT) == 0 and dq.dq_get_option(dq.OPT_ENCODE_BATCH_MIN) == 12345
    dq.dq_set_option(dq.OPT_STEP_POLL_LIMIT, -7)
    dq.dq_set_option(dq.OPT_ENCODE_BATCH_MIN, -1)
    assert dq.dq_get_option(dq.OPT_STEP_POLL_LIMIT) == -1 and dq.dq_get_option(dq.OPT_ENCODE_BATCH_MIN) == -1
    assert L.dq_set_option(99, 1) == -1 and L.dq_set_option(dq.OPT_STEP_POLL_LIMIT, 1 << 30) == -1
    assert dq.dq_get_option(99) == -1


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    monkeypatch.setattr(dq, "_lib", None)
    monkeypatch.setattr(dq, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(ImportError):
        dq.dq_build_tables(5, 2.625)


def test_budget_table_matches_record_split():
    for bits, (kr, vr, km, vm) in workloads.BUDGETS.items():
        assert workloads.record_split(bits) == (kr, vr)

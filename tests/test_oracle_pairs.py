"""Pins of the oracle's paired-symbol variant (opt-in; the paper's codec is the default and is
pinned in test_oracle_codec.py / test_oracle_drift.py).

One rANS symbol is the pair of levels of two consecutive values, u = m_2i * M + m_2i+1, over an
alphabet of M^2 <= 256 pairs whose model is the product of the sharpened level model with itself
(Sec. 3.1: the coder is Eq. rans unchanged, on a larger alphabet; Algorithm 2 then takes n / 2
steps for n values).  Drift (Algorithm 1) assigns a pair at a time.

Pinned by:
* the pair coder IS the single-symbol coder on an alphabet of M^2 symbols: byte-identical payloads
  against the (separately pinned) single-symbol coder driven with a hand-built M^2-level table;
* round trip, decoder returning to L, at most one refill byte per step, code length within
  (-8, 0.02] bits of the ideal cost of the pairs, budget test => fit;
* Drift: all M^n assignments enumerated -- feasible, and no assignment of equal or smaller code
  length has lower distortion; nearest rounding under an ample budget; on a table whose pair costs
  are exactly additive (uniform model) the pair search must return what per-value search returns;
  element order inside a pair (a = value 2i) by a stream whose even and odd values differ;
* the model: expected rate under the analytic cell probabilities within a few hundredths of a bit
  per value of the single-symbol table's (numpy restatement of the product + largest-remainder rule
  is only the cross-check, the rate and NMSE comparisons are the pin);
* whole encoder: records decode to the chosen symbols, fit, and quantise N(0,1) streams as well as
  the paper's codec at the benchmark's record sizes.
"""
import itertools
import math

import numpy as np
import pytest

import oracle

# (levels, n, record bytes, alpha)
TABLES = [(5, 128, 42, 1.4), (3, 128, 29, 1.4), (8, 128, 56, 1.4), (9, 128, 60, 1.4), (16, 128, 80, 1.0),
          (8, 1024, 335, 1.4), (6, 1024, 235, 1.4), (4, 128, 40, 0.0)]


def _draw_pairs(T, n, rng):
    """n values whose pairs follow the pair table's own distribution."""
    u = rng.choice(T.M * T.M, size=n // 2, p=np.array(T.pair_freqs()) / 256.0)
    sym = np.empty(n, np.uint8)
    sym[0::2] = u // T.M
    sym[1::2] = u % T.M
    return sym


def _single_table_over_pairs(T):
    """A single-symbol table (M^2 levels) with the pair table's frequencies, built field by field here."""
    K = T.M * T.M
    assert K <= oracle.MAX_LEVELS
    S = oracle.Table()
    S.M, S.n, S.rec, S.C, S.B, S.sigma = K, T.n // 2, T.rec, T.C, T.B, T.sigma
    c = 0
    for u, f in enumerate(T.pair_freqs()):
        S.f[u], S.c[u] = f, c
        for z in range(c, c + f):
            S.lut_m[z], S.lut_f[z], S.lut_d[z] = u, f, z - c
        c += f
    S.c[K] = c
    assert c == 256
    return S


# ------------------------------------------------------------------------ table

@pytest.mark.parametrize("M,n,rec,alpha", TABLES)
def test_pair_table_is_a_valid_rans_model(M, n, rec, alpha):
    T = oracle.build_table(M, n, rec, alpha, pair=True)
    T0 = oracle.build_table(M, n, rec, alpha)
    assert T.pair == 1 and T0.pair == 0 and T.freqs() == T0.freqs() and T.B == T0.B
    pf = T.pair_freqs()
    assert sum(pf) == 256 and min(pf) >= 1 and len(pf) == M * M
    assert [int(T.pc[u]) for u in range(M * M + 1)] == [0] + list(np.cumsum(pf))
    assert pf[T.ustar] == max(pf) and T.ustar == pf.index(max(pf))
    for u, f in enumerate(pf):
        assert T.pR[u] == math.ceil((8 - math.log2(f)) * 65536)
        assert abs(T.pr[u] - (8 - math.log2(f))) < 1e-6
        for z in range(T.pc[u], T.pc[u + 1]):
            assert (T.plut_u[z], T.plut_f[z], T.plut_d[z]) == (u, f, z - T.pc[u])
    # cross-check: product of the sharpened level model; raising the rare pairs to 1 is paid for by
    # the frequent ones, up to three units each
    q = np.array([T.q[m] for m in range(M)])
    t = 256.0 * np.outer(q, q).ravel()
    assert all(f == 1 or -3.0 < f - tt < 1.0 for f, tt in zip(pf, t))


def test_pair_model_rate_matches_level_model():
    """Expected bits per value under the analytic cell probabilities, pairs against single levels:
    equal to within 0.02 bit at the benchmark's level counts, within 0.08 bit up to 9 levels (rare
    pairs are floored at frequency 1 of 256)."""
    for (M, n, rec, tol) in [(5, 128, 42, 0.02), (3, 128, 29, 0.02), (4, 128, 37, 0.03), (6, 128, 42, 0.02),
                             (8, 1024, 335, 0.08), (6, 1024, 235, 0.05), (9, 128, 60, 0.08)]:
        T = oracle.build_table(M, n, rec, 1.4, pair=True)
        p = np.array([T.p[m] for m in range(M)])
        single = float((p * (8 - np.log2(np.array(T.freqs(), float)))).sum())
        pair = float((np.outer(p, p).ravel() * (8 - np.log2(np.array(T.pair_freqs(), float)))).sum()) / 2
        assert abs(pair - single) <= tol, (M, n, single, pair)
        assert pair >= -(p * np.log2(p)).sum() - 1e-9          # never below the source entropy


def test_pair_variant_arguments():
    with pytest.raises(ValueError):
        oracle.build_table(5, 127, 42, 1.4, pair=True)          # odd stream length
    T = oracle.build_table(5, 128, 42, 1.4, pair=True, sigma=24, early_exit=True)
    assert (T.pair, T.sigma, T.early_exit, T.B) == (1, 24, 1, 8 * 38 - 24)
    # feasibility is the all-central stream of n / 2 pairs
    assert T.feasible == int(64 * T.pR[T.ustar] <= T.B * 65536)


# ------------------------------------------------------------------------- rANS

@pytest.mark.parametrize("M,sigma", [(2, 32), (3, 32), (4, 32), (3, 24), (4, 24)])
def test_pair_coder_is_the_single_symbol_coder_on_pairs(M, sigma):
    """Same bytes as Eq. rans run by the single-symbol coder over the alphabet of pairs."""
    n = 128
    T = oracle.build_table(M, n, 60, 1.4, pair=True, sigma=sigma)
    S = _single_table_over_pairs(T)
    rng = np.random.default_rng(17 * M + sigma)
    for i in range(60):
        sym = _draw_pairs(T, n, rng) if i % 3 else rng.integers(0, M, n).astype(np.uint8)
        u = (sym[0::2].astype(np.int64) * M + sym[1::2]).astype(np.uint8)
        a, ka = oracle.rans_encode(sym, T, 300)
        b, kb = oracle.rans_encode(u, S, 300)
        assert ka == kb and np.array_equal(a, b)
        du, xe, pe = oracle.rans_decode(b, n // 2, S)
        ds, xs, ps = oracle.rans_decode(a, n, T)
        assert np.array_equal(du, u) and np.array_equal(ds, sym) and (xe, pe) == (xs, ps)


@pytest.mark.parametrize("M,n,rec,alpha", TABLES)
def test_pair_round_trip_and_state_interval(M, n, rec, alpha):
    T = oracle.build_table(M, n, rec, alpha, pair=True)
    rng = np.random.default_rng(M * 1000 + n)
    cases = [_draw_pairs(T, n, rng) for _ in range(30)]
    cases += [np.zeros(n, np.uint8), np.full(n, M - 1, np.uint8), (np.arange(n) % M).astype(np.uint8),
              (np.arange(n) % 2 * (M - 1)).astype(np.uint8), rng.integers(0, M, n).astype(np.uint8)]
    for sym in cases:
        payload, k = oracle.rans_encode(sym, T, 4 + n)
        assert payload is not None and k <= n // 2            # at most one byte per step
        dec, x_end, ptr = oracle.rans_decode(payload, n, T)
        assert np.array_equal(dec, sym)
        assert x_end == 1 << 23 and ptr == 4 + k
        assert not payload[4 + k:].any()
        assert (1 << 23) <= int.from_bytes(bytes(payload[:4]), "little") < (1 << 31)


def test_pair_decode_restated_with_one_refill_per_step():
    """Algorithm 2 on Python integers over the pair table, one conditional refill per step."""
    T = oracle.build_table(8, 128, 56, 1.4, pair=True)
    rng = np.random.default_rng(3)
    for _ in range(40):
        sym = rng.integers(0, 8, 128).astype(np.uint8)
        payload, k = oracle.rans_encode(sym, T, 200)
        x = int.from_bytes(bytes(payload[:4]), "little")
        ptr, out = 4, []
        for _step in range(64):
            z = x & 255
            out += [T.plut_u[z] // 8, T.plut_u[z] % 8]
            x = T.plut_f[z] * (x >> 8) + T.plut_d[z]
            if x < 1 << 23:
                x = (x << 8) | int(payload[ptr]); ptr += 1
            assert (1 << 23) <= x < (1 << 31)
        assert out == sym.tolist() and ptr == 4 + k and x == 1 << 23


@pytest.mark.parametrize("M,n,rec,alpha", TABLES)
def test_pair_code_length_tracks_ideal_cost(M, n, rec, alpha):
    T = oracle.build_table(M, n, rec, alpha, pair=True)
    r = 8 - np.log2(np.array(T.pair_freqs(), float))
    rng = np.random.default_rng(9)
    for i in range(40):
        sym = _draw_pairs(T, n, rng) if i % 3 else rng.integers(0, M, n).astype(np.uint8)
        payload, k = oracle.rans_encode(sym, T, 4 + n)
        ideal = r[sym[0::2].astype(np.int64) * M + sym[1::2]].sum()
        assert abs(T.code_length(sym) / 65536 - ideal) < n * 2.0 ** -16
        assert -8.0 < 8 * k - ideal <= 0.02               # 32-bit state: floor(x / f) loses < 2^-15 bit a step


@pytest.mark.parametrize("M,n,rec,alpha", TABLES)
def test_pair_budget_test_guarantees_fit(M, n, rec, alpha):
    T = oracle.build_table(M, n, rec, alpha, pair=True)
    rng = np.random.default_rng(13)
    worst = int(np.argmax(T.pair_freqs()[::-1]))            # some rarest pair
    worst = M * M - 1 - worst
    pR = [int(T.pR[u]) for u in range(M * M)]
    for trial in range(120 if n == 128 else 30):
        u = np.full(n // 2, T.ustar, np.int64)
        length = (n // 2) * pR[T.ustar]
        for i in rng.permutation(n // 2):
            cand = int(rng.integers(0, M * M)) if trial % 3 else (worst if trial % 2 else int(np.argmin(T.pair_freqs())))
            if length - pR[u[i]] + pR[cand] <= T.B * 65536:
                length += pR[cand] - pR[u[i]]
                u[i] = cand
        sym = np.empty(n, np.uint8)
        sym[0::2], sym[1::2] = u // M, u % M
        assert T.code_length(sym) == length <= T.B * 65536
        payload, k = oracle.rans_encode(sym, T, T.C)
        assert payload is not None and 4 + k <= T.C


# ------------------------------------------------------------------------ drift

def _tiny(M, n, alpha=1.4, early_exit=False):
    T = oracle.build_table(M, max(n, 2), 64, alpha, pair=True, early_exit=early_exit)
    T.n = n
    return T


@pytest.mark.parametrize("M,n", [(3, 6), (4, 4), (4, 6), (3, 8), (5, 4)])
@pytest.mark.parametrize("early_exit", [False, True])
def test_pair_drift_is_lagrangian_optimal_by_enumeration(M, n, early_exit):
    rng = np.random.default_rng(100 * M + n)
    all_m = np.array(list(itertools.product(range(M), repeat=n)), dtype=np.int64)
    T = _tiny(M, n, early_exit=early_exit)
    pR = np.array([T.pR[u] for u in range(M * M)], dtype=np.int64)
    L_all = pR[all_m[:, 0::2] * M + all_m[:, 1::2]].sum(1)
    checked = 0
    for trial in range(50):
        z = rng.standard_normal(n).astype(np.float32)
        o = float(z.min()); s = float((z.max() - z.min()) / (M - 1))
        near = np.clip(np.rint((z - np.float32(o)) / np.float32(s)), 0, M - 1).astype(np.int64)
        lo, hi = (n // 2) * pR.min(), T.code_length(near)
        T.B = int((lo + (hi - lo) * rng.uniform(0.2, 0.9)) // 65536) if trial % 2 else int(hi // 65536) + 2
        m, ln = oracle.drift(z, s, o, T)
        assert ln == T.code_length(m)
        if ln > T.B * 65536:
            continue
        checked += 1
        if trial % 2 == 0:
            assert np.array_equal(m, near)                  # ample budget: nearest rounding
        grid = np.float32(o) + np.arange(M, dtype=np.float32) * np.float32(s)
        D = ((z[None, :].astype(np.float64) - grid[all_m].astype(np.float64)) ** 2).sum(1)
        mine = ((z.astype(np.float64) - grid[m].astype(np.float64)) ** 2).sum()
        assert mine <= D[L_all <= ln].min() * (1 + 1e-5) + 1e-9
    assert checked >= 30


@pytest.mark.parametrize("M", [2, 4, 8, 16])
def test_pair_drift_on_additive_costs_equals_per_value_drift(M):
    """Uniform model (alpha = 0): f = 256 / M per level and 256 / M^2 per pair, so a pair costs exactly
    the sum of its levels and every assignment has the same length; both searches must return nearest
    rounding, value by value -- which also fixes which value of a pair is `a`."""
    n = 128
    bits = int(math.log2(M))
    rec = 4 + 4 + (n * bits + 7) // 8 + 2
    Tp = oracle.build_table(M, n, rec, 0.0, pair=True)
    Ts = oracle.build_table(M, n, rec, 0.0)
    assert set(Tp.pair_freqs()) == {256 // (M * M)} and set(Ts.freqs()) == {256 // M}
    rng = np.random.default_rng(M)
    for _ in range(50):
        z = rng.standard_normal(n).astype(np.float32)
        z[0::2] *= 0.25                                      # even and odd values are not exchangeable
        o = float(z.min()); s = float(np.float32((z.max() - z.min()) / np.float32(M - 1)))
        mp, lp = oracle.drift(z, s, o, Tp)
        ms, ls = oracle.drift(z, s, o, Ts)
        assert lp == ls == n * bits * 65536
        assert np.array_equal(mp, ms)


def test_pair_drift_meets_budget_and_changes_few_symbols():
    """App. C: drift moves few symbols and by one level."""
    rng = np.random.default_rng(5)
    for (M, n, rec) in [(5, 128, 42), (3, 128, 29), (8, 1024, 335)]:
        T = oracle.build_table(M, n, rec, 1.4, pair=True)
        changed = total = 0
        for _ in range(60 if n == 128 else 15):
            z = rng.standard_normal(n).astype(np.float32)
            o = float(z.min()); s = float(np.float32((z.max() - z.min()) / np.float32(M - 1)))
            m, ln = oracle.drift(z, s, o, T)
            assert ln <= T.B * 65536 and ln == T.code_length(m)
            near = np.clip(np.rint((z - np.float32(o)) / np.float32(s)), 0, M - 1).astype(np.int64)
            assert np.abs(m.astype(np.int64) - near).max() <= 1
            changed += int((m != near).sum()); total += n
        assert changed <= 0.25 * total


# ---------------------------------------------------------------------- encoder

@pytest.mark.parametrize("M,n,rec,alpha", TABLES[:7])
@pytest.mark.parametrize("sigma", [32, 24])
def test_pair_encoder_records_fit_and_decode(M, n, rec, alpha, sigma):
    if sigma == 24 and n > 640:
        pytest.skip("the 24-bit state is offered for streams of at most 640 values")
    T = oracle.build_table(M, n, rec, alpha, pair=True, sigma=sigma)
    rng = np.random.default_rng(M + n + sigma)
    fallback = 0
    for i in range(40 if n == 128 else 10):
        z = (rng.standard_normal(n) * (0.1, 1.0, 7.0)[i % 3] + (0.0, 2.0)[i % 2]).astype(np.float32)
        rec_b, sym, st = oracle.encode_stream(z, T)
        assert rec_b.shape == (rec,) and st[3] <= rec
        dec, _, ptr = oracle.rans_decode(rec_b[4:], n, T)
        assert np.array_equal(dec, sym)
        assert T.code_length(sym) <= T.B * 65536 or st[0] == 1
        assert not rec_b[4 + ptr:].any()
        fallback += int(st[0])
    assert fallback == 0
    # constant stream: all-central pairs, zero scale
    rec_b, sym, st = oracle.encode_stream(np.full(n, 3.0, np.float32), T)
    assert st[1] == 1 and rec_b[0] == 0 and rec_b[1] == 0
    assert set(zip(sym[0::2].tolist(), sym[1::2].tolist())) == {(T.ustar // M, T.ustar % M)}


def test_pair_quality_matches_the_paper_codec_at_benchmark_budgets():
    """NMSE on N(0,1) streams with the same records: pairs at most half a point above single levels
    (they come out slightly below: the pair table resolves the frequent pairs more finely)."""
    rng = np.random.default_rng(2)
    for (M, rec) in [(5, 42), (3, 29), (8, 56)]:
        Z = [rng.standard_normal(128).astype(np.float32) for _ in range(150)]
        out = []
        for pair in (False, True):
            T = oracle.build_table(M, 128, rec, 1.4, pair=pair)
            num = den = 0.0
            for z in Z:
                r, sym, _ = oracle.encode_stream(z, T)
                s = oracle.f16_bits_to_f32(int(r[0]) | int(r[1]) << 8)
                o = oracle.f16_bits_to_f32(int(r[2]) | int(r[3]) << 8)
                num += float(((z - (sym.astype(np.float64) * s + o)) ** 2).sum())
                den += float((z.astype(np.float64) ** 2).sum())
            out.append(num / den)
        assert -0.02 <= out[1] - out[0] <= 0.005, (M, rec, out)

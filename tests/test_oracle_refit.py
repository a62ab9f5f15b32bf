"""Direct pins of the Refit step of the oracle's one-stream encoder (Algorithm 1, lines 3-4:
least-squares refit of the grid to the drifted symbols, then FP16 rounding of both parameters;
App. B lists it as "least-squares refitting").

Two things are shown on thousands of random streams, per-head (n = 128) and token-wide
(n = 1024) alike:

* the (s, o) a record carries equal an independent least-squares solve (numpy.linalg.lstsq in
  binary64 on the symbols of the first Drift) rounded once to binary16 by numpy -- so a slip in
  the normal equations (n versus n - 1, a swapped sum, o solved from the rounded s) fails;
* the fixed summation order the oracle uses for the two floating-point sums (per 128 values: 32
  partial sums of consecutive elements joined by a butterfly; blocks in order) is a harmless
  reading: a plain left-to-right binary64 sum and the exactly rounded sum (math.fsum) give the
  same binary16 pair on every stream.
"""
import math

import numpy as np
import pytest

import oracle

# (levels, stream length n, record bytes, alpha; alpha < 0 = automatic rule)
CASES = [(3, 128, 29, 1.4), (5, 128, 42, 1.4), (16, 128, 36, -1.0), (8, 128, 56, 1.4),
         (8, 1024, 335, 1.4), (6, 1024, 235, 1.4)]
N_STREAMS = {128: 2400, 1024: 2000}


def _streams(n, count, seed):
    """Gaussian streams with a spread of scales and offsets, plus a few heavy-tailed ones."""
    rng = np.random.default_rng(seed)
    for i in range(count):
        z = rng.standard_normal(n)
        if i % 7 == 3:
            z = rng.standard_t(5, n) / math.sqrt(5.0 / 3.0)
        scale = (0.05, 1.0, 3.0, 17.0)[i % 4]
        shift = (0.0, -0.7, 2.5)[i % 3]
        yield (z * scale + shift).astype(np.float32)


def _f16_pair(rec):
    return int(rec[0]) | int(rec[1]) << 8, int(rec[2]) | int(rec[3]) << 8


def _first_drift(z, T):
    """Symbols of the first Drift: on the min-max grid of Eq. (affine_token), binary32."""
    mn, mx = np.float32(z.min()), np.float32(z.max())
    s0 = np.float32((mx - mn) / np.float32(T.M - 1))
    m, _ = oracle.drift(z, float(s0), float(mn), T)
    return m, s0, mn


def _half_bits(v):
    return int(np.array([v], dtype=np.float64).astype(np.float16).view(np.uint16)[0])


@pytest.mark.parametrize("M,n,rec,alpha", CASES)
def test_record_grid_equals_independent_least_squares(M, n, rec, alpha):
    T = oracle.build_table(M, n, rec, alpha)
    checked = kept_minmax = 0
    for z in _streams(n, N_STREAMS[n], seed=100 * M + n):
        r, _, st = oracle.encode_stream(z, T)
        assert st[2] == 0, "refit rejected on an ordinary stream"
        assert st[1] == 0
        m, s0, o0 = _first_drift(z, T)
        if len(set(m.tolist())) < 2:                     # singular normal equations: grid kept
            assert _f16_pair(r) == (_half_bits(float(s0)), _half_bits(float(o0)))
            kept_minmax += 1
            continue
        A = np.stack([m.astype(np.float64), np.ones(n)], axis=1)
        (s_ls, o_ls), *_ = np.linalg.lstsq(A, z.astype(np.float64), rcond=None)
        assert _f16_pair(r) == (_half_bits(s_ls), _half_bits(o_ls)), (s_ls, o_ls)
        checked += 1
    assert checked >= 0.95 * N_STREAMS[n] and kept_minmax <= 0.05 * N_STREAMS[n]


@pytest.mark.parametrize("M,n,rec,alpha", CASES)
def test_summation_order_of_refit_changes_no_record(M, n, rec, alpha):
    """Normal equations solved from (a) a left-to-right binary64 running sum and (b) the exactly
    rounded sums: both must round to the record's binary16 pair.  The count of differing
    streams is the evidence; it is asserted to be zero."""
    T = oracle.build_table(M, n, rec, alpha)
    differ_seq = differ_exact = total = 0
    for z in _streams(n, N_STREAMS[n], seed=7 * M + n):
        r, _, _ = oracle.encode_stream(z, T)
        m, _, _ = _first_drift(z, T)
        if len(set(m.tolist())) < 2:
            continue
        zd, md = z.astype(np.float64), m.astype(np.float64)
        Sm, Smm = int(m.astype(np.int64).sum()), int((m.astype(np.int64) ** 2).sum())
        den = n * Smm - Sm * Sm
        prod = md * zd                                    # exact: a small integer times a binary32
        for kind, (Sz, Smz) in (("seq", (np.cumsum(zd)[-1], np.cumsum(prod)[-1])),
                                ("exact", (math.fsum(zd.tolist()), math.fsum(prod.tolist())))):
            s = (n * Smz - Sm * Sz) / den
            o = (Sz - s * Sm) / n
            if (_half_bits(s), _half_bits(o)) != _f16_pair(r):
                if kind == "seq":
                    differ_seq += 1
                else:
                    differ_exact += 1
        total += 1
    assert total >= 0.95 * N_STREAMS[n]
    assert (differ_seq, differ_exact) == (0, 0), f"{differ_seq} / {differ_exact} of {total} streams differ"


def test_refit_uses_unrounded_scale_for_offset():
    """Reading of Alg. 1 lines 3-4: o comes from the unrounded least-squares s, and only then are
    both rounded.  Solving o from the binary16-rounded s instead gives a different record on a
    noticeable share of streams, so the pin above does separate the two readings."""
    T = oracle.build_table(5, 128, 42, 1.4)
    other = total = 0
    for z in _streams(128, 600, seed=11):
        r, _, _ = oracle.encode_stream(z, T)
        m, _, _ = _first_drift(z, T)
        if len(set(m.tolist())) < 2:
            continue
        md, zd = m.astype(np.float64), z.astype(np.float64)
        A = np.stack([md, np.ones(128)], axis=1)
        (s_ls, _), *_ = np.linalg.lstsq(A, zd, rcond=None)
        s_h = float(np.float16(s_ls))
        o_alt = (zd.sum() - s_h * md.sum()) / 128.0
        total += 1
        other += _half_bits(o_alt) != _f16_pair(r)[1]
    assert other >= 0.05 * total, (other, total)

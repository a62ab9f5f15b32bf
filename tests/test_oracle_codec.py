"""Pins of the oracle's rANS codec (Eq. rans, Algorithm 2), fp16 rounding and Hadamard."""
import math

import numpy as np
import pytest
from scipy.linalg import hadamard

import oracle

TABLES = [(5, 128, 42, 1.4), (3, 128, 29, 1.4), (16, 128, 75, 1.4), (16, 128, 36, -1.0),
          (8, 1024, 335, 1.4), (6, 1024, 235, 1.4), (4, 128, 40, 0.0)]


def _draw(T, n, rng):
    return rng.choice(T.M, size=n, p=np.array(T.freqs()) / 256.0).astype(np.uint8)


# ------------------------------------------------------------------ single step

def test_single_step_enc_dec_are_inverse_on_integers():
    """Eq. (rans) without renormalisation, in exact integer arithmetic written here:
    Dec(Enc(x, m)) = x and the slot x mod 2^p of Enc(x, m) lies in [c_m, c_m + f_m)."""
    T = oracle.build_table(5, 128, 42, 1.4)
    f, c = T.freqs(), T.cum()
    rng = np.random.default_rng(1)
    for _ in range(2000):
        x = int(rng.integers(1, 2 ** 40))
        m = int(rng.integers(0, T.M))
        y = (x // f[m]) * 256 + (x % f[m]) + c[m]
        z = y % 256
        assert c[m] <= z < c[m] + f[m] and T.lut_m[z] == m
        assert f[m] * (y // 256) + z - c[m] == x


# ------------------------------------------------------------------- round trip

@pytest.mark.parametrize("M,n,rec,alpha", TABLES)
def test_round_trip_identity(M, n, rec, alpha):
    T = oracle.build_table(M, n, rec, alpha)
    rng = np.random.default_rng(M * 1000 + n)
    cases = [_draw(T, n, rng) for _ in range(40)]
    cases += [np.full(n, T.mstar, np.uint8), np.zeros(n, np.uint8), np.full(n, M - 1, np.uint8),
              (np.arange(n) % M).astype(np.uint8), rng.integers(0, M, n).astype(np.uint8)]
    for sym in cases:
        payload, k = oracle.rans_encode(sym, T, 4 + 2 * n)
        assert payload is not None
        dec, x_end, ptr = oracle.rans_decode(payload, n, T)
        assert np.array_equal(dec, sym)
        assert x_end == 1 << 23 and ptr == 4 + k      # decoder returns to the initial state
        assert not payload[4 + k:].any()              # zero padding after the used bytes
        state = int.from_bytes(bytes(payload[:4]), "little")
        assert (1 << 23) <= state < (1 << 31)


# ------------------------------------------------------------ length vs Shannon

@pytest.mark.parametrize("M,n,rec,alpha", TABLES)
def test_code_length_tracks_ideal_cost(M, n, rec, alpha):
    """8k stays within (-8, +0.01] bits of sum_j r(m_j): byte granularity below, the
    accumulated floor(x/f) loss above (n * log2(1 + 2^-15))."""
    T = oracle.build_table(M, n, rec, alpha)
    r = np.array([8 - math.log2(f) for f in T.freqs()])
    rng = np.random.default_rng(7)
    for i in range(60):
        sym = _draw(T, n, rng) if i % 3 else rng.integers(0, M, n).astype(np.uint8)
        payload, k = oracle.rans_encode(sym, T, 4 + 2 * n)
        ideal = r[sym].sum()
        assert -8.0 < 8 * k - ideal <= 0.01
        assert k <= math.floor((ideal + 0.01) / 8)


def test_mean_rate_close_to_entropy():
    """On iid draws from the table's own distribution the payload rate approaches H(f/256)."""
    T = oracle.build_table(8, 1024, 335, 1.4)
    rng = np.random.default_rng(3)
    ks = [oracle.rans_encode(_draw(T, 1024, rng), T, 4096)[1] for _ in range(300)]
    rate = 8 * np.mean(ks) / 1024
    assert abs(rate - T.entropy()) < 0.01


@pytest.mark.parametrize("M,n,rec,alpha", TABLES)
def test_budget_test_guarantees_fit(M, n, rec, alpha):
    """If the fixed-point cost sum_j R(m_j) <= 65536 B then the stream fits its C bytes
    (Eq. budget with sigma = 32), including worst cases that sit exactly at the budget."""
    T = oracle.build_table(M, n, rec, alpha)
    R = np.array([T.R[m] for m in range(M)], dtype=np.int64)
    rng = np.random.default_rng(11)
    tried = 0
    for _ in range(400):
        sym = np.full(n, T.mstar, np.uint8)
        order = rng.permutation(n)
        for j in order:                                # greedily load expensive symbols
            cand = int(rng.integers(0, M))
            if R[sym].sum() - R[sym[j]] + R[cand] <= T.B * 65536:
                sym[j] = cand
        assert R[sym].sum() <= T.B * 65536
        payload, k = oracle.rans_encode(sym, T, T.C)
        assert payload is not None and 4 + k <= T.C
        tried += 1
    assert tried == 400


def test_at_most_one_refill_byte_per_symbol():
    """After a decode step the state is >= 2^15, so one byte always restores x >= L."""
    T = oracle.build_table(16, 128, 36, -1.0)
    rng = np.random.default_rng(5)
    for _ in range(50):
        sym = rng.integers(0, 16, 128).astype(np.uint8)
        payload, k = oracle.rans_encode(sym, T, 400)
        x = int.from_bytes(bytes(payload[:4]), "little")
        ptr = 4
        for j in range(128):
            z = x & 255
            x = T.lut_f[z] * (x >> 8) + T.lut_d[z]
            assert x >= 1 << 15
            if x < 1 << 23:
                x = (x << 8) | int(payload[ptr]); ptr += 1
            assert x >= 1 << 23


def test_decoder_never_reads_past_the_container():
    """A corrupted record yields wrong symbols but the read pointer stays inside."""
    T = oracle.build_table(5, 128, 42, 1.4)
    rng = np.random.default_rng(9)
    for _ in range(100):
        junk = rng.integers(0, 256, T.C).astype(np.uint8)
        sym, x_end, ptr = oracle.rans_decode(junk, 128, T)
        assert ptr <= T.C and sym.max() < T.M


# ---------------------------------------------------------------------- fp16

def test_fp16_rounding_matches_numpy():
    rng = np.random.default_rng(2)
    vals = np.concatenate([
        rng.standard_normal(20000) * 10.0 ** rng.integers(-9, 6, 20000),
        np.array([0.0, -0.0, 1.0, 65504.0, 65519.99, 65520.0, 1e6, -1e6, 2.0 ** -24, 2.0 ** -25,
                  2.0 ** -25 * (1 + 1e-12), 3 * 2.0 ** -25, 6.1e-5, 6.103515625e-05, 1.0009765625,
                  1.00048828125, 1.00146484375, 2047.5, 2048.5, 1e-30, np.inf, -np.inf]),
        np.float16(rng.standard_normal(2000)).astype(np.float64) * (1 + 2.0 ** -12),   # near ties
    ])
    with np.errstate(over="ignore"):
        ref = vals.astype(np.float16)
    for v, r in zip(vals, ref):
        bits = oracle.f64_to_f16_bits(v)
        assert bits == int(r.view(np.uint16)), v
        if np.isfinite(r):
            assert oracle.f16_bits_to_f32(bits) == float(r)


def test_fp16_decode_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    for b in range(0, 65536, 7):
        v = oracle.f16_bits_to_f32(b)
        assert (math.isnan(v) and math.isnan(ref[b])) or v == ref[b]


# ------------------------------------------------------------------ Hadamard

@pytest.mark.parametrize("n", [32, 128, 1024])
def test_hadamard_matches_sylvester_matrix(n):
    H = hadamard(n).astype(np.float64) / math.sqrt(n)
    rng = np.random.default_rng(n)
    x = rng.standard_normal((6, n))
    y32 = oracle.fwht_f32(x.astype(np.float32))
    y64 = oracle.fwht_f64(x)
    assert np.allclose(y64, x @ H.T, atol=1e-12)
    assert np.allclose(y32, x.astype(np.float32).astype(np.float64) @ H.T, atol=2e-5)
    assert np.allclose(oracle.fwht_f64(y64), x, atol=1e-12)          # self-inverse
    assert np.allclose(oracle.fwht_f32(y32), x, atol=2e-5)
    assert np.allclose(np.linalg.norm(y64, axis=1), np.linalg.norm(x, axis=1), rtol=1e-12)


def test_hadamard_unit_vectors_are_exact():
    """Seven +- stages on a unit vector are exact, the scale is fp32(1/sqrt(128))."""
    sc = np.array([0x3DB504F3], dtype=np.uint32).view(np.float32)[0]
    assert sc == np.float32(1.0 / math.sqrt(128.0))
    H = hadamard(128)
    for i in (0, 1, 5, 64, 127):
        e = np.zeros(128, np.float32); e[i] = 1.0
        y = oracle.fwht_f32(e)
        assert np.array_equal(y, H[:, i].astype(np.float32) * sc)

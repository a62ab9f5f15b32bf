"""Pins of the oracle's probability model, rANS tables and storage accounting.

Everything here is checked against something the paper or mathematics fixes, never
against the CUDA library: the paper's storage figures (closed form), the feasibility
boundary of its Table 2, quadrature by an independent library routine, and textbook
special cases.
"""
import math

import numpy as np
import pytest
from scipy import integrate, stats

import oracle


def _constants(golden_dir):
    out = {}
    with open(f"{golden_dir}/paper_storage_constants.txt") as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            name, val = line.split()[:2]
            out[name] = float(val)
    return out


def _table2(golden_dir):
    rows = []
    with open(f"{golden_dir}/paper_table2_nmse.txt") as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            m, k, v = line.split()
            rows.append((int(m), float(k), float(v)))
    return rows


def test_storage_accounting_closes_on_paper_figures(golden_dir):
    """2.68 / 1.84 / 2.26 bits follow from 331 / 231-byte containers, n = 1024, two fp16
    metadata values per stream and one INT8 mean per key channel per 128-token window."""
    c = _constants(golden_dir)
    n = int(c["stream_values"])
    key = (c["key_container_bytes"] * 8 + 32) / n + 8.0 / oracle.WINDOW
    val = (c["value_container_bytes"] * 8 + 32) / n
    assert round(key, 2) == c["key_bpe"]
    assert round(val, 2) == c["value_bpe"]
    assert round((key + val) / 2, 2) == c["average_bpe"]
    # the oracle's record = container + 4 metadata bytes, budget B = 8C - 32 (Eq. budget)
    T = oracle.build_table(8, n, int(c["key_container_bytes"]) + 4, c["alpha"])
    assert T.C == 331 and T.B == 8 * 331 - 32 and T.rec == 335
    # INT2, group 128, fp16 scale and zero point: 2.25 bits per value (Sec. 3.1)
    assert (2 * 128 + 32) / 128 == c["int2_g128_fp16_bpv"]
    assert oracle.rec_bytes(2.25, 128) == 36


def test_fixed_width_equivalent_levels(golden_dir):
    c = _constants(golden_dir)
    n = c["stream_values"]
    assert math.floor(2 ** (c["key_container_bytes"] * 8 / n)) == c["fixed_width_key_levels"]
    assert math.floor(2 ** (c["value_container_bytes"] * 8 / n)) == c["fixed_width_value_levels"]


@pytest.mark.parametrize("n", [128, 1024, 32])
def test_expected_max_matches_independent_quadrature(n):
    f = lambda x: x * n * stats.norm.pdf(x) * stats.norm.cdf(x) ** (n - 1)
    ref, _ = integrate.quad(f, -12, 12, epsabs=1e-13, epsrel=1e-13, limit=400)
    assert abs(oracle.expected_max(n) - ref) < 1e-9
    # sanity against sampling: mean of maxima of n normals
    rng = np.random.default_rng(0)
    mc = rng.standard_normal((20000, n)).max(axis=1).mean()
    assert abs(oracle.expected_max(n) - mc) < 0.02


def test_expected_max_closed_forms():
    assert abs(oracle.expected_max(1)) < 1e-12
    assert abs(oracle.expected_max(2) - 1.0 / math.sqrt(math.pi)) < 1e-10
    assert abs(oracle.expected_max(3) - 1.5 / math.sqrt(math.pi)) < 1e-10


def test_table2_feasibility_boundary(golden_dir):
    """Table 2: at the 231-byte value container M <= 11 fits and M = 12, 14 do not; at the
    331-byte key container every listed alphabet fits."""
    for M, key_nmse, val_nmse in _table2(golden_dir):
        Tk = oracle.build_table(M, 1024, 331 + 4, 1.4, allow_infeasible=True)
        Tv = oracle.build_table(M, 1024, 231 + 4, 1.4, allow_infeasible=True)
        assert bool(Tk.feasible) == math.isfinite(key_nmse), M
        assert bool(Tv.feasible) == math.isfinite(val_nmse), M


@pytest.mark.parametrize("M,n,rec,alpha", [(8, 1024, 335, 1.4), (6, 1024, 235, 1.4), (5, 128, 42, 1.4),
                                           (3, 128, 29, 1.4), (16, 128, 75, 1.4), (16, 128, 36, -1.0),
                                           (2, 128, 24, 1.4), (9, 128, 52, 1.4), (7, 64, 40, 2.0)])
def test_table_invariants(M, n, rec, alpha):
    T = oracle.build_table(M, n, rec, alpha)
    f, c = T.freqs(), T.cum()
    assert sum(f) == 256 and min(f) >= 1 and max(f) <= 255
    assert c[0] == 0 and all(c[m + 1] - c[m] == f[m] for m in range(M))
    # symmetric model: frequencies differ from their mirror by at most the remainder unit
    assert all(abs(f[m] - f[M - 1 - m]) <= 1 for m in range(M))
    p = np.array([T.p[m] for m in range(M)])
    assert abs(p.sum() - 1) < 1e-12 and np.allclose(p, p[::-1], atol=0, rtol=0)
    # probabilities peak in the centre (normal cells), costs follow -log2(f/256)
    assert p.argmax() in ((M - 1) // 2, M // 2)
    for m in range(M):
        r = 8.0 - math.log2(f[m])
        assert T.r[m] == np.float32(r)
        assert T.R[m] == math.ceil(r * 65536) and T.R[m] >= r * 65536
    assert f[T.mstar] == max(f) and T.mstar == f.index(max(f))
    for z in range(256):
        m = T.lut_m[z]
        assert c[m] <= z < c[m + 1] and T.lut_f[z] == f[m] and T.lut_d[z] == z - c[m]
    assert T.feasible == (n * T.R[T.mstar] <= T.B * 65536)


def test_cell_probabilities_against_library_cdf():
    """Cell masses of the +-E[max] grid, recomputed with scipy's normal CDF."""
    for M, n in [(8, 1024), (5, 128), (3, 128)]:
        T = oracle.build_table(M, n, 400, 1.4)
        E = integrate.quad(lambda x: x * n * stats.norm.pdf(x) * stats.norm.cdf(x) ** (n - 1), -12, 12,
                           epsabs=1e-13, epsrel=1e-13, limit=400)[0]
        edges = np.clip(-E + (np.arange(M + 1) - 0.5) * (2 * E / (M - 1)), -E, E)
        p = np.diff(stats.norm.cdf(edges))
        p /= p.sum()
        assert np.allclose([T.p[m] for m in range(M)], p, atol=1e-10)
        q = p ** 1.4
        assert np.allclose([T.q[m] for m in range(M)], q / q.sum(), atol=1e-10)


def test_paper_default_tables_have_slack():
    """The paper's 8/6-level defaults sit comfortably inside their containers (App. C):
    table entropy well below the per-value budget at alpha = 1.4."""
    Tk = oracle.build_table(8, 1024, 335, 1.4)
    Tv = oracle.build_table(6, 1024, 235, 1.4)
    assert Tk.freqs() == [1, 3, 30, 94, 94, 30, 3, 1]
    assert Tv.freqs() == [1, 14, 113, 113, 14, 1]
    assert Tk.entropy() < Tk.B / 1024 and Tv.entropy() < Tv.B / 1024


def test_coding_gain_of_model_near_paper(golden_dir):
    """Table 1 reports 0.72 / 0.86 bits of coding gain for an eight-level per-token grid;
    the analytic model's log2(8) - H(p) must land between and near them (soft pin)."""
    c = _constants(golden_dir)
    T = oracle.build_table(8, 1024, 335, 1.4)
    gain = 3.0 - T.model_entropy()
    assert c["coding_gain_key"] - 0.1 <= gain <= c["coding_gain_value"] + 0.1


def test_alpha_zero_is_fixed_width():
    """alpha = 0 with M = 2^b levels gives the uniform table: every symbol costs b bits."""
    for b in (1, 2, 3, 4):
        T = oracle.build_table(2 ** b, 128, 128 * b // 8 + 8, 0.0)
        assert T.freqs() == [256 >> b] * (2 ** b)
        assert all(T.R[m] == b * 65536 for m in range(2 ** b))


def test_auto_alpha_rule():
    """Automatic alpha: smallest of 1.4, 1.5, ... whose table fits; the paper's own
    operating points keep 1.4, the over-subscribed 16-level / 36-byte case does not."""
    assert oracle.build_table(8, 1024, 335, -1.0).alpha == 1.4
    assert oracle.build_table(6, 1024, 235, -1.0).alpha == 1.4
    T = oracle.build_table(16, 128, 36, -1.0)
    assert T.alpha > 1.4 and T.feasible and T.entropy() <= T.B / 128
    prev = oracle.build_table(16, 128, 36, round(T.alpha - 0.1, 1), allow_infeasible=True)
    assert (not prev.feasible) or prev.entropy() > prev.B / 128
    with pytest.raises(ValueError):
        oracle.build_table(16, 128, 36, 1.4)  # infeasible as given


def test_level_rule_reproduces_budget_table():
    """Benchmark level choice: V takes the largest M <= 16 with H(p_M) <= B/n, K the largest
    with H(p_M) <= 0.875 B/n, floor 3; at the paper's sizes the rule returns 8 / 6."""
    from paper_2609_19880_b200 import workloads

    def pick(n, rec, frac):
        best = 3
        for M in range(2, 17):
            T = oracle.build_table(M, n, rec, 1.4, allow_infeasible=True)
            if T.model_entropy() <= frac * T.B / n:
                best = max(best, M)
        return best

    assert pick(1024, 335, 0.875) == 8 and pick(1024, 235, 1.0) == 6
    for bits, (kr, vr, km, vm) in workloads.BUDGETS.items():
        assert workloads.record_split(bits) == (kr, vr)
        assert pick(128, kr, 0.875) == km, bits
        assert pick(128, vr, 1.0) == vm, bits
        # and the chosen tables are feasible at alpha = 1.4
        assert oracle.build_table(km, 128, kr, -1.0).alpha == 1.4
        assert oracle.build_table(vm, 128, vr, -1.0).alpha == 1.4
    assert (42 + 29 + 1) * 8 / 256 == 2.25

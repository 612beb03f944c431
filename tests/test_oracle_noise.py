"""Pins for the oracle's noise generator (CPU only)."""
import math
import os

import numpy as np
import pytest
from scipy import stats

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _kat_rows():
    rows = []
    with open(os.path.join(GOLD, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            v = [int(t, 16) for t in line.split()]
            rows.append((v[0:4], v[4:6], v[6:10]))
    return rows


@pytest.mark.parametrize("ctr,key,want", _kat_rows())
def test_philox_known_answers(ctr, key, want):
    got = oracle.philox4x32_10(ctr, key)
    assert [int(x) for x in got] == want


def test_philox_is_a_bijection_on_counters():
    # For a fixed key the block function permutes counters: distinct counters never collide.
    seen = set()
    for q in range(2000):
        seen.add(tuple(int(x) for x in oracle.philox4x32_10([q, 3, 1, 0], [5, 6])))
    assert len(seen) == 2000


def _normals(seed, layer, p, which, count, r=1):
    return oracle.noise_factor(seed, layer, p, which, count // r, r).reshape(-1)


def test_normal_is_box_muller_of_the_stream():
    # Independent restatement from the Philox words, in Python floats, for a handful of elements.
    seed, layer, p = 0x1234567812345678, 7, 11
    z = _normals(seed, layer, p, 1, 64)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for e in (0, 1, 2, 3, 17, 42, 63):
        x = oracle.philox4x32_10([e >> 2, p, layer, 1], key)
        lane = e & 3
        xa, xb = int(x[(lane >> 1) * 2]), int(x[(lane >> 1) * 2 + 1])
        u1 = ((xa >> 9) + 1) * 2.0 ** -23
        u2 = (xb >> 9) * 2.0 ** -23
        rho = math.sqrt(-2.0 * math.log(u1))
        want = rho * (math.sin(2 * math.pi * u2) if lane & 1 else math.cos(2 * math.pi * u2))
        assert z[e] == float(np.float32(want))


def test_normal_moments_and_distribution():
    z = np.concatenate([_normals(1, 0, p, p & 1, 1 << 18) for p in range(16)])   # 4.2M samples
    n = z.size
    assert abs(z.mean()) < 4.0 / math.sqrt(n)
    assert abs(z.var() - 1.0) < 4.0 * math.sqrt(2.0 / n)
    assert abs(stats.skew(z)) < 4.0 * math.sqrt(6.0 / n)
    assert abs(stats.kurtosis(z, fisher=False) - 3.0) < 4.0 * math.sqrt(24.0 / n)
    assert np.abs(z).max() <= 5.65                    # sqrt(-2 ln 2^-23) = 5.647
    # Kolmogorov-Smirnov against the exact normal CDF on a subsample
    d, pval = stats.kstest(z[:200000], "norm")
    assert pval > 1e-3, (d, pval)


def test_factor_entries_are_uncorrelated_across_lanes_members_and_factors():
    a = _normals(3, 2, 0, 0, 1 << 16)
    b = _normals(3, 2, 0, 1, 1 << 16)
    a2 = _normals(3, 2, 1, 0, 1 << 16)
    a3 = _normals(4, 2, 0, 0, 1 << 16)
    a4 = _normals(3, 5, 0, 0, 1 << 16)
    tol = 4.5 / math.sqrt(a.size)
    for u, v in ((a, b), (a, a2), (a, a3), (a, a4), (a[0::2], a[1::2]), (a[0::4], a[2::4]), (a[:-1], a[1:])):
        assert abs(np.mean(u * v)) < tol * (1 if u.size == a.size else 2)


def test_element_map_is_row_major_over_rank_columns():
    # element (j,k) has flat index j*r+k: the r=4 factor is the r=1 stream reshaped
    flat = _normals(9, 1, 5, 0, 64)
    f4 = oracle.noise_factor(9, 1, 5, 0, 16, 4)
    assert np.array_equal(f4.reshape(-1), flat)
    f16 = oracle.noise_factor(9, 1, 5, 0, 4, 16)
    assert np.array_equal(f16.reshape(-1), flat)


@pytest.mark.parametrize("r,kurt", [(1, 9.0), (4, 4.5), (16, 3.375)])
def test_low_rank_matrix_has_identity_covariance(r, kurt):
    # Cov(vec E) = I for E = A B^T / sqrt r (Assumption 1 and the analysis section); kurtosis 3 + 6/r.
    m, n, P = 12, 10, 6000
    E = np.zeros((P, m, n))
    for p in range(P):
        A = oracle.noise_factor(11, 0, p, 0, m, r)
        B = oracle.noise_factor(11, 0, p, 1, n, r)
        E[p] = A @ B.T / math.sqrt(r)
    V = E.reshape(P, -1)
    C = V.T @ V / P
    assert np.abs(np.diag(C) - 1.0).max() < 6.0 * math.sqrt((kurt - 1.0) / P)
    off = C - np.diag(np.diag(C))
    assert np.abs(off).max() < 6.0 / math.sqrt(P)
    k = np.mean(V ** 4) / np.mean(V ** 2) ** 2
    assert abs(k - kurt) < 0.15 * kurt

"""Pins for the oracle's integer path (CPU only)."""
import numpy as np
import pytest

import oracle
import workloads


def _plain_scaled(X, W, shift):
    acc = X.astype(np.int64) @ W.astype(np.int64).T
    return np.clip(np.floor_divide(acc, 1 << shift), -127, 127).astype(np.int8)


def test_zero_table_reduces_to_the_plain_scaled_matmul():
    # u @ M := I8(u M / (16 sqrt n)), a shift by 4 + d for n = 4^d (Matrix Multiplication)
    n, m, N, T = 64, 48, 6, 2            # n = 4^3 -> shift 7
    X = workloads.int8_activations(1, 30, (N * T, n))
    W = workloads.int8_matrix(1, 31, (m, n))
    table = np.zeros(1 << 10, dtype=np.int8)
    Y = oracle.perturbed_linear_i8(X, W, np.arange(N), T, 3, 5, oracle.ANTITHETIC, 8, 7, table)
    assert np.array_equal(Y, _plain_scaled(X, W, 7))
    # 16 sqrt(64) = 128 = 2^7: the shift is the stated division, floored
    acc = X.astype(np.int64) @ W.astype(np.int64).T
    assert np.array_equal(Y, np.clip(np.floor(acc / (16 * np.sqrt(n))), -127, 127).astype(np.int8))


def test_perturbed_matmul_step_by_step_in_python():
    n, m, N, T, L = 16, 12, 8, 1, 12
    sigma_shift, out_shift = 4 + 2, 4 + 2
    X = workloads.int8_activations(2, 30, (N * T, n))
    W = workloads.int8_matrix(2, 31, (m, n))
    table = workloads.noise_table(2, L)
    Y = oracle.perturbed_linear_i8(X, W, np.arange(N), T, 9, 1234, oracle.ANTITHETIC, sigma_shift, out_shift, table)
    mask = (1 << L) - 1
    for i in range(N):
        p, sign = i >> 1, 1 - 2 * (i & 1)
        x = oracle.philox4x32_10([0, p, 9, 2], [1234, 0])
        offa, offb = int(x[0]) & mask, int(x[1]) & mask
        A = np.array([int(table[(offa + j) & mask]) for j in range(m)])
        B = np.array([int(table[(offb + l) & mask]) for l in range(n)])
        u = X[i].astype(int)
        t = sign * int(u @ B)
        for j in range(m):
            acc = int(u @ W[j].astype(int))
            pert = (t * int(A[j])) >> sigma_shift           # Python >> floors
            y = max(-127, min(127, (acc + pert) >> out_shift))
            assert Y[i, j] == y


def test_shift_is_floor_so_a_huge_sigma_shift_leaves_minus_one_or_zero():
    n, m, N = 16, 8, 16
    X = workloads.int8_activations(3, 30, (N, n))
    W = np.zeros((m, n), dtype=np.int8)
    table = workloads.noise_table(3, 10)
    Y = oracle.perturbed_linear_i8(X, W, np.arange(N), 1, 0, 0, 0, 31, 0, table)
    assert set(np.unique(Y)) <= {-1, 0} and (Y == -1).any() and (Y == 0).any()


def test_outputs_saturate_and_never_hit_minus_128():
    n, m = 256, 32
    X = np.full((4, n), 127, dtype=np.int8)
    W = np.full((m, n), -127, dtype=np.int8)
    W[: m // 2] = 127
    table = workloads.noise_table(4, 10)
    Y = oracle.perturbed_linear_i8(X, W, np.arange(4), 1, 0, 0, 0, 8, 8, table)
    assert Y.min() == -127 and Y.max() == 127


def test_antithetic_partners_agree_under_a_zero_table_and_differ_otherwise():
    n, m, N = 64, 64, 8
    X = workloads.int8_activations(5, 30, (N, n))
    X[1::2] = X[0::2]
    W = workloads.int8_matrix(5, 31, (m, n))
    Yz = oracle.perturbed_linear_i8(X, W, np.arange(N), 1, 0, 0, oracle.ANTITHETIC, 5, 7, np.zeros(1024, np.int8))
    assert np.array_equal(Yz[0::2], Yz[1::2])
    Y = oracle.perturbed_linear_i8(X, W, np.arange(N), 1, 0, 0, oracle.ANTITHETIC, 5, 7, workloads.noise_table(5, 10))
    assert not np.array_equal(Y[0::2], Y[1::2])


def test_overflow_is_reported():
    n = 4096
    X = np.full((1, n), 127, dtype=np.int8)
    W = np.full((1, n), 127, dtype=np.int8)
    table = np.full(1024, 127, dtype=np.int8)
    with pytest.raises(OverflowError):
        oracle.perturbed_linear_i8(X, W, np.arange(1), 1, 0, 0, 0, 0, 0, table)


def test_integer_update_is_the_matrix_product_and_moves_one_bin():
    m, n, P, L = 10, 14, 32, 12
    table = workloads.noise_table(6, L)
    F = workloads.rng(6, 40).integers(-1, 2, size=P).astype(np.int8)
    W = workloads.int8_matrix(6, 31, (m, n))
    W[0, 0], W[0, 1] = 127, -127
    mask = (1 << L) - 1
    A = np.zeros((P, m), dtype=np.int64)
    B = np.zeros((P, n), dtype=np.int64)
    for p in range(P):
        offa, offb = oracle.i8_offsets(17, 2, p, L)
        A[p] = table[(offa + np.arange(m)) & mask]
        B[p] = table[(offb + np.arange(n)) & mask]
    E_want = (F.astype(np.int64)[:, None] * A).T @ B                # (diag(F) A)^T B
    thr = int(np.median(np.abs(E_want)))
    Wn, E = oracle.es_update_i8(W, F, 2, 17, thr, table)
    assert np.array_equal(E, E_want)
    step = np.where(np.abs(E_want) >= thr, np.sign(E_want), 0)
    assert np.array_equal(Wn, np.clip(W.astype(np.int64) + step, -127, 127).astype(np.int8))
    assert np.abs(Wn.astype(int) - W.astype(int)).max() == 1
    # threshold 0 moves every element whose E is non-zero by exactly one bin (before saturation)
    W0 = np.zeros((m, n), dtype=np.int8)
    Wn0, _ = oracle.es_update_i8(W0, F, 2, 17, 0, table)
    assert np.array_equal(Wn0, np.sign(E_want).astype(np.int8))


def test_threshold_reading_fraction_updated_is_about_alpha():
    # thr = I32(16 Phi^-1(1 - alpha/2)) * I32(16 sqrt K): with F = +-1 the share of |E| >= thr is near alpha.
    from scipy import stats
    m, n, P, L, alpha = 64, 64, 4096, 16, 0.5
    table = workloads.noise_table(8, L)
    F = (workloads.rng(8, 40).integers(0, 2, size=P) * 2 - 1).astype(np.int8)
    thr = int(16 * stats.norm.ppf(1 - alpha / 2)) * int(16 * np.sqrt(P))
    assert thr == 10 * 1024
    Wn, E = oracle.es_update_i8(np.zeros((m, n), np.int8), F, 0, 1, thr, table)
    frac = np.mean(np.abs(E) >= thr)
    assert abs(frac - alpha) < 0.06
    assert np.mean(Wn != 0) == frac

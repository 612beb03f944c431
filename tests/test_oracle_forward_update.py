"""Pins for the oracle's forward and update against what the paper and linear algebra fix (CPU only)."""
import math

import numpy as np
import pytest

import oracle
import workloads


def _E(seed, layer, p, m, n, r):
    A = oracle.noise_factor(seed, layer, p, 0, m, r)
    B = oracle.noise_factor(seed, layer, p, 1, n, r)
    return A @ B.T / math.sqrt(r)


@pytest.mark.parametrize("m,n,r,T,anti", [(5, 7, 1, 1, False), (10, 12, 4, 3, True), (6, 9, 16, 2, True),
                                          (8, 8, 2, 1, False)])
def test_forward_equals_numpy_on_explicitly_perturbed_weights(m, n, r, T, anti):
    # Section 4.2 left-hand side, with numpy doing the product on W + sigma E_i.
    N, seed, layer, sigma = 6, 21, 3, 0.3
    W, X = workloads.linear_layer(5, m, n, N * T, bf16=False)
    flags = oracle.ANTITHETIC if anti else 0
    Y = oracle.perturbed_linear(X, W, np.arange(N), T, r, layer, seed, flags, sigma)
    for i in range(N):
        p, sign = ((i >> 1), 1 - 2 * (i & 1)) if anti else (i, 1)
        Wi = W.astype(np.float64) + sigma * sign * _E(seed, layer, p, m, n, r)
        want = X[i * T:(i + 1) * T].astype(np.float64) @ Wi.T
        np.testing.assert_allclose(Y[i * T:(i + 1) * T], want, rtol=1e-12, atol=1e-12)


def test_factored_form_equals_explicit_form():
    # u (M + sigma E)^T = u M^T + (sigma / sqrt r)(u B) A^T  (Section 4.2)
    for (m, n, r, T, anti) in [(16, 24, 1, 2, True), (9, 5, 4, 1, False), (7, 33, 16, 3, True)]:
        N = 8
        W, X = workloads.linear_layer(2, m, n, N * T, bf16=False)
        flags = oracle.ANTITHETIC if anti else 0
        a = oracle.perturbed_linear(X, W, np.arange(N), T, r, 1, 99, flags, 0.05)
        b = oracle.perturbed_linear_factored(X, W, np.arange(N), T, r, 1, 99, flags, 0.05)
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-12)


def test_sigma_zero_is_a_plain_matmul_and_member_subsets_are_consistent():
    W, X = workloads.linear_layer(3, 11, 13, 10, bf16=False)
    Y = oracle.perturbed_linear(X, W, np.arange(10), 1, 4, 0, 1, 0, 0.0)
    np.testing.assert_allclose(Y, X.astype(np.float64) @ W.astype(np.float64).T, rtol=1e-13, atol=1e-13)
    full = oracle.perturbed_linear(X, W, np.arange(10), 1, 4, 0, 1, 0, 0.2)
    sel = np.array([7, 2, 9])
    part = oracle.perturbed_linear(X[sel], W, sel, 1, 4, 0, 1, 0, 0.2)
    assert np.array_equal(part, full[sel])


def test_antithetic_partners_mirror_around_the_unperturbed_output():
    N, T, m, n, r = 8, 2, 6, 10, 4
    W, X = workloads.linear_layer(4, m, n, N * T, bf16=False)
    X = workloads.pair_shared_rows(X, T)
    Y = oracle.perturbed_linear(X, W, np.arange(N), T, r, 2, 5, oracle.ANTITHETIC, 0.5)
    Y0 = X.astype(np.float64) @ W.astype(np.float64).T
    Ym = Y.reshape(N // 2, 2, T, m)
    Y0m = Y0.reshape(N // 2, 2, T, m)
    np.testing.assert_allclose(Ym[:, 0] + Ym[:, 1], 2 * Y0m[:, 0], rtol=1e-12, atol=1e-12)
    assert np.abs(Ym[:, 0] - Ym[:, 1]).min() > 0


def test_noise_depends_on_seed_layer_and_member():
    W, X = workloads.linear_layer(4, 6, 6, 4, bf16=False)
    X[:] = X[0]
    base = oracle.perturbed_linear(X, W, np.arange(4), 1, 1, 0, 0, 0, 1.0)
    assert len({tuple(np.round(row, 9)) for row in base}) == 4
    assert not np.allclose(base, oracle.perturbed_linear(X, W, np.arange(4), 1, 1, 0, 1, 0, 1.0))
    assert not np.allclose(base, oracle.perturbed_linear(X, W, np.arange(4), 1, 1, 1, 0, 0, 1.0))


# ------------------------------------------------------------------------------------------ update
@pytest.mark.parametrize("m,n,r,N,anti", [(6, 9, 1, 10, False), (8, 5, 4, 12, True), (4, 4, 16, 6, True)])
def test_update_equals_sum_of_outer_products_and_gemm_form(m, n, r, N, anti):
    seed, layer, alpha = 77, 4, 0.37
    f = workloads.raw_fitness(1, N).astype(np.float64)
    flags = oracle.ANTITHETIC if anti else 0
    W = workloads.linear_layer(1, m, n, 1, bf16=False)[0]
    Wn, dW = oracle.es_update(W, f, r, layer, seed, flags, alpha)
    # (a) boxed update: (alpha/N) sum_i f_i E_i with E_i = sign_i A_p B_p^T / sqrt r
    want = np.zeros((m, n))
    for i in range(N):
        p, sign = ((i >> 1), 1 - 2 * (i & 1)) if anti else (i, 1)
        want += f[i] * sign * _E(seed, layer, p, m, n, r)
    want *= alpha / N
    np.testing.assert_allclose(dW, want, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(Wn, W.astype(np.float64) + want, rtol=1e-12, atol=1e-13)
    # (b) one matrix product (diag(f) A)^T B over the stacked factors (Section 4.2, last sentences)
    P = N // 2 if anti else N
    g = (f[0::2] - f[1::2]) if anti else f
    At = np.concatenate([oracle.noise_factor(seed, layer, p, 0, m, r).T for p in range(P)], axis=0)   # [P*r, m]
    Bt = np.concatenate([oracle.noise_factor(seed, layer, p, 1, n, r).T for p in range(P)], axis=0)   # [P*r, n]
    gk = np.repeat(g, r)
    gemm = (gk[:, None] * At).T @ Bt * (alpha / (N * math.sqrt(r)))
    np.testing.assert_allclose(dW, gemm, rtol=1e-11, atol=1e-13)


def test_update_blocks_tile_the_full_matrix():
    f = workloads.raw_fitness(2, 8)
    full = oracle.es_update_block(f, 4, 0, 3, 0, 0.1, 0, 10, 0, 14)
    blk = oracle.es_update_block(f, 4, 0, 3, 0, 0.1, 3, 9, 5, 12)
    np.testing.assert_allclose(blk, full[3:9, 5:12], rtol=1e-13, atol=1e-15)


def test_antithetic_pairs_cancel_exactly_under_constant_fitness():
    f = np.full(16, 3.25)
    dW = oracle.es_update_block(f, 4, 1, 2, oracle.ANTITHETIC, 0.5, 0, 9, 0, 7)
    assert np.all(dW == 0.0)
    # and with constant fitness inside each pair only
    f2 = np.repeat(workloads.raw_fitness(0, 8), 2)
    assert np.all(oracle.es_update_block(f2, 1, 1, 2, oracle.ANTITHETIC, 0.5, 0, 9, 0, 7) == 0.0)


@pytest.mark.parametrize("N,r,m,n", [(1, 1, 8, 9), (3, 1, 8, 9), (2, 2, 8, 9), (3, 4, 8, 9), (1, 16, 8, 9)])
def test_update_rank_is_min_Nr_m_n(N, r, m, n):
    # "the overall EGGROLL matrix parameter update has rank min(Nr, m, n) almost surely"
    f = 1.0 + np.arange(N, dtype=np.float64)
    dW = oracle.es_update_block(f, r, 0, 8, 0, 1.0, 0, m, 0, n)
    s = np.linalg.svd(dW, compute_uv=False)
    assert int((s > 1e-10 * s[0]).sum()) == min(N * r, m, n)


def test_linear_fitness_recovers_its_gradient():
    # f(W) = <G, W>: E[(1/N) sum_i E_i f(M + sigma E_i)] = sigma G because Cov(vec E) = I.
    m, n, r, N, sigma, alpha = 4, 5, 2, 40000, 0.1, 1.0
    G = workloads.rng(5).standard_normal((m, n))
    M = workloads.rng(6).standard_normal((m, n))
    f = np.zeros(N)
    for i in range(N):
        f[i] = np.sum(G * (M + sigma * _E(12, 0, i, m, n, r)))
    dW = oracle.es_update_block(f - f.mean(), r, 0, 12, 0, alpha, 0, m, 0, n)
    # per-entry standard error ~ sigma * ||G||_F / sqrt N
    tol = 5.0 * sigma * np.linalg.norm(G) / math.sqrt(N)
    assert np.abs(dW - alpha * sigma * G).max() < tol
    assert np.abs(dW - alpha * sigma * G).max() < 0.25 * np.abs(sigma * G).max()


# ----------------------------------------------------------------------------- element-wise function after the layer
def test_activation_matches_independent_definitions():
    """tanh against its exponential form, GELU against x Phi(x) with the standard library's normal distribution
    function and against torch's CPU routine, relu against the positive part."""
    import math
    import statistics
    import torch
    x = np.concatenate([np.linspace(-6, 6, 241), [0.0, 1e-9, -1e-9, 30.0, -30.0]])
    t = oracle.activation(x, oracle.ACT_TANH)
    np.testing.assert_allclose(t, np.expm1(2 * x) / (np.exp(2 * x) + 1), rtol=1e-12, atol=1e-15)
    g = oracle.activation(x, oracle.ACT_GELU)
    phi = np.array([statistics.NormalDist().cdf(v) for v in x])
    np.testing.assert_allclose(g, x * phi, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(g, torch.nn.functional.gelu(torch.tensor(x, dtype=torch.float64)).numpy(), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(g - oracle.activation(-x, oracle.ACT_GELU), x, rtol=1e-12, atol=1e-12)   # x Phi(x) + x Phi(-x) = x
    assert abs(g[np.argmin(np.abs(x - 1.0))] - 0.8413447460685429) < 1e-12                               # Phi(1) from tables
    r = oracle.activation(x, oracle.ACT_RELU)
    assert np.array_equal(r, np.where(x > 0, x, 0.0))
    assert oracle.activation(x, 0) is not None and np.array_equal(oracle.activation(x, 0), x)
    assert math.isclose(float(oracle.activation(np.array([0.5]), oracle.ACT_TANH)[0]), math.tanh(0.5), rel_tol=1e-15)


def test_forward_with_activation_is_the_function_of_the_plain_forward():
    g = np.random.default_rng(5)
    W = g.standard_normal((6, 8)) / 3
    X = g.standard_normal((8, 8))
    args = (X, W, np.arange(4), 2, 2, 3, 11)
    base = oracle.perturbed_linear(*args, oracle.ANTITHETIC, 0.3)
    for act, fn in ((oracle.ACT_TANH, np.tanh), (oracle.ACT_RELU, lambda v: np.maximum(v, 0))):
        np.testing.assert_allclose(oracle.perturbed_linear(*args, oracle.ANTITHETIC | act, 0.3), fn(base), rtol=1e-14)
        np.testing.assert_allclose(oracle.perturbed_linear_factored(*args, oracle.ANTITHETIC | act, 0.3), fn(base), rtol=1e-10)
    gl = oracle.perturbed_linear(*args, oracle.ANTITHETIC | oracle.ACT_GELU, 0.3)
    assert np.all(np.abs(gl) <= np.abs(base) + 1e-15) and np.all((gl >= -0.17) | (base > 0))   # min of x Phi(x) is -0.16997
    big = base > 4
    np.testing.assert_allclose(gl[big], base[big], rtol=1e-4)


def test_library_matmul_form_of_the_explicit_forward_equals_the_loops():
    # perturbed_linear_blas forms W + sigma E_i and applies it with numpy's matrix product (used where the plain loops
    # would take minutes); it has to be the same function as the loop form, activation bits and pair signs included
    W, X = workloads.linear_layer(21, 70, 130, 24, bf16=False)
    members = np.array([3, 4, 7, 10])
    for flags in (0, oracle.ANTITHETIC, oracle.ANTITHETIC | oracle.ACT_GELU, oracle.ACT_TANH):
        for r in (1, 4):
            a = oracle.perturbed_linear(X, W, members, 6, r, 9, 77, flags, 0.3)
            b = oracle.perturbed_linear_blas(X, W, members, 6, r, 9, 77, flags, 0.3)
            assert np.abs(a - b).max() < 1e-12
    base = X.astype(np.float64) @ W.astype(np.float64).T
    assert np.abs(oracle.perturbed_linear_blas(X, W, members, 6, 2, 9, 77, 0, 0.0) - base).max() < 1e-12


def test_token_log_likelihood_is_the_log_softmax_at_the_target():
    from scipy.special import log_softmax
    g = workloads.rng(22, 1)
    Z = g.standard_normal((17, 101)) * 3.0
    t = g.integers(0, 101, size=17)
    t[3], t[5] = -1, 101                                      # positions that are not scored
    got = oracle.token_log_likelihood(Z, t)
    want = log_softmax(Z, axis=1)
    for i in range(17):
        assert got[i] == 0.0 if not (0 <= t[i] < 101) else abs(got[i] - want[i, t[i]]) < 1e-12
    # closed forms: constant logits give -log V; adding a constant to a row changes nothing; probabilities sum to one
    assert abs(oracle.token_log_likelihood(np.full((1, 32000), 2.5), [7])[0] + math.log(32000)) < 1e-12
    assert np.abs(oracle.token_log_likelihood(Z + 1000.0, t) - got).max() < 1e-9
    allp = np.array([np.exp(oracle.token_log_likelihood(Z[:1].repeat(101, 0), np.arange(101))).sum()])
    assert abs(allp[0] - 1.0) < 1e-12

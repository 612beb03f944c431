"""Pins for the per-channel int8 / discretised-Adam oracle (appendix "Fine-tuning of Integer Quantised Models"):
closed forms, invariants, brute force on tiny inputs and an independent library optimiser."""
import math

import numpy as np

import oracle
import workloads
from oracle import q8


def test_bf16_round_is_nearest_even_on_the_8_bit_significand():
    # 1 + 2^-8 lies half way between 1 and 1 + 2^-7: ties go to the even significand (1.0); 1 + 3*2^-8 goes up
    assert q8.bf16_round(np.float32(1 + 2.0 ** -8)) == np.float32(1.0)
    assert q8.bf16_round(np.float32(1 + 3 * 2.0 ** -8)) == np.float32(1 + 2.0 ** -6)
    assert q8.bf16_round(np.float32(1 + 2.0 ** -8 + 2.0 ** -20)) == np.float32(1 + 2.0 ** -7)
    x = workloads.rng(31, 0).standard_normal(4096).astype(np.float32)
    r = q8.bf16_round(x)
    assert np.all((r.view(np.uint32) & 0xFFFF) == 0)
    assert np.all(np.abs(r - x) <= np.abs(x) * 2.0 ** -8)
    assert np.array_equal(q8.bf16_round(r), r)


def test_quantisation_error_scale_and_symmetries():
    g = workloads.rng(31, 1)
    W = (g.standard_normal((37, 53)) * np.exp(g.standard_normal((37, 1)))).astype(np.float32)
    W[5] = 0.0
    Q, s = q8.quantize_per_channel(W, 1e-8)
    assert Q.dtype == np.int8 and np.abs(Q.astype(int)).max() <= 127
    # the stored scale is the bf16 value of absmax / 127 (eps for a zero channel)
    want = np.maximum(np.abs(W).max(axis=1) / 127.0, 1e-8)
    assert np.all(np.abs(s - want) <= want * 2.0 ** -8)
    assert np.all((s.view(np.uint32) & 0xFFFF) == 0)
    assert np.all(Q[5] == 0)
    # nearest lattice point with the stored scale: error at most half a bin (no clipping loss: |W|/s <= 127.25)
    err = np.abs(q8.dequantize(Q, s) - W.astype(np.float64))
    assert np.all(err <= 0.5 * s[:, None].astype(np.float64) * (1 + 1e-6))
    # every non-zero channel uses the end of the range
    nz = np.abs(W).max(axis=1) > 0
    assert np.all(np.abs(Q[nz].astype(int)).max(axis=1) == 127)
    # odd symmetry, and invariance of the codes under a power-of-two rescaling of the matrix
    Qn, sn = q8.quantize_per_channel(-W, 1e-8)
    assert np.array_equal(Qn, -Q) and np.array_equal(sn, s)
    Q4, s4 = q8.quantize_per_channel(4.0 * W, 1e-8)
    assert np.array_equal(Q4[nz], Q[nz]) and np.array_equal(s4[nz], 4.0 * s[nz])


def test_quantisation_round_half_to_even():
    # one channel with absmax 127 -> scale exactly 1; halves go to the even integer
    W = np.array([[127.0, 0.5, 1.5, 2.5, -0.5, -1.5, 126.5]], dtype=np.float32)
    Q, s = q8.quantize_per_channel(W)
    assert s[0] == 1.0
    assert Q[0].tolist() == [127, 0, 2, 2, 0, -2, 126]


def test_forward_reduces_to_scaled_matmul_and_to_the_plain_perturbed_layer():
    g = workloads.rng(31, 2)
    m, n, N, T, r = 12, 20, 6, 3, 2
    W = g.standard_normal((m, n)).astype(np.float32)
    Q, s = q8.quantize_per_channel(W)
    X = g.standard_normal((N * T, n))
    members = np.arange(N)
    s_x = 0.75
    y0 = q8.perturbed_linear_q8(X, Q, s, s_x, members, T, r, 3, 9, oracle.ANTITHETIC, 0.0)
    np.testing.assert_allclose(y0, (X * s_x) @ q8.dequantize(Q, s).T, rtol=1e-12, atol=1e-12)
    # unit scales: the layer of Section 4.2 applied to the integer matrix
    y1 = q8.perturbed_linear_q8(X, Q, np.ones(m), 1.0, members, T, r, 3, 9, oracle.ANTITHETIC, 0.3)
    want = oracle.perturbed_linear(X, Q.astype(np.float64), members, T, r, 3, 9, oracle.ANTITHETIC, 0.3)
    np.testing.assert_allclose(y1, want, rtol=1e-11, atol=1e-11)


def test_forward_brute_force_effective_matrix_with_scale_noise():
    g = workloads.rng(31, 3)
    m, n, N, T, r = 5, 8, 4, 2, 1
    Q = g.integers(-127, 128, size=(m, n)).astype(np.int8)
    s = q8.bf16_round((0.01 + 0.02 * g.random(m)).astype(np.float32))
    X = g.standard_normal((N * T, n))
    sigma, sigma_s, s_x, seed, lid = 0.8, 0.003, 1.25, 11, 6
    y = q8.perturbed_linear_q8(X, Q, s, s_x, np.arange(N), T, r, lid, seed, oracle.ANTITHETIC, sigma, sigma_s)
    for i in range(N):
        p, sign = i // 2, (1.0 if i % 2 == 0 else -1.0)
        A = oracle.noise_factor(seed, lid, p, 0, m, r)
        B = oracle.noise_factor(seed, lid, p, 1, n, r)
        e = oracle.noise_factor(seed, lid, p, 3, m + 1, 1)[:, 0]
        Weff = (Q.astype(np.float64) + sign * sigma * (A @ B.T) / math.sqrt(r)) * (s + sign * sigma_s * e[:m])[:, None]
        want = (X[i * T:(i + 1) * T] * (s_x + sign * sigma_s * e[m])) @ Weff.T
        np.testing.assert_allclose(y[i * T:(i + 1) * T], want, rtol=1e-11, atol=1e-12)
    # antithetic partners see mirrored scales: their outputs average to the unperturbed one up to second order
    y_mid = q8.perturbed_linear_q8(X[:T], Q, s, s_x, [0], T, r, lid, seed, 0, 0.0)
    X2 = np.concatenate([X[:T], X[:T]])
    y_pair = q8.perturbed_linear_q8(X2, Q, s, s_x, [0, 1], T, r, lid, seed, oracle.ANTITHETIC, 1e-4, 1e-6)
    assert np.abs(0.5 * (y_pair[:T] + y_pair[T:]) - y_mid).max() < 1e-6 * np.abs(y_mid).max()


def test_scale_gradient_definition_cancellation_and_moments():
    m, N, seed, lid = 6, 64, 4, 2
    f = workloads.rng(31, 4).standard_normal(N)
    g = q8.es_scale_gradient(f, m, lid, seed, oracle.ANTITHETIC)
    want = np.zeros(m + 1)
    for p in range(N // 2):
        want += (f[2 * p] - f[2 * p + 1]) * oracle.noise_factor(seed, lid, p, 3, m + 1, 1)[:, 0]
    np.testing.assert_allclose(g, want / N, rtol=1e-12, atol=1e-14)
    # constant fitness: antithetic partners cancel exactly
    assert np.all(q8.es_scale_gradient(np.full(N, 3.0), m, lid, seed, oracle.ANTITHETIC) == 0.0)
    # fitness equal to one coordinate of the noise recovers that coordinate (law of large numbers)
    Nb = 4096
    e = np.stack([oracle.noise_factor(seed, lid, p, 3, m + 1, 1)[:, 0] for p in range(Nb)])
    gb = q8.es_scale_gradient(e[:, 2], m, lid, seed, 0)
    assert abs(gb[2] - 1.0) < 0.1 and np.abs(np.delete(gb, 2)).max() < 0.08
    # the matrix pathway is the boxed update without the step size
    blk = q8.es_gradient_block(f, 2, lid, seed, oracle.ANTITHETIC, 0, 4, 0, 5)
    np.testing.assert_allclose(blk, oracle.es_update_block(f, 2, lid, seed, oracle.ANTITHETIC, 0.5, 0, 4, 0, 5) * 2.0, rtol=1e-13)


def test_adam_first_step_closed_form_and_fixed_point():
    g = np.array([0.3, -2.0, 1e-3, 0.0, 5.0], dtype=np.float32)
    z = np.zeros_like(g)
    lr, b1, b2, eps = 0.01, 0.9, 0.999, 1e-8
    u, m1, v1 = q8.adam_proposal(g, z, z, 1, lr, b1, b2, eps)
    # t = 1 from zero moments: m_hat = g, v_hat = g^2, so u = lr g / (|g| + eps) = lr sign(g)
    np.testing.assert_allclose(u, lr * np.sign(g), rtol=2.0 ** -8)
    np.testing.assert_allclose(m1, 0.1 * g, rtol=2.0 ** -8)
    np.testing.assert_allclose(v1, 0.001 * g * g, rtol=2.0 ** -7)
    # moments already at their fixed point (m = g, v = g^2) stay there for a constant gradient
    gg = q8.bf16_round(g)
    u2, m2, v2 = q8.adam_proposal(gg, gg, q8.bf16_round(gg * gg), 10 ** 6, lr, b1, b2, eps)
    np.testing.assert_allclose(m2, gg, rtol=2.0 ** -7)
    np.testing.assert_allclose(u2[gg != 0], lr * np.sign(gg[gg != 0]), rtol=2.0 ** -6)


def test_adam_matches_an_independent_library_optimiser():
    """torch.optim.Adam (maximize=True, fp32 state) over several steps; the oracle keeps its moments in bf16, so the
    proposals agree to bf16 accuracy.  A wrong bias correction, a misplaced epsilon or a wrong sign would be far
    outside that band."""
    import torch
    g = workloads.rng(31, 5)
    lr, b1, b2, eps = 3e-3, 0.9, 0.95, 1e-8
    n = 512
    p = torch.zeros(n, dtype=torch.float32, requires_grad=True)
    opt = torch.optim.Adam([p], lr=lr, betas=(b1, b2), eps=eps, maximize=True)
    m = np.zeros(n, np.float32)
    v = np.zeros(n, np.float32)
    scale = np.where(np.arange(n) < 8, 1e-8, 1.0)          # a few gradients of the size of eps: its placement shows
    for t in range(1, 7):
        grad = (g.standard_normal(n) * scale).astype(np.float32)
        before = p.detach().clone().numpy()
        p.grad = torch.from_numpy(grad.copy())
        opt.step()
        u_lib = p.detach().numpy() - before
        u, m, v = q8.adam_proposal(grad, m, v, t, lr, b1, b2, eps)
        np.testing.assert_allclose(u, u_lib, rtol=0.03, atol=lr * 5e-3)   # moments near zero lose relative accuracy in bf16


def test_unit_step_threshold_fraction_sign_and_limits():
    g = workloads.rng(31, 6)
    u = q8.bf16_round((1e-3 * g.standard_normal(200_000) + 4e-4).astype(np.float32))
    for tau in (0.5, 1.0, 2.0):
        d = q8.unit_step(u, tau)
        frac = np.mean(d != 0)
        expect = math.erfc(tau / math.sqrt(2.0))             # P(|z| >= tau) for a Gaussian
        assert abs(frac - expect) < 0.01
        z = (u.astype(np.float64) - u.astype(np.float64).mean()) / (u.astype(np.float64).std() + 1e-8)
        clear = np.abs(np.abs(z) - tau) > 1e-3                # away from the threshold the decision is unambiguous
        assert np.array_equal(d[clear], (np.sign(z) * (np.abs(z) >= tau)).astype(np.int8)[clear])
    assert np.all(q8.unit_step(u, 1e9) == 0)
    d0 = q8.unit_step(u, 0.0)
    assert np.all(np.abs(d0[u != np.float32(u.astype(np.float64).mean())]) == 1)
    # shifting all proposals by a constant that bf16 represents exactly does not change the step
    u2 = np.array([0.25, 0.5, 0.75, 1.0, 4.0], dtype=np.float32)
    assert np.array_equal(q8.unit_step(u2, 1.0), q8.unit_step(u2 + np.float32(8.0), 1.0))
    assert q8.unit_step(u2, 1.0).tolist() == [0, 0, 0, 0, 1]


def test_adam_step_q8_stays_on_the_lattice_and_saturates():
    g = workloads.rng(31, 7)
    Q = g.integers(-127, 128, size=(16, 32)).astype(np.int8)
    Q[0, :4] = [127, 127, -127, -127]
    grad = g.standard_normal((16, 32)).astype(np.float32)
    grad[0, :4] = [50.0, -50.0, 50.0, -50.0]
    z = np.zeros((16, 32), np.float32)
    Qn, m1, v1, u, delta = q8.adam_step_q8(Q, grad, z, z, 1, 1e-2, 0.9, 0.999, 1e-8, 0.5)
    assert Qn.dtype == np.int8 and np.abs(Qn.astype(int)).max() <= 127
    assert np.all(np.abs(Qn.astype(int) - Q.astype(int)) <= 1)
    assert Qn[0, :4].tolist() == [127, 126, -126, -127]
    moved = delta != 0
    assert np.array_equal(np.sign(delta[moved]), np.sign((u - u.mean())[moved]).astype(np.int8))
    # bf16 leaf: one step moves every entry by about lr along the sign of its gradient
    p0 = q8.bf16_round(g.standard_normal(64).astype(np.float32) * 0.01)
    gr = g.standard_normal(64).astype(np.float32)
    p1, _, _ = q8.adam_step_bf16(p0, gr, np.zeros(64, np.float32), np.zeros(64, np.float32), 1, 1e-3, 0.9, 0.999, 1e-8)
    np.testing.assert_allclose(p1 - p0, 1e-3 * np.sign(gr), rtol=0.05, atol=2e-4)

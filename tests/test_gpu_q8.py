"""Parity of the per-channel int8 / discretised-Adam entry points (include/egr_q8.h) with the CPU oracle.

Integer results (codes, unit steps, bf16 bit patterns of the moments) are compared bit for bit; the forward and the
gradient estimates within the bf16-operand tolerance (relative Frobenius error 1e-2) and the fp32 one (1e-5)."""
import numpy as np
import pytest

import oracle
import workloads
from oracle import q8
from util import rel_fro

pytestmark = pytest.mark.gpu


def _bf16_tensor(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda().to(torch.bfloat16)


def _np(t):
    return t.float().cpu().numpy()


@pytest.mark.parametrize("m,n,pitch", [(37, 53, 64), (256, 1024, 1024), (5, 8, 16), (130, 2051, 2064)])
def test_quantize_bit_exact(m, n, pitch):
    import torch
    import paper_2511_16652_b200 as egr
    g = workloads.rng(32, m * 131 + n)
    W = (g.standard_normal((m, n)) * np.exp(g.standard_normal((m, 1)))).astype(np.float32)
    W[m // 2] = 0.0
    W[0, 0] = 0.5 * np.abs(W[0]).max()                                    # a tie-prone value
    Qo, so = q8.quantize_per_channel(W, 1e-8)
    Wd = torch.from_numpy(W).cuda()
    Q = torch.full((m, pitch), 99, dtype=torch.int8, device="cuda")
    s = torch.empty(m, dtype=torch.bfloat16, device="cuda")
    egr.egr_q8_quantize(Wd, 1e-8, Q[:, :n], s)
    assert np.array_equal(Q[:, :n].cpu().numpy(), Qo)
    assert np.all(Q[:, n:].cpu().numpy() == 99)                            # the padding is not touched
    assert np.array_equal(_np(s), so)


@pytest.mark.parametrize("m,n,N,T,r,flags,sigma_s,y32", [
    (64, 128, 16, 1, 1, 1, 0.0, False),
    (72, 200, 10, 3, 4, 1, 2e-3, True),          # ragged tile in both directions, scale noise, fp32 output
    (300, 264, 257, 1, 1, 0, 1e-3, False),       # several row tiles, odd member count
    (513, 512, 8, 40, 2, 1, 5e-4, False),        # d_out = 1 mod 4: the input-scale element shares a generator block
    (96, 64, 12, 2, 1, 2, 1e-3, False),          # perturbations switched off: scaled unperturbed inference
])
def test_forward_q8_matches_oracle(m, n, N, T, r, flags, sigma_s, y32):
    import torch
    import paper_2511_16652_b200 as egr
    g = workloads.rng(33, m + 7 * n + N)
    W = (g.standard_normal((m, n)) / np.sqrt(n)).astype(np.float32)
    Qo, so = q8.quantize_per_channel(W)
    X = workloads.round_to_bf16(g.standard_normal((N * T, n)).astype(np.float32))
    s_x, sigma, seed, lid = 0.5, 8.0, 21, 4          # codes are O(40) rms: sigma = 8 is a 20 % perturbation
    pitch = (n + 15) // 16 * 16
    Q = torch.zeros((m, pitch), dtype=torch.int8, device="cuda")
    Q[:, :n] = torch.from_numpy(Qo).cuda()
    s = _bf16_tensor(so)
    Xd = _bf16_tensor(X)
    ldy = (m + 7) // 8 * 8
    Y = torch.zeros((N * T, ldy), dtype=torch.float32 if y32 else torch.bfloat16, device="cuda")
    L = egr.Layer(n, m, N, T, r, layer_id=lid, seed=seed, flags=flags, x_dtype=egr.BF16, w_dtype=egr.I8,
                  y_dtype=egr.F32 if y32 else egr.BF16, ldw=pitch, ldy=ldy)
    ws = egr.Workspace()
    egr.egr_perturbed_linear_q8(L, Xd, Q, s, s_x, sigma, sigma_s, Y, ws)
    assert egr.egr_workspace_status(ws) == 0
    no_pert = bool(flags & 2)
    want = q8.perturbed_linear_q8(X.astype(np.float64), Qo, so, s_x, np.arange(N), T, r, lid, seed, flags & 1,
                                  0.0 if no_pert else sigma, 0.0 if no_pert else sigma_s)
    got = _np(Y)[:, :m]
    assert rel_fro(got, want) < (2e-3 if y32 else 1e-2)
    # the perturbation is really there (and really absent with the flag)
    base = q8.perturbed_linear_q8(X.astype(np.float64), Qo, so, s_x, np.arange(N), T, r, lid, seed, flags & 1, 0.0, 0.0)
    if no_pert:
        assert rel_fro(got, base) < 1e-2
    else:
        assert rel_fro(base, want) > 0.05
    assert np.all(_np(Y)[:, m:] == 0)


def test_forward_q8_scale_noise_alone_is_resolved():
    """sigma = 0, fp32 output: what remains of the difference to the unperturbed layer is the scale noise only."""
    import torch
    import paper_2511_16652_b200 as egr
    m, n, N, T, seed, lid = 128, 256, 32, 2, 3, 9
    g = workloads.rng(33, 99)
    Qo = g.integers(-127, 128, size=(m, n)).astype(np.int8)
    so = q8.bf16_round((0.01 + 0.01 * g.random(m)).astype(np.float32))
    X = workloads.round_to_bf16(g.standard_normal((N * T, n)).astype(np.float32))
    Y = torch.empty((N * T, m), dtype=torch.float32, device="cuda")
    L = egr.Layer(n, m, N, T, 1, layer_id=lid, seed=seed, flags=egr.ANTITHETIC, x_dtype=egr.BF16, w_dtype=egr.I8, y_dtype=egr.F32)
    ws = egr.Workspace()
    egr.egr_perturbed_linear_q8(L, _bf16_tensor(X), torch.from_numpy(Qo).cuda(), _bf16_tensor(so), 1.0, 0.0, 1e-3, Y, ws)
    assert egr.egr_workspace_status(ws) == 0
    want = q8.perturbed_linear_q8(X.astype(np.float64), Qo, so, 1.0, np.arange(N), T, 1, lid, seed, 1, 0.0, 1e-3)
    base = q8.perturbed_linear_q8(X.astype(np.float64), Qo, so, 1.0, np.arange(N), T, 1, lid, seed, 1, 0.0, 0.0)
    assert rel_fro(_np(Y) - base, want - base) < 1e-3


def test_es_gradient_blocks_match_oracle():
    import torch
    import paper_2511_16652_b200 as egr
    m, n, N, r, seed, lid = 300, 520, 96, 4, 6, 2
    f = workloads.rng(34, 1).standard_normal(N).astype(np.float32)
    L = egr.Layer(n, m, N, 1, r, layer_id=lid, seed=seed, flags=egr.ANTITHETIC)
    G = torch.full((m, n), 7.0, dtype=torch.float32, device="cuda")
    ws = egr.Workspace()
    egr.egr_es_gradient(L, torch.from_numpy(f).cuda(), G, ws)
    assert egr.egr_workspace_status(ws) == 0
    got = G.cpu().numpy()
    for (j0, l0) in [(0, 0), (m - 40, n - 40), (128, 256)]:
        want = q8.es_gradient_block(f, r, lid, seed, 1, j0, j0 + 40, l0, l0 + 40)
        assert rel_fro(got[j0:j0 + 40, l0:l0 + 40], want) < 1e-2


@pytest.mark.parametrize("m,N,flags", [(6, 64, 1), (1027, 700, 0), (4096, 2048, 1)])
def test_scale_gradient_matches_oracle(m, N, flags):
    import torch
    import paper_2511_16652_b200 as egr
    seed, lid = 8, 3
    f = workloads.rng(34, m + N).standard_normal(N).astype(np.float32)
    L = egr.Layer(16, m, N, 1, 1, layer_id=lid, seed=seed, flags=flags)
    gd = torch.empty(m + 1, dtype=torch.float32, device="cuda")
    ws = egr.Workspace()
    egr.egr_es_scale_gradient(L, torch.from_numpy(f).cuda(), gd, ws)
    got = gd.cpu().numpy()
    if m <= 1027:
        want = q8.es_scale_gradient(f, m, lid, seed, flags)
        assert rel_fro(got, want) < 1e-5
    else:
        # sampled coordinates (first, last = the input scale, a few inside), each from the definition
        P = N // 2 if flags else N
        gp = (f[0::2] - f[1::2]) if flags else f
        e = np.stack([oracle.noise_factor(seed, lid, p, 3, m + 1, 1)[:, 0] for p in range(P)])
        want = (gp.astype(np.float64)[:, None] * e).sum(axis=0) / N
        assert rel_fro(got, want) < 1e-5
    # constant fitness under antithetic pairs cancels exactly
    if flags:
        egr.egr_es_scale_gradient(L, torch.full((N,), 2.5, device="cuda"), gd, ws)
        assert np.all(gd.cpu().numpy() == 0.0)


@pytest.mark.parametrize("m,n,pitch,tau", [(16, 32, 32, 0.5), (257, 1032, 1040, 1.0), (1024, 4096, 4096, 1.25)])
def test_adam_step_q8_bit_exact_over_three_steps(m, n, pitch, tau):
    import torch
    import paper_2511_16652_b200 as egr
    g = workloads.rng(35, m + n)
    Qo = g.integers(-127, 128, size=(m, n)).astype(np.int8)
    Qo[0, :4] = [127, 127, -127, -127]
    mo = np.zeros((m, n), np.float32)
    vo = np.zeros((m, n), np.float32)
    Q = torch.full((m, pitch), 55, dtype=torch.int8, device="cuda")
    Q[:, :n] = torch.from_numpy(Qo).cuda()
    m1 = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
    v1 = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
    changed = torch.zeros(1, dtype=torch.int64, device="cuda")
    ws = egr.Workspace()
    lr, b1, b2, eps = 1e-2, 0.9, 0.98, 1e-8
    for t in (1, 2, 3):
        grad = (g.standard_normal((m, n)) * np.exp(g.standard_normal((m, 1)))).astype(np.float32)
        grad[0, :4] = [50.0, -50.0, 50.0, -50.0]
        Qn, mo, vo, u, delta = q8.adam_step_q8(Qo, grad, mo, vo, t, lr, b1, b2, eps, tau)
        egr.egr_adam_step_q8(Q[:, :n], torch.from_numpy(grad).cuda(), m1, v1, t, lr, b1, b2, eps, tau, ws, n_changed=changed)
        assert np.array_equal(_np(m1), mo)
        assert np.array_equal(_np(v1), vo)
        assert np.array_equal(Q[:, :n].cpu().numpy(), Qn)
        assert int(changed.item()) == int(np.count_nonzero(Qn != Qo))
        if tau <= 1.0:                 # Adam's proposals are bounded (|u| <~ lr): |z| seldom reaches 2, never at t = 1
            assert 0 < int(changed.item()) < m * n
        Qo = Qn
    assert np.all(Q[:, n:].cpu().numpy() == 55)


def test_adam_step_bf16_bit_exact():
    import torch
    import paper_2511_16652_b200 as egr
    g = workloads.rng(35, 7)
    n = 4097
    po = q8.bf16_round((0.01 * g.random(n)).astype(np.float32))
    mo = np.zeros(n, np.float32)
    vo = np.zeros(n, np.float32)
    p, m1, v1 = _bf16_tensor(po), _bf16_tensor(mo), _bf16_tensor(vo)
    for t in (1, 2, 3, 4):
        grad = g.standard_normal(n).astype(np.float32)
        po, mo, vo = q8.adam_step_bf16(po, grad, mo, vo, t, 1e-4, 0.9, 0.999, 1e-8)
        egr.egr_adam_step_bf16(p, torch.from_numpy(grad).cuda(), m1, v1, t, 1e-4, 0.9, 0.999, 1e-8)
        assert np.array_equal(_np(p), po) and np.array_equal(_np(m1), mo) and np.array_equal(_np(v1), vo)


def test_chain_gradient_to_unit_step_agrees_away_from_the_threshold():
    """Shaped fitness -> gradient estimate (tensor cores, bf16 factors) -> discretised Adam, two steps, each side
    carrying its own state.  The gradient differs from the fp64 oracle within tolerance, so unit steps may differ only
    where |z| is within that tolerance of tau."""
    import torch
    import paper_2511_16652_b200 as egr
    m, n, N, r, lid = 128, 256, 64, 1, 5
    g = workloads.rng(36, 0)
    Qo = g.integers(-100, 101, size=(m, n)).astype(np.int8)
    mo = np.zeros((m, n), np.float32)
    vo = np.zeros((m, n), np.float32)
    Q = torch.from_numpy(Qo).cuda()
    m1 = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
    v1 = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
    G = torch.empty((m, n), dtype=torch.float32, device="cuda")
    ws = egr.Workspace()
    # t = 1: every proposal is +-lr, so tau = 0.5 moves every entry along the sign of its gradient;
    # t = 2: the proposals spread out and tau = 1 cuts through them
    for t, seed, tau, margin in ((1, 12, 0.5, 0.2), (2, 13, 1.0, 0.1)):
        f = oracle.fitness_shape(g.standard_normal(N), oracle.SHAPE_CENTERED_RANK).astype(np.float32)
        G_o = q8.es_gradient_block(f, r, lid, seed, 1, 0, m, 0, n).astype(np.float32)
        Qn_o, mo, vo, u_o, delta_o = q8.adam_step_q8(Qo, G_o, mo, vo, t, 1e-2, 0.9, 0.999, 1e-8, tau)
        L = egr.Layer(n, m, N, 1, r, layer_id=lid, seed=seed, flags=egr.ANTITHETIC)
        egr.egr_es_gradient(L, torch.from_numpy(f).cuda(), G, ws)
        before = Q.cpu().numpy().astype(int)
        egr.egr_adam_step_q8(Q, G, m1, v1, t, 1e-2, 0.9, 0.999, 1e-8, tau, ws)
        delta = Q.cpu().numpy().astype(int) - before
        u64 = u_o.astype(np.float64)
        z = (u64 - u64.mean()) / (u64.std() + 1e-8)
        clear = (np.abs(np.abs(z) - tau) > margin) & (np.abs(G_o) > 1e-2 * np.abs(G_o).mean())
        assert clear.mean() > 0.5
        assert np.mean(delta[clear] != delta_o[clear].astype(int)) < 2e-3
        assert np.mean(delta != delta_o) < 0.05
        assert np.any(delta != 0)
        Qo = Qn_o


def test_q8_argument_errors():
    import torch
    import paper_2511_16652_b200 as egr
    ws = egr.Workspace()
    Q = torch.zeros((8, 24), dtype=torch.int8, device="cuda")            # pitch 24 is not a multiple of 16
    s = torch.ones(8, dtype=torch.bfloat16, device="cuda")
    X = torch.zeros((4, 24), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((4, 8), dtype=torch.bfloat16, device="cuda")
    L = egr.Layer(24, 8, 4, 1, 1, x_dtype=egr.BF16, w_dtype=egr.I8, y_dtype=egr.BF16)
    with pytest.raises(egr.EgrError) as e:
        egr.egr_perturbed_linear_q8(L, X, Q, s, 1.0, 0.1, 0.0, Y, ws)
    assert e.value.code == -2
    Lb = egr.Layer(24, 8, 4, 1, 1, x_dtype=egr.BF16, w_dtype=egr.F32, y_dtype=egr.BF16, ldw=32)
    with pytest.raises(egr.EgrError) as e:
        egr.egr_perturbed_linear_q8(Lb, X, Q, s, 1.0, 0.1, 0.0, Y, ws)
    assert e.value.code == -3
    G = torch.zeros((8, 24), dtype=torch.float32, device="cuda")
    mom = torch.zeros((8, 24), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(egr.EgrError) as e:
        egr.egr_adam_step_q8(Q, G, mom, mom.clone(), 0, 1e-3, 0.9, 0.999, 1e-8, 1.0, ws)      # t = 0
    assert e.value.code == -1


def test_q8_matrix_step_equals_the_entry_points_and_the_oracle_leaf_update():
    """The plumbing class chains the same calls a user would make by hand; the scale leaf after one step matches the
    oracle's Adam step on the oracle's scale gradient."""
    import torch
    import paper_2511_16652_b200 as egr
    from paper_2511_16652_b200.q8 import Q8Matrix
    m, n, N, r, seed = 64, 128, 256, 2, 17
    g = workloads.rng(37, 0)
    W = (g.standard_normal((m, n)) / np.sqrt(n)).astype(np.float32)
    f = oracle.fitness_shape(g.standard_normal(N), oracle.SHAPE_CENTERED_RANK).astype(np.float32)
    fd = torch.from_numpy(f).cuda()
    ws = egr.Workspace()
    P = Q8Matrix(torch.from_numpy(W).cuda(), s_x=0.5, layer_id=9)
    Qo, so = q8.quantize_per_channel(W)
    assert np.array_equal(P.Q.cpu().numpy(), Qo) and np.array_equal(_np(P.scales), so) and P.s_x == 0.5
    Q_hand = P.Q.clone()
    moved = int(P.update(fd, N, r, seed, egr.ANTITHETIC, 1e-2, 0.5, ws, lr_scales=1e-3).item())
    # by hand
    L = egr.Layer(n, m, N, 1, r, layer_id=9, seed=seed, flags=egr.ANTITHETIC)
    G = torch.empty((m, n), dtype=torch.float32, device="cuda")
    egr.egr_es_gradient(L, fd, G, ws)
    m1 = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
    v1 = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
    egr.egr_adam_step_q8(Q_hand, G, m1, v1, 1, 1e-2, 0.9, 0.999, 1e-8, 0.5, ws)
    assert torch.equal(Q_hand, P.Q) and torch.equal(m1, P.mom1) and torch.equal(v1, P.mom2)
    assert moved == int((Q_hand.cpu().numpy() != Qo).sum()) and moved > 0
    # scale leaf: first Adam step moves every entry by lr along the sign of its gradient (bf16 rounding of the sum)
    g_o = q8.es_scale_gradient(f, m, 9, seed, oracle.ANTITHETIC)
    leaf_o, _, _ = q8.adam_step_bf16(np.concatenate([so, [0.5]]).astype(np.float32), g_o.astype(np.float32),
                                     np.zeros(m + 1, np.float32), np.zeros(m + 1, np.float32), 1, 1e-3, 0.9, 0.999, 1e-8)
    clear = np.abs(g_o) > 1e-6 * np.abs(g_o).max()
    np.testing.assert_allclose(_np(P.leaf)[clear], leaf_o[clear], rtol=2.0 ** -7)
    assert abs(P.s_x - float(leaf_o[m])) <= 2.0 ** -7 * abs(float(leaf_o[m]))


def test_q8_training_reduces_the_loss_of_a_toy_regression():
    """End to end on the GPU: perturbed forward -> per-member loss -> centred ranks -> gradient -> discretised Adam,
    40 steps on a 64 x 64 regression whose codes start a few bins away from the target's."""
    import torch
    import paper_2511_16652_b200 as egr
    from paper_2511_16652_b200.q8 import Q8Matrix
    m = n = 64
    N, T, r = 2048, 8, 1
    g = workloads.rng(37, 1)
    Wstar = (g.standard_normal((m, n)) / np.sqrt(n)).astype(np.float32)
    Qs, ss = q8.quantize_per_channel(Wstar)
    start = (np.clip(Qs.astype(int) + g.integers(-6, 7, size=(m, n)), -127, 127) * ss[:, None]).astype(np.float32)
    Xh = workloads.round_to_bf16(g.standard_normal((T, n)).astype(np.float32))
    X = torch.from_numpy(np.tile(Xh, (N, 1))).cuda().to(torch.bfloat16)            # every member sees the same T inputs
    target = torch.from_numpy((Xh.astype(np.float64) @ q8.dequantize(Qs, ss).T).astype(np.float32)).cuda()
    P = Q8Matrix(torch.from_numpy(start).cuda(), layer_id=3)
    ws, ws2 = egr.Workspace(), egr.Workspace()
    Y = torch.empty((N * T, m), dtype=torch.float32, device="cuda")
    shaped = torch.empty(N, dtype=torch.float32, device="cuda")

    def loss_unperturbed():
        P.forward(X[:T * 2], Y[:T * 2], 2, T, r, 0, egr.NO_PERTURB, 0.0, 0.0, ws)
        return float(((Y[:T] - target) ** 2).mean().item())

    first = loss_unperturbed()
    for step in range(40):
        P.forward(X, Y, N, T, r, 100 + step, egr.ANTITHETIC, 4.0, 0.0, ws)
        fit = -((Y.view(N, T, m) - target.unsqueeze(0)) ** 2).mean(dim=(1, 2))
        egr.egr_fitness_shape(fit.contiguous(), egr.SHAPE_CENTERED_RANK, shaped, ws2)
        P.update(shaped, N, r, 100 + step, egr.ANTITHETIC, 1e-2, 1.5, ws)
    last = loss_unperturbed()
    assert np.abs(P.Q.cpu().numpy().astype(int)).max() <= 127
    assert last < 0.6 * first, (first, last)


def test_forward_q8_with_a_pre_expanded_matrix_is_identical():
    import torch
    import paper_2511_16652_b200 as egr
    m, n, N, T, r = 200, 264, 48, 2, 2
    g = workloads.rng(38, 0)
    Qo = g.integers(-127, 128, size=(m, n)).astype(np.int8)
    so = q8.bf16_round((0.01 + 0.01 * g.random(m)).astype(np.float32))
    X = _bf16_tensor(workloads.round_to_bf16(g.standard_normal((N * T, n)).astype(np.float32)))
    pitch = (n + 15) // 16 * 16
    Q = torch.zeros((m, pitch), dtype=torch.int8, device="cuda")
    Q[:, :n] = torch.from_numpy(Qo).cuda()
    Qb = torch.full((m, pitch), -1.0, dtype=torch.bfloat16, device="cuda")
    egr.egr_q8_expand(Q[:, :n], Qb)
    assert np.array_equal(_np(Qb)[:, :n], Qo.astype(np.float32))
    s = _bf16_tensor(so)
    ws = egr.Workspace()
    Y1 = torch.empty((N * T, m), dtype=torch.bfloat16, device="cuda")
    Y2 = torch.empty_like(Y1)
    L1 = egr.Layer(n, m, N, T, r, layer_id=2, seed=8, flags=egr.ANTITHETIC, x_dtype=egr.BF16, w_dtype=egr.I8, ldw=pitch)
    L2 = egr.Layer(n, m, N, T, r, layer_id=2, seed=8, flags=egr.ANTITHETIC, x_dtype=egr.BF16, w_dtype=egr.BF16, ldw=pitch)
    egr.egr_perturbed_linear_q8(L1, X, Q, s, 0.5, 3.0, 1e-3, Y1, ws)
    egr.egr_perturbed_linear_q8(L2, X, Qb, s, 0.5, 3.0, 1e-3, Y2, ws)
    assert torch.equal(Y1, Y2)

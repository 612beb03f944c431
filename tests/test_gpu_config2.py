"""Config 2 of the benchmark set: 3-layer tanh MLP 784 -> 1024 -> 1024 -> 10, bf16 weights and inputs with fp32
accumulation, N = 4096 antithetic members, r = 4, sigma = 0.02, 8 inputs per member, fitness = -cross-entropy
against uniform-random labels, centred ranks, alpha = 0.5, 5 ES steps, all three layers perturbed.

The activation and the loss are the model's business (plain torch ops here); every linear layer, the shaping and
the update go through the C ABI.  Each step is teacher-forced from the oracle's weights (ranks are discontinuous
in the fitness), and activations are rounded to bf16 between layers on both sides."""
import numpy as np
import pytest

import oracle
import workloads
from util import rel_fro

pytestmark = pytest.mark.gpu

DIMS = [(784, 1024), (1024, 1024), (1024, 10)]
N, T, R_, SIGMA, ALPHA, STEPS = 4096, 8, 4, 0.02, 0.5, 5


def _oracle_forward(Ws, X, members, seed, explicit):
    fn = oracle.perturbed_linear if explicit else oracle.perturbed_linear_factored
    h = X
    for li, W in enumerate(Ws):
        y = fn(h, W, members, T, R_, li, seed, oracle.ANTITHETIC, SIGMA)
        if li < 2:
            h = workloads.round_to_bf16(np.tanh(y).astype(np.float32))
    return y


def _neg_ce(logits, labels):
    z = logits - logits.max(axis=1, keepdims=True)
    logp = z - np.log(np.exp(z).sum(axis=1, keepdims=True))
    ce = -logp[np.arange(len(labels)), labels]
    return -ce.reshape(-1, T).mean(axis=1)


def test_config2_five_steps():
    import torch
    import paper_2511_16652_b200 as egr
    egr.load_library()
    g = workloads.rng(2, 1)
    masters = [workloads.round_to_bf16((g.standard_normal((m, n)) / np.sqrt(n)).astype(np.float32)).astype(np.float64)
               for (n, m) in DIMS]
    X = workloads.pair_shared_rows(workloads.round_to_bf16(g.standard_normal((N * T, 784)).astype(np.float32)), T)
    labels = np.repeat(g.integers(0, 10, size=(N // 2, T)), 2, axis=0).reshape(-1)     # partners share labels
    Xd = torch.from_numpy(X).cuda().to(torch.bfloat16)
    ws = egr.Workspace()
    ws2 = egr.Workspace()
    sample = np.array([0, 1, 2046, 2047, 4094, 4095])
    rows = (sample[:, None] * T + np.arange(T)).reshape(-1)
    for step in range(STEPS):
        seed = 100 + step
        shadows = [workloads.round_to_bf16(W.astype(np.float32)) for W in masters]
        # ---- oracle: fitness of every member (factored form), explicit form on the sampled members
        logits_o = _oracle_forward(shadows, X, np.arange(N), seed, explicit=False)
        fit_o = _neg_ce(logits_o, labels)
        logits_s = _oracle_forward(shadows, X[rows], sample, seed, explicit=True)
        assert rel_fro(logits_o[rows], logits_s) < 1e-9
        shaped_o = oracle.fitness_shape(fit_o.astype(np.float32), oracle.SHAPE_CENTERED_RANK)
        # ---- GPU forward
        Wm = [torch.from_numpy(W.astype(np.float32)).cuda() for W in masters]
        Wsh = [w.to(torch.bfloat16) for w in Wm]
        h = Xd
        for li, (n, m) in enumerate(DIMS):
            # hidden layers: tanh fused into the layer's epilogue (fp32 in, one rounding to bf16 out); last layer fp32
            hidden = li < 2
            ldy = (m + 7) // 8 * 8 if hidden else (m + 3) // 4 * 4
            L = egr.Layer(n, m, N, T, R_, layer_id=li, seed=seed, flags=egr.ANTITHETIC | (egr.ACT_TANH if hidden else 0),
                          x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16 if hidden else egr.F32, ldy=ldy)
            Y = torch.empty((N * T, ldy), dtype=torch.bfloat16 if hidden else torch.float32, device="cuda")
            egr.egr_perturbed_linear(L, h, Wsh[li], SIGMA, Y, ws)
            assert egr.egr_workspace_status(ws) == 0
            if hidden:
                h = Y
        logits = Y[:, :10].double()
        logp = torch.log_softmax(logits, dim=1)
        fit = -(-logp[torch.arange(N * T, device="cuda"), torch.from_numpy(labels).cuda()]).reshape(N, T).mean(dim=1)
        assert rel_fro(logits.cpu().numpy(), logits_o) < 1e-2
        assert rel_fro(fit.cpu().numpy(), fit_o) < 1e-2
        # shaping of the oracle's raw fitness is bit-exact
        shaped = torch.empty(N, dtype=torch.float32, device="cuda")
        egr.egr_fitness_shape(torch.from_numpy(fit_o.astype(np.float32)).cuda(), egr.SHAPE_CENTERED_RANK, shaped, ws2)
        assert np.array_equal(shaped.cpu().numpy().astype(np.float64), shaped_o)
        # ---- update of every layer, checked on sampled blocks; the oracle's masters advance with the GPU's dW
        for li, (n, m) in enumerate(DIMS):
            L = egr.Layer(n, m, N, T, R_, layer_id=li, seed=seed, flags=egr.ANTITHETIC, x_dtype=egr.BF16,
                          w_dtype=egr.BF16, y_dtype=egr.BF16)
            dW = torch.empty((m, n), dtype=torch.float32, device="cuda")
            egr.egr_es_update(L, Wm[li], shaped, ALPHA, ws, W_shadow=Wsh[li], dW_out=dW)
            assert egr.egr_workspace_status(ws) == 0
            got = dW.cpu().numpy().astype(np.float64)
            for (j0, l0) in [(0, 0), (m - min(m, 16), n - 16), (m // 3, n // 2)]:
                j1, l1 = min(m, j0 + 16), l0 + 16
                want = oracle.es_update_block(shaped_o, R_, li, seed, oracle.ANTITHETIC, ALPHA, j0, j1, l0, l1)
                assert rel_fro(got[j0:j1, l0:l1], want) < 1e-2
            assert torch.equal(Wsh[li], Wm[li].to(torch.bfloat16))
            masters[li] = masters[li] + got

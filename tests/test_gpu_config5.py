"""Config 5 of the benchmark set (the workload bench.py times): one 4096 x 4096 bf16 layer, one token per member.
At these sizes the oracle evaluates sampled members (forward) and sampled 32 x 32 blocks (update)."""
import numpy as np
import pytest

import oracle
import workloads
from util import rel_fro

pytestmark = pytest.mark.gpu

D = 4096


@pytest.mark.parametrize("N,r", [(256, 16), (4096, 4), (65536, 1)])
def test_config5_sampled(N, r):
    import torch
    import paper_2511_16652_b200 as egr
    egr.load_library()
    W = workloads.linear_layer(0, D, D, 1, bf16=True)[0]
    gen = torch.Generator().manual_seed(7)
    Xd = torch.randn((N, D), generator=gen, dtype=torch.float32).to(torch.bfloat16).cuda()
    Wd = torch.from_numpy(W).cuda().to(torch.bfloat16)
    Y = torch.empty((N, D), dtype=torch.bfloat16, device="cuda")
    L = egr.Layer(D, D, N, 1, r, layer_id=0, seed=3, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16)
    ws = egr.Workspace()
    egr.egr_perturbed_linear(L, Xd, Wd, 0.01, Y, ws)
    assert egr.egr_workspace_status(ws) == 0
    sel = np.unique(np.concatenate([[0, 1, 127, 128, N - 1], workloads.rng(N, 5).integers(0, N, size=11)]))
    Xs = Xd[torch.from_numpy(sel).cuda()].float().cpu().numpy()
    want = oracle.perturbed_linear(Xs, W, sel, 1, r, 0, 3, 0, 0.01)
    got = Y[torch.from_numpy(sel).cuda()].float().cpu().numpy()
    assert rel_fro(got, want) < 1e-2
    base = Xs.astype(np.float64) @ W.astype(np.float64).T
    assert rel_fro(got - base, want - base) < 5e-2          # the rank-r term alone, seen through bf16 outputs
    # update on sampled blocks
    f = workloads.raw_fitness(N, N)
    shaped_o = oracle.fitness_shape(f, oracle.SHAPE_CENTERED_RANK)
    shaped = torch.empty(N, dtype=torch.float32, device="cuda")
    egr.egr_fitness_shape(torch.from_numpy(f).cuda(), egr.SHAPE_CENTERED_RANK, shaped, egr.Workspace())
    assert np.array_equal(shaped.cpu().numpy().astype(np.float64), shaped_o)
    Wm = torch.from_numpy(W).cuda()
    dW = torch.empty((D, D), dtype=torch.float32, device="cuda")
    egr.egr_es_update(L, Wm, shaped, 0.5, ws, W_shadow=Wd, dW_out=dW)
    assert egr.egr_workspace_status(ws) == 0
    for (j0, l0) in [(0, 0), (D - 32, D - 32), (1000, 2200)]:
        want = oracle.es_update_block(shaped_o, r, 0, 3, 0, 0.5, j0, j0 + 32, l0, l0 + 32)
        assert rel_fro(dW[j0:j0 + 32, l0:l0 + 32].cpu().numpy(), want) < 1e-2
    assert torch.equal(Wd, Wm.to(torch.bfloat16))

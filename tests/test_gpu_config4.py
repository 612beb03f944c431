"""Config 4 of the benchmark set, at reduced depth and population so that the CPU oracle finishes in seconds:
decoder-only transformer, d_model 2048, 16 heads, FFN 8192 with exact-erf GELU, vocab 32000, RMSNorm, learned
absolute positions, untied LM head, bf16 weights ~ N(0, 0.02^2); every linear layer perturbed with r = 1,
sigma = 1e-3; each member scores one sequence of uniform-random token ids; fitness = log-likelihood of the
tokens; one forward, centred ranks, one update step.

Only the linear layers, the shaping and the update belong to the method and go through the C ABI.  The glue
(embedding lookup, RMSNorm, causal softmax attention, GELU, log-softmax) is the model's business and is NOT
fixed by the paper ("parity unpinned" for the glue): it is plain torch on the GPU side and plain numpy fp64 on
the oracle side, with tensors rounded to bf16 wherever they are handed from one kernel to the next.
Layer ids: 16*layer + {0: Q, 1: K, 2: V, 3: O, 4: up, 5: down}, head 1001."""
import math

import numpy as np
import pytest

import oracle
import workloads
from util import rel_fro

pytestmark = pytest.mark.gpu

D, H, FF, V, LAYERS = 2048, 16, 8192, 32000, 2
N, T, SIGMA, ALPHA, SEED = 8, 64, 1e-3, 0.01, 5
HD = D // H


def _weights():
    g = workloads.rng(4, 1)
    w = lambda m, n: workloads.round_to_bf16((g.standard_normal((m, n)) * 0.02).astype(np.float32))
    layers = [dict(q=w(D, D), k=w(D, D), v=w(D, D), o=w(D, D), up=w(FF, D), down=w(D, FF)) for _ in range(LAYERS)]
    return dict(layers=layers, head=w(V, D), emb=w(V, D), pos=w(T, D))


def _bf(a):
    return workloads.round_to_bf16(np.asarray(a, dtype=np.float32)).astype(np.float64)


def _rms(x):
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + 1e-6)


def _oracle_forward(Wt, tokens):
    members = np.arange(N)
    lin = lambda x, W, lid: oracle.perturbed_linear_factored(x, W, members, T, 1, lid, SEED, 0, SIGMA)
    x = _bf(Wt["emb"][tokens.reshape(-1)].astype(np.float64) + np.tile(Wt["pos"].astype(np.float64), (N, 1)))
    from scipy.special import erf
    for li, L in enumerate(Wt["layers"]):
        h = _bf(_rms(x))
        q, k, v = (_bf(lin(h, L[n], 16 * li + i)) for i, n in enumerate(("q", "k", "v")))
        att = np.zeros_like(q)
        mask = np.triu(np.ones((T, T), bool), 1)
        for i in range(N):
            for hd in range(H):
                sl = (slice(i * T, (i + 1) * T), slice(hd * HD, (hd + 1) * HD))
                s = q[sl] @ k[sl].T / math.sqrt(HD)
                s[mask] = -np.inf
                p = np.exp(s - s.max(axis=1, keepdims=True))
                p /= p.sum(axis=1, keepdims=True)
                att[sl] = p @ v[sl]
        x = _bf(x + _bf(lin(_bf(att), L["o"], 16 * li + 3)))
        h = _bf(_rms(x))
        u = lin(h, L["up"], 16 * li + 4)
        u = _bf(0.5 * u * (1.0 + erf(u / math.sqrt(2.0))))
        x = _bf(x + _bf(lin(u, L["down"], 16 * li + 5)))
    logits = lin(_bf(_rms(x)), Wt["head"], 1001)
    return logits


def _fitness(logits, tokens):
    z = logits - logits.max(axis=1, keepdims=True)
    logp = z - np.log(np.exp(z).sum(axis=1, keepdims=True))
    lp = logp.reshape(N, T, V)
    tgt = tokens[:, 1:]
    return np.array([lp[i, np.arange(T - 1), tgt[i]].sum() for i in range(N)])


def test_config4_reduced_forward_and_update():
    import torch
    import paper_2511_16652_b200 as egr
    egr.load_library()
    Wt = _weights()
    tokens = workloads.rng(4, 2).integers(0, V, size=(N, T))
    logits_o = _oracle_forward(Wt, tokens)
    fit_o = _fitness(logits_o, tokens)

    dev = lambda a: torch.from_numpy(a).cuda().to(torch.bfloat16)
    ws = egr.Workspace()

    def lin(x, W, lid, out_f32=False, act=0):
        m, n = W.shape
        L = egr.Layer(n, m, N, T, 1, layer_id=lid, seed=SEED, flags=act, x_dtype=egr.BF16, w_dtype=egr.BF16,
                      y_dtype=egr.F32 if out_f32 else egr.BF16)
        Y = torch.empty((N * T, m), dtype=torch.float32 if out_f32 else torch.bfloat16, device="cuda")
        egr.egr_perturbed_linear(L, x.contiguous(), W, SIGMA, Y, ws)
        assert egr.egr_workspace_status(ws) == 0
        return Y

    rms = lambda x: (x.float() * torch.rsqrt((x.float() ** 2).mean(dim=-1, keepdim=True) + 1e-6)).to(torch.bfloat16)
    tok = torch.from_numpy(tokens).cuda()
    x = (dev(Wt["emb"])[tok.reshape(-1)].float() + dev(Wt["pos"]).float().repeat(N, 1)).to(torch.bfloat16)
    causal = torch.triu(torch.ones(T, T, dtype=torch.bool, device="cuda"), 1)
    for li, Lw in enumerate(Wt["layers"]):
        h = rms(x)
        q, k, v = (lin(h, dev(Lw[n]), 16 * li + i) for i, n in enumerate(("q", "k", "v")))
        qh, kh, vh = (t.float().reshape(N, T, H, HD).permute(0, 2, 1, 3) for t in (q, k, v))
        s = qh @ kh.transpose(-1, -2) / math.sqrt(HD)
        s = s.masked_fill(causal, float("-inf"))
        att = (torch.softmax(s, dim=-1) @ vh).permute(0, 2, 1, 3).reshape(N * T, D).to(torch.bfloat16)
        x = (x.float() + lin(att, dev(Lw["o"]), 16 * li + 3).float()).to(torch.bfloat16)
        h = rms(x)
        u = lin(h, dev(Lw["up"]), 16 * li + 4, act=egr.ACT_GELU)        # GELU in the epilogue, one rounding to bf16
        x = (x.float() + lin(u, dev(Lw["down"]), 16 * li + 5).float()).to(torch.bfloat16)
    logits = lin(rms(x), dev(Wt["head"]), 1001, out_f32=True)
    assert rel_fro(logits.cpu().numpy(), logits_o) < 1e-2
    logp = torch.log_softmax(logits.double(), dim=-1).reshape(N, T, V)
    fit = torch.stack([logp[i, torch.arange(T - 1), tok[i, 1:]].sum() for i in range(N)])
    assert rel_fro(fit.cpu().numpy(), fit_o) < 1e-2

    # shaping and update of two of the matrices (K = N*r = 8: the update is bandwidth-bound here)
    shaped_o = oracle.fitness_shape(fit_o.astype(np.float32), oracle.SHAPE_CENTERED_RANK)
    shaped = torch.empty(N, dtype=torch.float32, device="cuda")
    egr.egr_fitness_shape(torch.from_numpy(fit_o.astype(np.float32)).cuda(), egr.SHAPE_CENTERED_RANK, shaped, egr.Workspace())
    assert np.array_equal(shaped.cpu().numpy().astype(np.float64), shaped_o)
    for W, lid in ((Wt["layers"][1]["up"], 16 + 4), (Wt["head"], 1001)):
        m, n = W.shape
        L = egr.Layer(n, m, N, T, 1, layer_id=lid, seed=SEED, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16)
        Wm = torch.from_numpy(W).cuda()
        Wsh = Wm.to(torch.bfloat16)
        dW = torch.empty((m, n), dtype=torch.float32, device="cuda")
        egr.egr_es_update(L, Wm, shaped, ALPHA, ws, W_shadow=Wsh, dW_out=dW)
        assert egr.egr_workspace_status(ws) == 0
        got = dW.cpu().numpy()
        for (j0, l0) in [(0, 0), (m - 32, n - 32), (m // 2 + 7, 1000)]:
            want = oracle.es_update_block(shaped_o, 1, lid, SEED, 0, ALPHA, j0, j0 + 32, l0, l0 + 32)
            assert rel_fro(got[j0:j0 + 32, l0:l0 + 32], want) < 1e-2
        assert torch.equal(Wsh, Wm.to(torch.bfloat16))

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


# ---------------------------------------------------------------------------------------------- full size
def test_config4_full_size_sampled_members_and_update_blocks():
    """Config 4 as stated: 24 layers, N = 1024 members x 256 tokens, vocab 32000, every linear layer perturbed with r = 1.
    The GPU runs the whole population; the oracle runs the whole forward for three sampled members (the explicit form
    W + sigma E_i applied with the library matrix product) and, for the update, sampled 32 x 32 blocks of dW summed over
    all 1024 members for four matrices - two of them updated the way a caller does it, without the test-only dW_out."""
    import torch
    import paper_2511_16652_b200 as egr
    egr.load_library()
    NL, Nm, Tm, seed = 24, 1024, 256, 11
    R = Nm * Tm
    sampled = [0, 511, 1023]
    mk = lambda stream, m, n: workloads.bf16_normal_matrix_torch(4, stream, m, n, 0.02, "cuda")
    names = ("q", "k", "v", "o", "up", "down")
    shapes = dict(q=(D, D), k=(D, D), v=(D, D), o=(D, D), up=(FF, D), down=(D, FF))
    layers = [{nm: mk(16 * li + i, *shapes[nm]) for i, nm in enumerate(names)} for li in range(NL)]
    head, emb, pos = mk(1001, V, D), mk(2000, V, D), mk(2001, Tm, D)
    tokens = workloads.rng(4, 3).integers(0, V, size=(Nm, Tm))
    tok = torch.from_numpy(tokens).cuda()
    ws = egr.Workspace()

    def lin(x, W, lid, members=Nm, base=0, act=0, out_f32=False):
        m, n = W.shape
        L = egr.Layer(n, m, members, Tm, 1, layer_id=lid, seed=seed, flags=act, member_base=base, x_dtype=egr.BF16,
                      w_dtype=egr.BF16, y_dtype=egr.F32 if out_f32 else egr.BF16)
        Y = torch.empty((members * Tm, m), dtype=torch.float32 if out_f32 else torch.bfloat16, device="cuda")
        egr.egr_perturbed_linear(L, x, W, SIGMA, Y, ws)
        return Y

    rms = lambda x: (x.float() * torch.rsqrt((x.float() ** 2).mean(dim=-1, keepdim=True) + 1e-6)).to(torch.bfloat16)
    rows_s = torch.cat([torch.arange(i * Tm, (i + 1) * Tm) for i in sampled]).cuda()
    keep = {}                                                          # (layer, name) -> (input rows, output rows) of the sampled members
    probe_layers = (0, 11, 23)

    def lin_keep(li, nm, xin, W, lid, **kw):
        y = lin(xin, W, lid, **kw)
        if li in probe_layers:
            keep[(li, nm)] = (xin[rows_s].float().cpu().numpy(), y[rows_s].float().cpu().numpy(), lid, kw.get("act", 0))
        return y

    x = (emb[tok.reshape(-1)].float() + pos.float().repeat(Nm, 1)).to(torch.bfloat16)
    causal = torch.triu(torch.ones(Tm, Tm, dtype=torch.bool, device="cuda"), 1)
    for li, Lw in enumerate(layers):
        h = rms(x)
        q, k, v = (lin_keep(li, nm, h, Lw[nm], 16 * li + i) for i, nm in enumerate(("q", "k", "v")))
        att = torch.empty((R, D), dtype=torch.bfloat16, device="cuda")
        for c0 in range(0, Nm, 256):                                   # fp32 attention in slices of 256 members
            sl = slice(c0 * Tm, (c0 + 256) * Tm)
            qh, kh, vh = (z[sl].float().view(256, Tm, H, HD).transpose(1, 2) for z in (q, k, v))
            sc = (qh @ kh.transpose(-1, -2) / math.sqrt(HD)).masked_fill(causal, float("-inf"))      # plain fp32 products
            att[sl] = (torch.softmax(sc, dim=-1) @ vh).transpose(1, 2).reshape(256 * Tm, D).to(torch.bfloat16)
            del sc
        del q, k, v, h
        x = (x.float() + lin_keep(li, "o", att, Lw["o"], 16 * li + 3).float()).to(torch.bfloat16)
        u = lin_keep(li, "up", rms(x), Lw["up"], 16 * li + 4, act=egr.ACT_GELU)
        x = (x.float() + lin_keep(li, "down", u, Lw["down"], 16 * li + 5).float()).to(torch.bfloat16)
        del att, u
    assert egr.egr_workspace_status(ws) == 0
    xn = rms(x)
    fit = torch.empty(Nm, dtype=torch.float64, device="cuda")
    for c0 in range(0, Nm, 64):                                        # the vocabulary head in slices of 64 members
        logits = lin(xn[c0 * Tm:(c0 + 64) * Tm], head, 1001, members=64, base=c0, out_f32=True)
        lp = torch.log_softmax(logits.double(), dim=-1).view(64, Tm, V)
        fit[c0:c0 + 64] = lp[:, :-1].gather(-1, tok[c0:c0 + 64, 1:].unsqueeze(-1)).squeeze(-1).sum(-1)
        del logits, lp
    assert egr.egr_workspace_status(ws) == 0
    # the same fitness from the head that ends in the log-likelihood (one call over all 262144 rows, no logits written)
    tgt = torch.full((Nm, Tm), -1, dtype=torch.int32, device="cuda")
    tgt[:, :-1] = tok[:, 1:].to(torch.int32)
    logp = torch.empty(R, dtype=torch.float32, device="cuda")
    Lh = egr.Layer(D, V, Nm, Tm, 1, layer_id=1001, seed=seed, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16)
    egr.egr_perturbed_linear_loglik(Lh, xn, head, SIGMA, tgt.reshape(-1), logp, ws)
    assert egr.egr_workspace_status(ws) == 0
    fit_fused = logp.double().view(Nm, Tm).sum(dim=1)
    assert float((fit_fused - fit).abs().max()) < 2e-2          # 255 terms of about -10.4 each, fp32 sums on both sides
    logits_s = torch.cat([lin(xn[i * Tm:(i + 1) * Tm], head, 1001, members=1, base=i, out_f32=True) for i in sampled]).cpu().numpy()
    xn_s = xn[rows_s].float().cpu().numpy()

    # ---- the oracle on the sampled members
    S = np.array(sampled)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    olin = lambda xx, W, lid, act=0: oracle.perturbed_linear_blas(xx, f64(W), S, Tm, 1, lid, seed, act, SIGMA)
    from scipy.special import erf
    xo = _bf(f64(emb)[tokens[S].reshape(-1)] + np.tile(f64(pos), (len(S), 1)))
    mask = np.triu(np.ones((Tm, Tm), bool), 1)
    for li, Lw in enumerate(layers):
        h = _bf(_rms(xo))
        q, k, v = (_bf(olin(h, Lw[nm], 16 * li + i)) for i, nm in enumerate(("q", "k", "v")))
        att = np.zeros_like(q)
        for i in range(len(S)):
            for hd in range(H):
                sl = (slice(i * Tm, (i + 1) * Tm), slice(hd * HD, (hd + 1) * HD))
                s = q[sl] @ k[sl].T / math.sqrt(HD)
                s[mask] = -np.inf
                p = np.exp(s - s.max(axis=1, keepdims=True))
                p /= p.sum(axis=1, keepdims=True)
                att[sl] = p @ v[sl]
        xo = _bf(xo + _bf(olin(_bf(att), Lw["o"], 16 * li + 3)))
        u = olin(_bf(_rms(xo)), Lw["up"], 16 * li + 4)
        u = _bf(0.5 * u * (1.0 + erf(u / math.sqrt(2.0))))
        xo = _bf(xo + _bf(olin(u, Lw["down"], 16 * li + 5)))
    logits_o = olin(_bf(_rms(xo)), head, 1001)
    # (1) every probed linear layer on the inputs the GPU actually gave it: the tolerance of a bf16-input, fp32-accumulate path
    worst = 0.0
    for (li, nm), (xin, yout, lid, act) in keep.items():
        want = olin(xin, layers[li][nm], lid, act)
        err = rel_fro(yout, _bf(want))
        worst = max(worst, err)
        assert err < 1e-2, (li, nm, err)
    err_head = rel_fro(logits_s, olin(xn_s, head, 1001))
    assert err_head < 1e-2
    # (2) the whole 24-layer chain, free-running on both sides.  Two correct bf16 pipelines do not stay within one
    # layer's tolerance of each other: once two activations differ at all, rounding both to bf16 turns a difference d
    # (below one ulp) into a one-ulp difference with probability d / ulp, i.e. a mean square of d * ulp instead of d^2, so
    # any difference grows to the size of the rounding noise itself (2^-9 relative) within a few hand-overs and then
    # adds up like independent noise over the ~100 hand-overs on the residual path: about 2^-9 * sqrt(100) = 2e-2.
    err_chain = rel_fro(logits_s, logits_o)
    assert err_chain < 3e-2
    z = logits_o - logits_o.max(axis=1, keepdims=True)
    logp = (z - np.log(np.exp(z).sum(axis=1, keepdims=True))).reshape(len(S), Tm, V)
    fit_o = np.array([logp[i, np.arange(Tm - 1), tokens[S[i], 1:]].sum() for i in range(len(S))])
    fit_g = fit.cpu().numpy()
    assert rel_fro(fit_g[S], fit_o) < 1e-2
    assert rel_fro(fit_fused.cpu().numpy()[S], fit_o) < 1e-2
    print("config 4 full size: worst probed layer %.2e, head %.2e, free-running logits %.2e, fitness abs err %.3g "
          "(population std %.3g)" % (worst, err_head, err_chain, np.abs(fit_g[S] - fit_o).max(), fit_g.std()))

    # ---- shaping over the whole population, then the update of four matrices on sampled blocks
    fit32 = fit.float().contiguous()
    shaped = torch.empty(Nm, dtype=torch.float32, device="cuda")
    egr.egr_fitness_shape(fit32, egr.SHAPE_CENTERED_RANK, shaped, egr.Workspace())
    shaped_o = oracle.fitness_shape(fit32.cpu().numpy(), oracle.SHAPE_CENTERED_RANK)
    assert np.array_equal(shaped.cpu().numpy().astype(np.float64), shaped_o)
    g = workloads.rng(4, 9)
    for W, lid, with_dw in ((layers[0]["q"], 0, True), (layers[23]["down"], 16 * 23 + 5, False), (layers[11]["up"], 16 * 11 + 4, True),
                            (head, 1001, False)):
        m, n = W.shape
        L = egr.Layer(n, m, Nm, Tm, 1, layer_id=lid, seed=seed, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16)
        W0 = W.float()
        Wm = W0.clone()
        Wsh = torch.zeros_like(W)
        dW = torch.empty((m, n), dtype=torch.float32, device="cuda") if with_dw else None
        egr.egr_es_update(L, Wm, shaped, ALPHA, ws, W_shadow=Wsh, dW_out=dW)
        assert egr.egr_workspace_status(ws) == 0
        got = (dW if with_dw else (Wm - W0)).cpu().numpy()
        blocks = [(0, 0), (m - 32, n - 32)] + [(int(g.integers(0, m - 32)), int(g.integers(0, n - 32))) for _ in range(14)]
        for (j0, l0) in blocks:
            want = oracle.es_update_block(shaped_o, 1, lid, seed, 0, ALPHA, j0, j0 + 32, l0, l0 + 32)
            # without dW_out the change is read off the fp32 master, whose rounding (ulp of 0.02-sized weights) is
            # 1e-3 of these steps: it stays inside the tolerance
            assert rel_fro(got[j0:j0 + 32, l0:l0 + 32], want) < 1e-2, (lid, j0, l0)
        assert torch.equal(Wsh, Wm.to(torch.bfloat16))
        del W0, Wm, Wsh, dW

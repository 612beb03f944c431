"""Throughput of the library on the benchmark configurations, beyond the single line bench.py prints.

    python bench_suite.py [--out FILE.json] [--quick]

For every point it reports the perturbed forward, the library's own unperturbed kernel, torch.matmul (library
comparison), the update, and -- for the one-token-per-member sweep -- a naive full-rank-ES baseline in which every
member's W + sigma*E_i is materialised (torch ops, random factors standing in for the noise) and applied with a
batched matrix-vector product.  Times are medians of ten individually timed calls (CUDA events) after three warm-up
calls, with L2 flushed before each call of the memory-bound pieces; all inputs are synthetic.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    import torch

    import paper_2511_16652_b200 as egr
    import workloads

    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None)
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--only", default=None, choices=["c2", "c3", "c4", "c4model", "c5", "rates", "q8"], help="run one configuration only")
    ap.add_argument("--seq-len", type=int, default=128, help="config 3: bytes per sequence (a short one keeps a profiler capture of the one-launch kernel small)")
    args = ap.parse_args()
    egr.load_library()
    ws = egr.Workspace()
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = json.load(open(peaks_path)).get("bf16_tflops_sustained", 1400.0) if os.path.exists(peaks_path) else 1400.0

    flush = torch.empty(160 << 20, dtype=torch.uint8, device="cuda")      # larger than the 126 MB L2
    # a quarter of a second of dense work first: the first measurements of a cold process otherwise see the clocks ramp
    _a = torch.randn((8192, 8192), device="cuda").to(torch.bfloat16)
    for _ in range(200):
        torch.matmul(_a, _a)
    torch.cuda.synchronize()
    del _a

    def t(fn, reps=10, warm=3, flush_l2=False):
        """Median of `reps` individually timed, back-to-back calls (CUDA events) after `warm` warm-up calls; flush_l2 writes a buffer
        larger than L2 before every timed call (for the memory-bound pieces whose operands would otherwise stay cached)."""
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        marks = []
        for _ in range(reps):                 # back to back: the calls see the clocks of a sustained run
            if flush_l2:
                flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            marks.append((e0, e1))
        torch.cuda.synchronize()
        times = [a.elapsed_time(b) for a, b in marks]
        return float(np.median(times))

    rows = []

    def linear_point(tag, N, T, n, m, r, sigma, naive=False, base_flags=0):
        R = N * T
        X = torch.randn((R, n), device="cuda").to(torch.bfloat16)
        W = (torch.randn((m, n), device="cuda") / np.sqrt(n)).to(torch.bfloat16)
        Wm = W.float()
        Y = torch.empty((R, m), dtype=torch.bfloat16, device="cuda")
        shaped = torch.randn(N, device="cuda")
        L = lambda flags=0: egr.Layer(n, m, N, T, r, seed=1, flags=flags | base_flags)
        res = dict(config=tag, N=N, T=T, n=n, m=m, r=r)
        res["fwd_ms"] = t(lambda: egr.egr_perturbed_linear(L(), X, W, sigma, Y, ws))
        res["plain_ms"] = t(lambda: egr.egr_perturbed_linear(L(egr.NO_PERTURB), X, W, sigma, Y, ws))
        res["torch_ms"] = t(lambda: torch.matmul(X, W.t(), out=Y))
        res["upd_ms"] = t(lambda: egr.egr_es_update(L(), Wm, shaped, 0.01, ws, W_shadow=W))
        assert egr.egr_workspace_status(ws) == 0
        fl = 2.0 * R * n * m
        res["tokens_per_s"] = R / (res["fwd_ms"] * 1e-3)
        res["fwd_tflops"] = fl / (res["fwd_ms"] * 1e-3) / 1e12
        res["fwd_frac_of_peak"] = res["fwd_tflops"] / peak
        res["pct_of_plain"] = 100 * res["plain_ms"] / res["fwd_ms"]
        res["pct_of_torch"] = 100 * res["torch_ms"] / res["fwd_ms"]
        K = (N // 2 if base_flags & egr.ANTITHETIC else N) * r
        res["upd_tflops"] = 2.0 * m * n * K / (res["upd_ms"] * 1e-3) / 1e12
        res["upd_w_gbs"] = m * n * 10 / (res["upd_ms"] * 1e-3) / 1e9
        if naive:
            # naive full-rank ES on a chunk of 64 members: materialise W + sigma a b^T per member, then a batched matvec
            C = min(64, N)
            a = torch.randn((C, m, 1), device="cuda", dtype=torch.bfloat16)
            b = torch.randn((C, 1, n), device="cuda", dtype=torch.bfloat16)
            Wp = torch.empty((C, m, n), device="cuda", dtype=torch.bfloat16)
            xc = X[:C].reshape(C, n, 1)

            def materialise():
                torch.baddbmm(W.unsqueeze(0).expand(C, m, n), a, b, alpha=sigma, out=Wp)

            def apply_only():
                torch.bmm(Wp, xc)
            materialise()
            ms_mat, ms_app = t(materialise), t(apply_only)
            res["naive_ms_extrapolated"] = (ms_mat + ms_app) * N / C
            res["naive_apply_only_ms_extrapolated"] = ms_app * N / C
            res["speedup_vs_naive"] = res["naive_ms_extrapolated"] / res["fwd_ms"]
            res["speedup_vs_naive_pregenerated"] = res["naive_apply_only_ms_extrapolated"] / res["fwd_ms"]
            del a, b, Wp
        rows.append(res)
        print(json.dumps(res), flush=True)
        del X, W, Wm, Y
        torch.cuda.empty_cache()

    # config 5: 4096 x 4096, one token per member
    want = lambda c: args.only in (None, c)
    Ns = [256, 4096, 65536] if args.quick else [256, 1024, 4096, 16384, 65536]
    for N in (Ns if want("c5") else []):
        for r in (1, 4, 16):
            linear_point("c5", N, 1, 4096, 4096, r, 0.01, naive=(r == 1))
    # config 4 layer shapes: 1024 members x 256 tokens
    for (n, m) in ([(2048, 2048), (2048, 8192), (8192, 2048), (2048, 32000)] if want("c4") else []):
        linear_point("c4", 1024, 256, n, m, 1, 1e-3)
    # config 2 layer shapes: 4096 antithetic members x 8 inputs
    for (n, m) in ([(784, 1024), (1024, 1024)] if want("c2") else []):
        linear_point("c2", 4096, 8, n, m, 4, 0.02, base_flags=egr.ANTITHETIC)

    if args.only == "c4model":
        # config 4 end to end: decoder-only transformer, d_model 2048, 24 layers, 16 heads, FFN 8192 (GELU), vocab 32000,
        # N = 1024 members x 256 tokens, r = 1, sigma = 1e-3.  Linear layers through the library (perturbed or with the
        # unperturbed flag, GELU fused into the up-projection), glue (RMSNorm, causal attention, residuals, log-softmax) in torch; then centred ranks and
        # the update of every matrix.
        import torch.nn.functional as Fn
        Dm, H, FF, V, NL, Nm, T = 2048, 16, 8192, 32000, 24, 1024, 256
        R = Nm * T
        g = torch.Generator(device="cuda").manual_seed(0)
        mk = lambda m, n: (torch.randn((m, n), device="cuda", generator=g) * 0.02).to(torch.bfloat16)
        layers = [dict(q=mk(Dm, Dm), k=mk(Dm, Dm), v=mk(Dm, Dm), o=mk(Dm, Dm), up=mk(FF, Dm), down=mk(Dm, FF)) for _ in range(NL)]
        head, emb, pos = mk(V, Dm), mk(V, Dm), mk(T, Dm)
        tokens = torch.randint(0, V, (Nm, T), device="cuda", generator=g)
        rms = lambda x: Fn.rms_norm(x, (Dm,), eps=1e-6)                 # fp32 statistics inside, gain 1, one kernel

        skip_linear = [False]                                         # glue-only pass: leave the outputs unwritten
        head_mode = ["fused"]                                         # or "logits": bf16 logits in slices + torch log_softmax
        next_tok = torch.full((Nm, T), -1, dtype=torch.int32, device="cuda")
        next_tok[:, :-1] = tokens[:, 1:].to(torch.int32)
        next_tok = next_tok.reshape(-1)

        def lin(x, W, lid, flags, members=Nm, base=0):
            m, n = W.shape
            L = egr.Layer(n, m, members, T, 1, layer_id=lid, seed=7, flags=flags, member_base=base)
            Y = torch.empty((members * T, m), dtype=torch.bfloat16, device="cuda")
            if skip_linear[0]:
                return Y.zero_()
            egr.egr_perturbed_linear(L, x, W, 1e-3, Y, ws)
            return Y

        def forward(flags):
            x = (emb[tokens.reshape(-1)] + pos.repeat(Nm, 1))
            for li, Lw in enumerate(layers):
                h = rms(x)
                q, k, v = (lin(h, Lw[nm], 16 * li + i, flags) for i, nm in enumerate(("q", "k", "v")))
                qh, kh, vh = (z.view(Nm, T, H, Dm // H).transpose(1, 2) for z in (q, k, v))
                att = Fn.scaled_dot_product_attention(qh, kh, vh, is_causal=True).transpose(1, 2).reshape(R, Dm)
                x = x + lin(att, Lw["o"], 16 * li + 3, flags)
                u = lin(rms(x), Lw["up"], 16 * li + 4, flags | egr.ACT_GELU)      # GELU in the layer's epilogue
                x = x + lin(u, Lw["down"], 16 * li + 5, flags)
                del h, q, k, v, att, u
            xn = rms(x)
            if head_mode[0] == "fused":
                # the head ends in the log-likelihood of the next token: no logits, no log-softmax pass
                logp = torch.empty(R, dtype=torch.float32, device="cuda")
                if skip_linear[0]:
                    return logp.zero_().view(Nm, T).sum(dim=1)
                Lh = egr.Layer(Dm, V, Nm, T, 1, layer_id=1001, seed=7, flags=flags)
                egr.egr_perturbed_linear_loglik(Lh, xn, head, 1e-3, next_tok, logp, ws)
                return logp.view(Nm, T).sum(dim=1)
            fit = torch.empty(Nm, dtype=torch.float32, device="cuda")
            chunk = 128                                              # members per slice of the vocabulary head
            for c0 in range(0, Nm, chunk):
                logits = lin(xn[c0 * T:(c0 + chunk) * T], head, 1001, flags, members=chunk, base=c0)
                lp = torch.log_softmax(logits.float(), dim=-1).view(chunk, T, V)
                tgt = tokens[c0:c0 + chunk, 1:]
                fit[c0:c0 + chunk] = lp[:, :-1].gather(-1, tgt.unsqueeze(-1)).squeeze(-1).sum(-1)
                del logits, lp
            return fit

        def timed_once(fn):
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); out = fn(); e1.record(); torch.cuda.synchronize()
            return e0.elapsed_time(e1), out

        forward(0)                                                    # warm-up
        ms_p, fit = timed_once(lambda: forward(0))
        ms_u, _ = timed_once(lambda: forward(egr.NO_PERTURB))
        assert egr.egr_workspace_status(ws) == 0
        head_mode[0] = "logits"
        forward(0)
        ms_p_logits, fit_logits = timed_once(lambda: forward(0))
        head_mode[0] = "fused"
        skip_linear[0] = True
        ms_glue, _ = timed_once(lambda: forward(0))                   # torch glue (plus zero-filling the outputs) alone
        skip_linear[0] = False
        shaped = torch.empty(Nm, dtype=torch.float32, device="cuda")
        egr.egr_fitness_shape(fit, egr.SHAPE_CENTERED_RANK, shaped, egr.Workspace())
        mats = [(Lw[nm], 16 * li + i) for li, Lw in enumerate(layers) for i, nm in enumerate(("q", "k", "v", "o", "up", "down"))] + [(head, 1001)]
        masters = None                                                # fp32 masters are created per matrix to bound memory

        def update_all():
            for W, lid in mats:
                m, n = W.shape
                Wm = W.float()
                egr.egr_es_update(egr.Layer(n, m, Nm, T, 1, layer_id=lid, seed=7), Wm, shaped, 0.01, ws, W_shadow=W)
                del Wm
        ms_upd, _ = timed_once(update_all)
        flops = 2.0 * R * (NL * (4 * Dm * Dm + 2 * Dm * FF) + Dm * V)
        res = dict(config="c4model", members=Nm, tokens=R, fwd_perturbed_ms=ms_p, fwd_unperturbed_ms=ms_u,
                   pct_of_unperturbed=100 * ms_u / ms_p, tokens_per_s=R / (ms_p * 1e-3),
                   glue_only_ms=ms_glue, linear_only_ms=ms_p - ms_glue,
                   linear_tflops=flops / ((ms_p - ms_glue) * 1e-3) / 1e12,
                   linear_frac_of_peak=flops / ((ms_p - ms_glue) * 1e-3) / 1e12 / peak,
                   frac_of_peak_incl_glue=flops / (ms_p * 1e-3) / 1e12 / peak,
                   update_all_ms_incl_master_casts=ms_upd, fwd_perturbed_ms_with_logits_and_log_softmax=ms_p_logits,
                   max_fitness_difference_between_the_two_heads=float((fit - fit_logits).abs().max()))
        rows.append(res); print(json.dumps(res), flush=True)
        if args.out:
            json.dump(rows, open(args.out, "w"), indent=1)
        return
    if args.only == "q8":
        # per-channel int8 weights with discretised Adam on the config-5 layer: 4096 x 4096, one token per member.
        # HBM figures use the algorithmic bytes of each piece and the measured copy bandwidth.
        hbm = json.load(open(peaks_path)).get("hbm_gbs", 6650.0) if os.path.exists(peaks_path) else 6650.0
        m = n = 4096
        Wf = torch.randn((m, n), device="cuda") / 64
        Q = torch.empty((m, n), dtype=torch.int8, device="cuda")
        sc = torch.empty(m, dtype=torch.bfloat16, device="cuda")
        ms = t(lambda: egr.egr_q8_quantize(Wf, 1e-8, Q, sc), flush_l2=True)
        res = dict(config="q8", what="quantize 4096x4096", ms=ms, gbs=m * n * 5 / (ms * 1e-3) / 1e9, bytes_per_element=5)
        res["frac_of_hbm"] = res["gbs"] / hbm
        rows.append(res); print(json.dumps(res), flush=True)
        for N in ([4096, 65536] if not args.quick else [4096]):
            X = torch.randn((N, n), device="cuda").to(torch.bfloat16)
            Y = torch.empty((N, m), dtype=torch.bfloat16, device="cuda")
            Wb = Q.to(torch.bfloat16)
            Lq = lambda fl=0: egr.Layer(n, m, N, 1, 1, seed=1, flags=fl, x_dtype=egr.BF16, w_dtype=egr.I8, y_dtype=egr.BF16)
            Lb = lambda fl=0: egr.Layer(n, m, N, 1, 1, seed=1, flags=fl)
            res = dict(config="q8", what="forward", N=N, n=n, m=m, r=1)
            res["q8_ms"] = t(lambda: egr.egr_perturbed_linear_q8(Lq(), X, Q, sc, 1.0, 4.0, 0.0, Y, ws))
            res["q8_scale_noise_ms"] = t(lambda: egr.egr_perturbed_linear_q8(Lq(), X, Q, sc, 1.0, 4.0, 1e-4, Y, ws))
            res["q8_unperturbed_ms"] = t(lambda: egr.egr_perturbed_linear_q8(Lq(egr.NO_PERTURB), X, Q, sc, 1.0, 4.0, 0.0, Y, ws))
            res["bf16_ms"] = t(lambda: egr.egr_perturbed_linear(Lb(), X, Wb, 4.0, Y, ws))
            res["torch_ms"] = t(lambda: torch.matmul(X, Wb.t(), out=Y))
            res["q8_tflops"] = 2.0 * N * n * m / (res["q8_ms"] * 1e-3) / 1e12
            res["q8_frac_of_peak"] = res["q8_tflops"] / peak
            res["pct_of_unperturbed"] = 100 * res["q8_unperturbed_ms"] / res["q8_ms"]
            res["pct_of_torch"] = 100 * res["torch_ms"] / res["q8_ms"]
            assert egr.egr_workspace_status(ws) == 0
            shaped = torch.randn(N, device="cuda")
            G = torch.empty((m, n), dtype=torch.float32, device="cuda")
            res["gradient_ms"] = t(lambda: egr.egr_es_gradient(Lb(), shaped, G, ws))
            res["gradient_tflops"] = 2.0 * m * n * N / (res["gradient_ms"] * 1e-3) / 1e12
            gs = torch.empty(m + 1, dtype=torch.float32, device="cuda")
            res["scale_gradient_ms"] = t(lambda: egr.egr_es_scale_gradient(Lb(), shaped, gs, ws))
            res["scale_gradient_normals_per_s"] = N * (m + 1) / (res["scale_gradient_ms"] * 1e-3)
            rows.append(res); print(json.dumps(res), flush=True)
            del X, Y, Wb
        m1 = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
        m2 = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
        G = torch.randn((m, n), device="cuda")
        step = [0]

        def adam():
            step[0] += 1
            egr.egr_adam_step_q8(Q, G, m1, m2, step[0], 1e-2, 0.9, 0.999, 1e-8, 1.0, ws)
        ms = t(adam, flush_l2=True)
        # per element: G 4 B, both moments read and written 8 B, u written and read 4 B, Q read and written 2 B
        res = dict(config="q8", what="adam_step_q8 4096x4096 (2 kernels)", ms=ms, gbs=m * n * 18 / (ms * 1e-3) / 1e9,
                   bytes_per_element=18)
        res["frac_of_hbm"] = res["gbs"] / hbm
        rows.append(res); print(json.dumps(res), flush=True)
        if args.out:
            json.dump(rows, open(args.out, "w"), indent=1)
        return
    if want("rates"):
        # two machine rates the rooflines of the noise-bound and integer pieces refer to
        # (a) pure generation: one factor of 2^26 normals written to memory (fast path, as in the bf16 kernels)
        cnt = 1 << 26
        out = torch.empty(cnt, dtype=torch.float32, device="cuda")
        Lg = egr.Layer(64, cnt // 16, 2, 1, 16, seed=3)
        ms = t(lambda: egr.egr_noise_materialize(Lg, 0, 0, False, out))
        res = dict(config="rates", what="noise_materialize fast path", normals=cnt, ms=ms, normals_per_s=cnt / (ms * 1e-3))
        rows.append(res); print(json.dumps(res), flush=True)
        del out
        # (b) int8 tensor-core GEMM of this library, 8192^3, with and without the rank-1 term
        n8 = 8192
        Xi = torch.randint(-127, 128, (n8, n8), dtype=torch.int8, device="cuda")
        Wi = torch.randint(-127, 128, (n8, n8), dtype=torch.int8, device="cuda")
        Yi = torch.empty((n8, n8), dtype=torch.int8, device="cuda")
        tab = torch.from_numpy(workloads.noise_table(0, 24)).cuda()
        for nm, fl in (("int8 GEMM 8192^3 unperturbed", egr.NO_PERTURB), ("int8 GEMM 8192^3 perturbed", 0)):
            Li = egr.Layer(n8, n8, n8, 1, 1, seed=1, flags=fl, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
            ms = t(lambda: egr.egr_perturbed_linear_i8(Li, Xi, Wi, 8, 10, tab, Yi, ws))
            res = dict(config="rates", what=nm, ms=ms, int8_tops=2.0 * n8 ** 3 / (ms * 1e-3) / 1e12)
            rows.append(res); print(json.dumps(res), flush=True)
        del Xi, Wi, Yi
    if not want("c3"):
        if args.out:
            json.dump(rows, open(args.out, "w"), indent=1)
        return
    # config 3: integer recurrent LM, N = 16384 members, 128 bytes per sequence
    D, l, N, n_seq, seq_len = 256, 4, 16384, 16, args.seq_len
    P = {k: torch.from_numpy(np.ascontiguousarray(v)).cuda() for k, v in workloads.egg_lm_params(0, D, l).items()}
    tokens = torch.from_numpy(workloads.markov_bytes(0, n_seq, seq_len)).cuda()
    table = torch.from_numpy(workloads.noise_table(0, 24)).cuda()
    mseq = torch.from_numpy(((np.arange(N) // 2) % n_seq).astype(np.int32)).cuda()
    state = torch.zeros((l, N, D), dtype=torch.int8, device="cuda")
    fit = torch.zeros(N, dtype=torch.int32, device="cuda")
    ms = t(lambda: egr.egr_i8lm_forward(P, N, 0, egr.ANTITHETIC, 8, table, tokens, mseq, state, fit, ws), reps=5, warm=2)
    macs = 3.21e6 * N * (seq_len - 1)
    res = dict(config="c3", N=N, positions=seq_len - 1, fwd_ms=ms, tokens_per_s=N * (seq_len - 1) / (ms * 1e-3),
               int8_tops=2 * macs / (ms * 1e-3) / 1e12)
    # the same pass captured once into a CUDA graph and replayed (the call is capturable; with the one-launch kernel there
    # is little host work left to remove)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            egr.egr_i8lm_forward(P, N, 0, egr.ANTITHETIC, 8, table, tokens, mseq, state, fit, ws)
    torch.cuda.synchronize()
    res["fwd_graph_replay_ms"] = t(graph.replay, reps=5, warm=2)
    res["tokens_per_s_graph_replay"] = N * (seq_len - 1) / (res["fwd_graph_replay_ms"] * 1e-3)
    # one whole integer-EGGROLL training step: forward, pair signs, one-bin update of all 26 perturbed matrices
    from paper_2511_16652_b200 import egg

    def step():
        state.zero_()
        egg.egg_step(P, N, 1, 8, table, tokens, mseq, state, 0.5, ws)
    res["egg_step_ms"] = t(step, reps=5, warm=2)
    res["egg_update_ms"] = res["egg_step_ms"] - ms
    rows.append(res)
    print(json.dumps(res), flush=True)
    if args.out:
        json.dump(rows, open(args.out, "w"), indent=1)


if __name__ == "__main__":
    main()

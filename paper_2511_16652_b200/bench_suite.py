"""Throughput of the library on the benchmark configurations, beyond the single line bench.py prints.

    python -m paper_2511_16652_b200.bench_suite [--out FILE.json] [--quick]

For every point it reports the perturbed forward, the library's own unperturbed kernel, torch.matmul (library
comparison), the update, and -- for the one-token-per-member sweep -- a naive full-rank-ES baseline in which every
member's W + sigma*E_i is materialised (torch ops, random factors standing in for the noise) and applied with a
batched matrix-vector product.  Times are CUDA-event averages after warm-up; all inputs are synthetic.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    import torch

    import paper_2511_16652_b200 as egr
    import workloads

    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default=None)
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--only", default=None, choices=["c2", "c3", "c4", "c5", "rates"], help="run one configuration only")
    args = ap.parse_args()
    egr.load_library()
    ws = egr.Workspace()
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = json.load(open(peaks_path)).get("bf16_tflops_sustained", 1400.0) if os.path.exists(peaks_path) else 1400.0

    def t(fn, reps=5, warm=2):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

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
        res["upd_ms"] = t(lambda: egr.egr_es_update(L(), Wm, shaped, 0.01, ws, W_shadow=W), reps=3, warm=1)
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
            ms_mat, ms_app = t(materialise, 3, 1), t(apply_only, 3, 1)
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

    if want("rates"):
        # two machine rates the rooflines of the noise-bound and integer pieces refer to
        # (a) pure generation: one factor of 2^26 normals written to memory (fast path, as in the bf16 kernels)
        cnt = 1 << 26
        out = torch.empty(cnt, dtype=torch.float32, device="cuda")
        Lg = egr.Layer(64, cnt // 16, 2, 1, 16, seed=3)
        ms = t(lambda: egr.egr_noise_materialize(Lg, 0, 0, False, out), reps=5, warm=2)
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
            ms = t(lambda: egr.egr_perturbed_linear_i8(Li, Xi, Wi, 8, 10, tab, Yi, ws), reps=5, warm=2)
            res = dict(config="rates", what=nm, ms=ms, int8_tops=2.0 * n8 ** 3 / (ms * 1e-3) / 1e12)
            rows.append(res); print(json.dumps(res), flush=True)
        del Xi, Wi, Yi
    if not want("c3"):
        if args.out:
            json.dump(rows, open(args.out, "w"), indent=1)
        return
    # config 3: integer recurrent LM, N = 16384 members, 128 bytes per sequence
    D, l, N, n_seq, seq_len = 256, 4, 16384, 16, 128
    P = {k: torch.from_numpy(np.ascontiguousarray(v)).cuda() for k, v in workloads.egg_lm_params(0, D, l).items()}
    tokens = torch.from_numpy(workloads.markov_bytes(0, n_seq, seq_len)).cuda()
    table = torch.from_numpy(workloads.noise_table(0, 24)).cuda()
    mseq = torch.from_numpy(((np.arange(N) // 2) % n_seq).astype(np.int32)).cuda()
    state = torch.zeros((l, N, D), dtype=torch.int8, device="cuda")
    fit = torch.zeros(N, dtype=torch.int32, device="cuda")
    ms = t(lambda: egr.egr_i8lm_forward(P, N, 0, egr.ANTITHETIC, 8, table, tokens, mseq, state, fit, ws), reps=2, warm=1)
    macs = 3.21e6 * N * (seq_len - 1)
    res = dict(config="c3", N=N, positions=seq_len - 1, fwd_ms=ms, tokens_per_s=N * (seq_len - 1) / (ms * 1e-3),
               int8_tops=2 * macs / (ms * 1e-3) / 1e12)
    rows.append(res)
    print(json.dumps(res), flush=True)
    if args.out:
        json.dump(rows, open(args.out, "w"), indent=1)


if __name__ == "__main__":
    main()

"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on identical seeded inputs.

Tolerances: bit-exact for the generator's integer stream, the integer path and every index decision;
relative Frobenius error <= 1e-5 for fp32 paths and <= 1e-2 for bf16-input / fp32-accumulate paths.
"""
import math

import numpy as np
import pytest

import oracle
import workloads
from util import padded, rel_fro, to_dev

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-5
TOL_BF16 = 1e-2


@pytest.fixture(scope="module")
def egr():
    import torch
    assert torch.cuda.is_available()
    import paper_2511_16652_b200 as m
    m.load_library()          # raises if the extension is missing: no fallback
    return m


@pytest.fixture()
def ws(egr):
    return egr.Workspace()


# ------------------------------------------------------------------------------------------ generator
def test_philox_stream_is_bit_exact(egr):
    import torch
    g = workloads.rng(1, 50)
    ctr = g.integers(0, 2 ** 32, size=(20000, 4), dtype=np.uint64).astype(np.uint32)
    ctr[0] = 0
    ctr[1] = 0xFFFFFFFF
    key = [0xDEADBEEF, 0x12345678]
    out = torch.zeros((ctr.shape[0], 4), dtype=torch.int32, device="cuda")
    egr.egr_philox4x32_10_device(to_dev(ctr.view(np.int32)), key, out)
    got = out.cpu().numpy().view(np.uint32)
    want = np.stack([oracle.philox4x32_10(c, key) for c in ctr])
    assert np.array_equal(got, want)


@pytest.mark.parametrize("r,which", [(1, 0), (4, 1), (16, 0), (2, 1), (8, 0)])
def test_noise_factors_match(egr, r, which):
    import torch
    L = egr.Layer(777 if which else 300, 300 if which else 777, 64, rank=r, layer_id=5, seed=0xABCDEF0123, flags=egr.ANTITHETIC)
    rows = 777
    for member in (0, 1, 37):
        want = oracle.noise_factor(0xABCDEF0123, 5, member >> 1, which, rows, r)
        for precise, tol in ((True, 2e-6), (False, 2e-5)):
            out = torch.zeros((rows, r), dtype=torch.float32, device="cuda")
            egr.egr_noise_materialize(L, member, which, precise, out)
            got = out.cpu().numpy().astype(np.float64)
            assert np.abs(got - want).max() < tol, (precise, np.abs(got - want).max())
            assert rel_fro(got, want) < (2e-7 if precise else 3e-6)


# ------------------------------------------------------------------------------------------ fp32 path
F32_CASES = [
    # N, T, m, n, r, antithetic, ldx_pad
    (32, 1, 64, 64, 1, True, 0),
    (70, 1, 10, 784, 4, False, 4),
    (18, 3, 130, 96, 16, True, 0),
    (9, 5, 67, 33, 2, False, 3),
    (6, 2, 200, 260, 8, True, 0),
]


@pytest.mark.parametrize("N,T,m,n,r,anti,pad", F32_CASES)
def test_forward_fp32(egr, ws, N, T, m, n, r, anti, pad):
    import torch
    W, X = workloads.linear_layer(3, m, n, N * T, bf16=False)
    ldx = (n + 3) // 4 * 4 + pad * 4
    ldw = (n + 3) // 4 * 4
    ldy = (m + 3) // 4 * 4
    flags = egr.ANTITHETIC if anti else 0
    L = egr.Layer(n, m, N, T, r, layer_id=2, seed=11, flags=flags, x_dtype=egr.F32, w_dtype=egr.F32, y_dtype=egr.F32,
                  ldx=ldx, ldw=ldw, ldy=ldy)
    Xd, Wd = padded(X, ldx), padded(W, ldw)
    Yd = torch.full((N * T, ldy), 7.0, dtype=torch.float32, device="cuda")
    egr.egr_perturbed_linear(L, Xd, Wd, 0.1, Yd, ws)
    torch.cuda.synchronize()
    want = oracle.perturbed_linear(X, W, np.arange(N), T, r, 2, 11, flags, 0.1)
    got = Yd.cpu().numpy()
    assert rel_fro(got[:, :m], want) < TOL_F32
    assert np.all(got[:, m:] == 7.0)                      # pitch padding untouched
    # the low-rank term alone must also agree (it is small next to the dense product)
    L0 = egr.Layer(n, m, N, T, r, layer_id=2, seed=11, flags=flags | egr.NO_PERTURB, x_dtype=egr.F32, w_dtype=egr.F32,
                   y_dtype=egr.F32, ldx=ldx, ldw=ldw, ldy=ldy)
    Y0 = torch.zeros_like(Yd)
    egr.egr_perturbed_linear(L0, Xd, Wd, 0.1, Y0, ws)
    base = X.astype(np.float64) @ W.astype(np.float64).T
    assert rel_fro(Y0.cpu().numpy()[:, :m], base) < TOL_F32
    assert rel_fro(got[:, :m] - base, want - base) < 2e-4


@pytest.mark.parametrize("N,m,n,r,anti", [(32, 64, 64, 1, True), (50, 70, 130, 4, False), (24, 10, 784, 16, True),
                                          (1000, 96, 64, 2, True), (7, 33, 65, 8, False)])
def test_update_fp32(egr, ws, N, m, n, r, anti):
    import torch
    W = workloads.linear_layer(4, m, n, 1, bf16=False)[0]
    f = workloads.raw_fitness(4, N)
    flags = egr.ANTITHETIC if anti else 0
    ldw = (n + 3) // 4 * 4 + 4
    L = egr.Layer(n, m, N, 1, r, layer_id=9, seed=2 ** 40 + 5, flags=flags, x_dtype=egr.F32, w_dtype=egr.F32,
                  y_dtype=egr.F32, ldw=ldw)
    Wd = padded(W, ldw)
    dW = torch.zeros((m, n), dtype=torch.float32, device="cuda")
    egr.egr_es_update(L, Wd, to_dev(f), 0.37, ws, dW_out=dW)
    torch.cuda.synchronize()
    Wn, dWo = oracle.es_update(W, f, r, 9, 2 ** 40 + 5, flags, 0.37)
    assert rel_fro(dW.cpu().numpy(), dWo) < TOL_F32
    assert rel_fro(Wd.cpu().numpy()[:, :n], Wn) < TOL_F32
    assert np.all(Wd.cpu().numpy()[:, n:] == 0)


def test_update_fp32_constant_fitness_cancels_exactly(egr, ws):
    import torch
    m, n, N = 64, 64, 32
    L = egr.Layer(n, m, N, 1, 4, flags=egr.ANTITHETIC, x_dtype=egr.F32, w_dtype=egr.F32, y_dtype=egr.F32)
    W = to_dev(workloads.linear_layer(4, m, n, 1, bf16=False)[0])
    W0 = W.clone()
    egr.egr_es_update(L, W, torch.full((N,), 2.5, device="cuda"), 0.5, ws)
    assert torch.equal(W, W0)


def test_config1_ten_es_steps(egr, ws):
    """Config 1: one fp32 64x64 layer, 16 antithetic pairs, r=1, centred ranks, 10 steps (teacher-forced and free)."""
    import torch
    c = workloads.config1()
    N, T, r, sigma, alpha = c["N"], c["T"], c["r"], c["sigma"], c["alpha"]
    X, t = c["X"], c["target"].astype(np.float64)
    flags = oracle.ANTITHETIC
    W_o = c["W"].astype(np.float64)
    W_free = to_dev(c["W"])
    Xd = to_dev(X)
    Y = torch.zeros((N, 64), dtype=torch.float32, device="cuda")
    shaped = torch.zeros(N, dtype=torch.float32, device="cuda")
    for step in range(c["steps"]):
        seed = c["seed"] + step
        L = egr.Layer(64, 64, N, T, r, layer_id=0, seed=seed, flags=egr.ANTITHETIC, x_dtype=egr.F32, w_dtype=egr.F32,
                      y_dtype=egr.F32)
        # oracle step
        Yo = oracle.perturbed_linear(X, W_o, np.arange(N), T, r, 0, seed, flags, sigma)
        fo = -np.sum((Yo - t) ** 2, axis=1)
        so = oracle.fitness_shape(fo.astype(np.float32), oracle.SHAPE_CENTERED_RANK)
        W_next, _ = oracle.es_update(W_o, so, r, 0, seed, flags, alpha)
        # teacher-forced GPU step from the oracle's weights
        W_tf = to_dev(W_o.astype(np.float32))
        egr.egr_perturbed_linear(L, Xd, W_tf, sigma, Y, ws)
        assert rel_fro(Y.cpu().numpy(), Yo) < TOL_F32
        fit = -((Y - to_dev(c["target"])) ** 2).sum(dim=1)
        egr.egr_fitness_shape(fit.contiguous(), egr.SHAPE_CENTERED_RANK, shaped, ws)
        gaps = np.diff(np.sort(fo))
        if gaps.min() > 1e-4 * np.abs(fo).max():          # ranks are discontinuous: only compare without near-ties
            assert np.array_equal(shaped.cpu().numpy().astype(np.float64), so)
        egr.egr_es_update(L, W_tf, to_dev(so.astype(np.float32)), alpha, ws)
        assert rel_fro(W_tf.cpu().numpy(), W_next) < TOL_F32
        # free-running GPU chain
        egr.egr_perturbed_linear(L, Xd, W_free, sigma, Y, ws)
        fit = -((Y - to_dev(c["target"])) ** 2).sum(dim=1)
        egr.egr_fitness_shape(fit.contiguous(), egr.SHAPE_CENTERED_RANK, shaped, ws)
        egr.egr_es_update(L, W_free, shaped, alpha, ws)
        W_o = W_next
    assert rel_fro(W_free.cpu().numpy(), W_o) < 1e-4        # free-running: rank flips at near-ties are allowed for


# ------------------------------------------------------------------------------------------ shaping
@pytest.mark.parametrize("N", [2, 32, 1000, 4097, 65536])
def test_centred_rank_bit_exact(egr, ws, N):
    import torch
    raw = workloads.raw_fitness(N, N)
    if N >= 1000:
        raw[::7] = raw[3]                 # many ties
        raw[5] = np.nan
        raw[11] = -0.0
        raw[12] = 0.0
    out = torch.zeros(N, dtype=torch.float32, device="cuda")
    egr.egr_fitness_shape(to_dev(raw), egr.SHAPE_CENTERED_RANK, out, ws)
    want = oracle.fitness_shape(raw, oracle.SHAPE_CENTERED_RANK)
    assert np.array_equal(out.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("kind", ["all_equal", "narrow_band", "integers", "two_values", "nan_heavy", "signed_zeros", "sorted_desc"])
@pytest.mark.parametrize("N", [1023, 1025, 65536, 300001])
def test_centred_rank_on_clustered_and_tied_fitness(egr, ws, N, kind):
    """Fitness values that crowd into a few distinct numbers or into a narrow band (log-likelihoods of similar
    members, integer scores, a constant): the ranks stay bit-exact and the cost does not depend on the distribution."""
    import torch
    g = workloads.rng(N, 77)
    if kind == "all_equal":
        raw = np.full(N, -2650.25, dtype=np.float32)
    elif kind == "narrow_band":
        raw = (-2650.0 + 2.0 * g.random(N) - 1.0).astype(np.float32)       # a few thousand distinct floats at most
    elif kind == "integers":
        raw = g.integers(-3, 4, size=N).astype(np.float32)
    elif kind == "two_values":
        raw = np.where(g.random(N) < 0.5, 1.0, -1.0).astype(np.float32)
    elif kind == "nan_heavy":
        raw = g.standard_normal(N).astype(np.float32)
        raw[g.random(N) < 0.3] = np.nan
    elif kind == "signed_zeros":
        raw = np.where(g.random(N) < 0.5, 0.0, -0.0).astype(np.float32)
        raw[::5] = g.standard_normal(len(raw[::5])).astype(np.float32) * 1e-30
    else:
        raw = np.sort(g.standard_normal(N).astype(np.float32))[::-1].copy()
    out = torch.zeros(N, dtype=torch.float32, device="cuda")
    egr.egr_fitness_shape(to_dev(raw), egr.SHAPE_CENTERED_RANK, out, ws)
    got = out.cpu().numpy()
    if N <= 65536:
        want = oracle.fitness_shape(raw, oracle.SHAPE_CENTERED_RANK)
        assert np.array_equal(got.astype(np.float64), want)
    else:
        # the definition's order: NaN first (worst), -0 == +0, ties by index
        key = np.where(np.isnan(raw), -np.inf, raw + np.float32(0.0)).astype(np.float64)
        order = np.argsort(key, kind="stable")
        asc = np.empty(N, dtype=np.int64)
        asc[order] = np.arange(N)
        want = ((2 * asc - (N - 1)).astype(np.float32) / np.float32(2 * (N - 1))).astype(np.float32)
        assert np.array_equal(got, want)


@pytest.mark.parametrize("N", [8, 1001, 65536])
def test_zscore_sign_and_copy(egr, ws, N):
    import torch
    raw = workloads.raw_fitness(N + 1, N) * 3 + 5
    out = torch.zeros(N, dtype=torch.float32, device="cuda")
    egr.egr_fitness_shape(to_dev(raw), egr.SHAPE_ZSCORE, out, ws)
    assert rel_fro(out.cpu().numpy(), oracle.fitness_shape(raw, oracle.SHAPE_ZSCORE)) < TOL_F32
    egr.egr_fitness_shape(to_dev(raw), egr.SHAPE_NONE, out, ws)
    assert np.array_equal(out.cpu().numpy(), raw)
    if N % 2 == 0:
        raw[4] = raw[5]
        egr.egr_fitness_shape(to_dev(raw), egr.SHAPE_ANTITHETIC_SIGN, out, ws)
        assert np.array_equal(out.cpu().numpy().astype(np.float64), oracle.fitness_shape(raw, oracle.SHAPE_ANTITHETIC_SIGN))
        ri = (raw * 1000).astype(np.int32)
        oi = torch.zeros(N // 2, dtype=torch.int8, device="cuda")
        egr.egr_fitness_shape_i8(to_dev(ri), oi)
        assert np.array_equal(oi.cpu().numpy(), oracle.fitness_shape_i8(ri))


# ------------------------------------------------------------------------------------------ integer path
@pytest.mark.parametrize("N,T,m,n,anti,sshift,oshift", [(64, 1, 256, 256, True, 8, 8), (10, 3, 100, 64, False, 5, 7),
                                                       (33, 1, 1024, 256, False, 8, 8), (16, 2, 256, 1024, True, 8, 9),
                                                       (5, 1, 7, 16, False, 0, 3)])
def test_forward_int8_bit_exact(egr, ws, N, T, m, n, anti, sshift, oshift):
    import torch
    X = workloads.int8_activations(1, 30, (N * T, n))
    W = workloads.int8_matrix(1, 31, (m, n))
    table = workloads.noise_table(1, 16)
    flags = egr.ANTITHETIC if anti else 0
    L = egr.Layer(n, m, N, T, 1, layer_id=1001, seed=77, flags=flags, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
    Y = torch.zeros((N * T, m), dtype=torch.int8, device="cuda")
    egr.egr_perturbed_linear_i8(L, to_dev(X), to_dev(W), sshift, oshift, to_dev(table), Y, ws)
    want = oracle.perturbed_linear_i8(X, W, np.arange(N), T, 1001, 77, flags, sshift, oshift, table)
    assert np.array_equal(Y.cpu().numpy(), want)
    assert Y.min().item() >= -127


@pytest.mark.parametrize("N,m,n,anti", [(128, 256, 256, True), (100, 70, 130, False), (8192, 64, 64, True),
                                        (600, 520, 304, False)])     # several tiles, ragged edges, padded noise indices
def test_update_int8_bit_exact(egr, ws, N, m, n, anti):
    import torch
    P = N // 2 if anti else N
    table = workloads.noise_table(2, 16)
    F = workloads.rng(2, 40).integers(-1, 2, size=P).astype(np.int8)
    W = workloads.int8_matrix(2, 31, (m, n))
    thr = int(16 * 0.6745) * int(16 * math.sqrt(P))
    flags = egr.ANTITHETIC if anti else 0
    L = egr.Layer(n, m, N, 1, 1, layer_id=3, seed=5, flags=flags, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
    Wd = to_dev(W)
    E = torch.zeros((m, n), dtype=torch.int32, device="cuda")
    egr.egr_es_update_i8(L, Wd, to_dev(F), thr, to_dev(table), ws, E_out=E)
    Wn, Eo = oracle.es_update_i8(W, F, 3, 5, thr, table)
    assert np.array_equal(E.cpu().numpy(), Eo)
    assert np.array_equal(Wd.cpu().numpy(), Wn)


# ------------------------------------------------------------------------------------------ bf16 tensor-core path
BF16_CASES = [
    # N, T, m, n, r, antithetic
    (128, 1, 256, 64, 1, False),          # exactly one tile, one k-block
    (300, 1, 520, 200, 4, True),          # ragged rows, columns and K
    (64, 8, 1024, 784, 4, True),          # config-2 first layer shape, 8 rows per member
    (40, 3, 10, 1024, 16, False),         # 10 output columns
    (257, 1, 264, 4096, 2, False),
    (96, 2, 512, 520, 8, True),
    (6, 64, 520, 200, 1, True),           # 32 | T: a warp's rows share one member (noise generated once per warp)
    (3, 96, 300, 264, 16, False),
    (10, 32, 264, 128, 4, True),
    (300, 1, 264, 136, 1, True),          # antithetic pairs, one token each: groups of 2 rows share the noise
    (64, 4, 264, 136, 16, True),          # groups of 8
    (40, 8, 520, 264, 2, False),          # groups of 8, rank 2
    (12, 16, 264, 128, 8, False),         # groups of 16
    (34, 6, 136, 264, 4, True),           # run of 12 rows: groups of 4
    (20, 16, 264, 200, 16, False),        # groups of 16, rank 16: the factors are exchanged in two rounds
    (6, 32, 136, 264, 8, True),           # whole warps of one member, rank 8
    (10, 16, 1000, 72, 4, True),          # runs of 32 rows, four column tiles, the last one ragged
    # long contractions (the skinny products come from the kernel's side warps): rows claimed one by one and in halves
    # of K, a ragged last band that is not split; and four-row claims with the first 2048 rows in halves, the last
    # tile of every CTA pair shared with the tail helpers
    (1000, 1, 520, 2048, 4, False),
    (3000, 1, 264, 1536, 1, True),
    (2300, 1, 520, 1280, 2, False),
]


def _check_status(egr, ws):
    rc = egr.egr_workspace_status(ws)
    assert rc == 0, egr.egr_strerror(rc)


@pytest.mark.parametrize("N,T,m,n,r,anti", BF16_CASES)
@pytest.mark.parametrize("y_f32", [False, True])
def test_forward_bf16(egr, ws, N, T, m, n, r, anti, y_f32):
    import torch
    W, X = workloads.linear_layer(6, m, n, N * T, bf16=True)
    flags = egr.ANTITHETIC if anti else 0
    ldx = (n + 7) // 8 * 8 + 8
    ldw = (n + 7) // 8 * 8
    ldy = (m + 7) // 8 * 8
    ydt = torch.float32 if y_f32 else torch.bfloat16
    L = egr.Layer(n, m, N, T, r, layer_id=4, seed=31, flags=flags, x_dtype=egr.BF16, w_dtype=egr.BF16,
                  y_dtype=egr.F32 if y_f32 else egr.BF16, ldx=ldx, ldw=ldw, ldy=ldy)
    Xd, Wd = padded(X, ldx, torch.bfloat16), padded(W, ldw, torch.bfloat16)
    Yd = torch.full((N * T, ldy), 3.0, dtype=ydt, device="cuda")
    sigma = 0.05
    egr.egr_perturbed_linear(L, Xd, Wd, sigma, Yd, ws)
    _check_status(egr, ws)
    want = oracle.perturbed_linear(X, W, np.arange(N), T, r, 4, 31, flags, sigma)
    got = Yd.float().cpu().numpy()
    assert rel_fro(got[:, :m], want) < (1e-4 if y_f32 else TOL_BF16)
    assert np.all(got[:, m:] == 3.0)
    L0 = egr.Layer(n, m, N, T, r, layer_id=4, seed=31, flags=flags | egr.NO_PERTURB, x_dtype=egr.BF16, w_dtype=egr.BF16,
                   y_dtype=egr.F32 if y_f32 else egr.BF16, ldx=ldx, ldw=ldw, ldy=ldy)
    Y0 = torch.zeros_like(Yd)
    egr.egr_perturbed_linear(L0, Xd, Wd, sigma, Y0, ws)
    _check_status(egr, ws)
    base = X.astype(np.float64) @ W.astype(np.float64).T
    assert rel_fro(Y0.float().cpu().numpy()[:, :m], base) < (1e-5 if y_f32 else TOL_BF16)
    if y_f32:
        assert rel_fro(got[:, :m] - base, want - base) < 1e-3      # the low-rank term alone


@pytest.mark.parametrize("N,m,n,r,anti", [(64, 128, 256, 1, False), (200, 300, 520, 4, True), (1000, 10, 784, 16, False),
                                          (4096, 264, 200, 2, True), (24, 1024, 1024, 8, False)])
def test_update_bf16(egr, ws, N, m, n, r, anti):
    import torch
    W = workloads.linear_layer(8, m, n, 1, bf16=True)[0]
    f = workloads.raw_fitness(8, N)
    flags = egr.ANTITHETIC if anti else 0
    ldw = (n + 7) // 8 * 8
    L = egr.Layer(n, m, N, 1, r, layer_id=6, seed=1234567, flags=flags, x_dtype=egr.BF16, w_dtype=egr.BF16,
                  y_dtype=egr.BF16, ldw=ldw)
    Wm = padded(W, ldw)                                  # fp32 master
    Wsh = torch.zeros((m, ldw), dtype=torch.bfloat16, device="cuda")
    dW = torch.zeros((m, n), dtype=torch.float32, device="cuda")
    alpha = 0.8
    egr.egr_es_update(L, Wm, to_dev(f), alpha, ws, W_shadow=Wsh, dW_out=dW)
    _check_status(egr, ws)
    Wn, dWo = oracle.es_update(W, f, r, 6, 1234567, flags, alpha)
    assert rel_fro(dW.cpu().numpy(), dWo) < TOL_BF16
    assert rel_fro(Wm.cpu().numpy()[:, :n] - W, dWo) < TOL_BF16
    assert torch.equal(Wsh[:, :n], Wm[:, :n].to(torch.bfloat16))     # shadow = RNE(master)


@pytest.mark.parametrize("N,m,n,r,anti,shadow", [
    (64, 128, 256, 1, False, True),        # one narrow-tile launch, K = 64
    (200, 300, 520, 4, True, True),        # ragged rows and columns, K = 400
    (1024, 264, 200, 2, True, False),      # no shadow, K = 1024
    (2048, 520, 776, 1, False, True),      # K = 2048: the longest contraction that takes this path
    (96, 1024, 1032, 8, False, True),      # several 256-wide tiles, K = 768
    (512, 40, 72, 1, True, False),         # fewer rows than one tile
    (300, 130, 203, 2, False, True),       # rows that are not whole 16-byte pieces: the register epilogue instead
])
def test_update_bf16_as_a_real_caller_runs_it(egr, ws, N, m, n, r, anti, shadow):
    """The boxed EGGROLL update without the test-only `dW_out`: short contractions (K = N r <= 2048) then add
    `scale * acc` to the fp32 master with bulk reduce-add stores and write the bf16 shadow in a pass of its own.
    Checked on what the caller sees: the change of the master against the oracle's sum of outer products, the
    shadow against the rounding of the master, and the pitch padding left alone."""
    import torch
    W = workloads.linear_layer(41, m, n, 1, bf16=True)[0]
    f = workloads.raw_fitness(41, N)
    flags = egr.ANTITHETIC if anti else 0
    ldw = (n + 7) // 8 * 8 + 8
    L = egr.Layer(n, m, N, 1, r, layer_id=3, seed=777, flags=flags, x_dtype=egr.BF16, w_dtype=egr.BF16,
                  y_dtype=egr.BF16, ldw=ldw)
    Wm = padded(W, ldw)
    Wm[:, n:] = 5.0                                       # canary in the padding
    Wsh = torch.full((m, ldw), 9.0, dtype=torch.bfloat16, device="cuda") if shadow else None
    alpha = 0.6
    egr.egr_es_update(L, Wm, to_dev(f), alpha, ws, W_shadow=Wsh)
    _check_status(egr, ws)
    Wn, dWo = oracle.es_update(W, f, r, 3, 777, flags, alpha)
    got = Wm.cpu().numpy()
    assert rel_fro(got[:, :n].astype(np.float64) - W, dWo) < TOL_BF16
    assert np.linalg.norm(got[:, :n] - Wn) < TOL_BF16 * np.linalg.norm(dWo)      # the new weights, on the scale of the change
    assert np.all(got[:, n:] == 5.0)
    if shadow:
        assert torch.equal(Wsh[:, :n], Wm[:, :n].to(torch.bfloat16))
        assert torch.all(Wsh[:, n:] == 9.0)


def test_update_bf16_without_dw_out_agrees_with_the_instrumented_call(egr, ws):
    """A transformer-sized matrix (2048 -> 8192, K = 1024, config 4's shapes): the caller's path and the path that
    also writes dW_out apply the same change (they differ by the rounding of scale * acc only), and sampled blocks
    of it equal the oracle's."""
    import torch
    m, n, N, r = 8192, 2048, 1024, 1
    W = workloads.linear_layer(42, m, n, 1, bf16=True, w_std=0.02)[0]
    f = workloads.raw_fitness(42, N)
    L = egr.Layer(n, m, N, 1, r, layer_id=20, seed=5, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16)
    fd = to_dev(f)
    Wa, Wb = to_dev(W), to_dev(W)
    Wsh = torch.zeros((m, n), dtype=torch.bfloat16, device="cuda")
    dW = torch.zeros((m, n), dtype=torch.float32, device="cuda")
    egr.egr_es_update(L, Wa, fd, 0.5, ws, W_shadow=Wsh)
    _check_status(egr, ws)
    egr.egr_es_update(L, Wb, fd, 0.5, ws, dW_out=dW)
    _check_status(egr, ws)
    W0 = to_dev(W)
    da, db = (Wa - W0).cpu().numpy(), (Wb - W0).cpu().numpy()
    assert rel_fro(da, db) < 1e-3            # W + d in fp32 loses the low bits of d on both paths
    assert torch.equal(Wsh, Wa.to(torch.bfloat16))
    for (j0, l0) in [(0, 0), (8160, 2016), (4000, 40), (128, 1920), (5000, 1000)]:
        want = oracle.es_update_block(f, r, 20, 5, 0, 0.5, j0, j0 + 32, l0, l0 + 32)
        assert rel_fro(dW.cpu().numpy()[j0:j0 + 32, l0:l0 + 32], want) < TOL_BF16
        assert rel_fro(da[j0:j0 + 32, l0:l0 + 32], want) < TOL_BF16


def test_update_bf16_multi_chunk_sampled_blocks(egr, ws):
    """K = 16384 > one staging chunk for a 2048x2048 layer; the oracle evaluates sampled 32x32 blocks."""
    import torch
    m = n = 2048
    N, r = 4096, 4
    W = workloads.linear_layer(9, m, n, 1, bf16=True)[0]
    f = workloads.raw_fitness(9, N)
    L = egr.Layer(n, m, N, 1, r, layer_id=1, seed=99, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16)
    Wm = to_dev(W)
    dW = torch.zeros((m, n), dtype=torch.float32, device="cuda")
    egr.egr_es_update(L, Wm, to_dev(f), 1.0, ws, dW_out=dW)
    _check_status(egr, ws)
    got = dW.cpu().numpy()
    for (j0, l0) in [(0, 0), (2016, 2016), (1000, 40), (128, 1920)]:
        want = oracle.es_update_block(f, r, 1, 99, 0, 1.0, j0, j0 + 32, l0, l0 + 32)
        assert rel_fro(got[j0:j0 + 32, l0:l0 + 32], want) < TOL_BF16
    assert rel_fro(Wm.cpu().numpy() - W, got) < 1e-3


# ------------------------------------------------------------------------------------------ edge cases
@pytest.mark.parametrize("N,T,m,n,r,anti", [(1, 1, 8, 8, 1, False), (2, 1, 16, 24, 16, True), (1, 300, 40, 72, 4, False),
                                            (129, 1, 8, 4096, 1, False), (3, 43, 257, 136, 2, False)])
def test_forward_bf16_degenerate_shapes(egr, ws, N, T, m, n, r, anti):
    """One member, one row, tiles that are almost empty, rows-per-member that do not divide the 128-row band."""
    import torch
    W, X = workloads.linear_layer(12, m, n, N * T, bf16=True)
    flags = egr.ANTITHETIC if anti else 0
    L = egr.Layer(n, m, N, T, r, layer_id=0xFFFFFFFF, seed=2 ** 63 + 12345, flags=flags, x_dtype=egr.BF16, w_dtype=egr.BF16,
                  y_dtype=egr.F32, ldy=(m + 3) // 4 * 4)
    Y = torch.zeros((N * T, (m + 3) // 4 * 4), dtype=torch.float32, device="cuda")
    egr.egr_perturbed_linear(L, to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16), 0.25, Y, ws)
    _check_status(egr, ws)
    want = oracle.perturbed_linear(X, W, np.arange(N), T, r, 0xFFFFFFFF, 2 ** 63 + 12345, flags, 0.25)
    assert rel_fro(Y.cpu().numpy()[:, :m], want) < 1e-4


def test_sigma_zero_equals_the_unperturbed_flag(egr, ws):
    import torch
    N, m, n = 200, 264, 520
    W, X = workloads.linear_layer(13, m, n, N, bf16=True)
    Xd, Wd = to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16)
    Y0 = torch.zeros((N, m), dtype=torch.bfloat16, device="cuda")
    Y1 = torch.zeros_like(Y0)
    egr.egr_perturbed_linear(egr.Layer(n, m, N, 1, 4, seed=1), Xd, Wd, 0.0, Y0, ws)
    egr.egr_perturbed_linear(egr.Layer(n, m, N, 1, 4, seed=1, flags=egr.NO_PERTURB), Xd, Wd, 0.3, Y1, ws)
    assert torch.equal(Y0, Y1)


def test_forward_is_deterministic_and_seed_sensitive(egr, ws):
    import torch
    N, m, n = 300, 512, 256
    W, X = workloads.linear_layer(14, m, n, N, bf16=True)
    Xd, Wd = to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16)
    outs = []
    for seed in (5, 5, 6):
        Y = torch.zeros((N, m), dtype=torch.bfloat16, device="cuda")
        egr.egr_perturbed_linear(egr.Layer(n, m, N, 1, 2, seed=seed), Xd, Wd, 0.1, Y, ws)
        outs.append(Y)
    assert torch.equal(outs[0], outs[1])
    assert not torch.equal(outs[0], outs[2])


@pytest.mark.parametrize("N,n,r", [(1500, 2048, 2), (5000, 1536, 1), (700, 4096, 4)])
def test_forward_over_a_long_contraction_gives_the_same_bits_every_time(egr, ws, N, n, r):
    """Above K = 1024 the skinny products of the first rows are added up from two halves of K by whichever side warps
    claim them; two addends onto zero must not make the result depend on who came first.  fp32 output, so that the
    low-rank term is not hidden by the output rounding."""
    import torch
    m = 264
    W, X = workloads.linear_layer(33, m, n, N, bf16=True)
    Xd, Wd = to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16)
    L = egr.Layer(n, m, N, 1, r, layer_id=2, seed=9, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.F32)
    outs = []
    for _ in range(4):
        Y = torch.zeros((N, m), dtype=torch.float32, device="cuda")
        egr.egr_perturbed_linear(L, Xd, Wd, 0.3, Y, ws)
        _check_status(egr, ws)
        outs.append(Y)
    assert all(torch.equal(outs[0], o) for o in outs[1:])
    want = oracle.perturbed_linear(X, W, np.arange(N), 1, r, 2, 9, 0, 0.3)
    assert rel_fro(outs[0].cpu().numpy(), want) < 1e-4


def test_int8_unperturbed_flag_is_the_plain_scaled_matmul(egr, ws):
    import torch
    N, m, n = 130, 256, 256
    X = workloads.int8_activations(15, 30, (N, n))
    W = workloads.int8_matrix(15, 31, (m, n))
    table = workloads.noise_table(15, 12)
    L = egr.Layer(n, m, N, 1, 1, flags=egr.NO_PERTURB, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
    Y = torch.zeros((N, m), dtype=torch.int8, device="cuda")
    egr.egr_perturbed_linear_i8(L, to_dev(X), to_dev(W), 8, 8, to_dev(table), Y, ws)
    acc = X.astype(np.int64) @ W.astype(np.int64).T
    assert np.array_equal(Y.cpu().numpy(), np.clip(acc >> 8, -127, 127).astype(np.int8))


def test_int8_forward_unaligned_pitch_takes_the_dp4a_kernel(egr, ws):
    """Pitches that are not multiples of 16 bytes cannot be fed by TMA; the dp4a kernel handles them, same bits."""
    import torch
    N, m, n = 40, 100, 68
    X = workloads.int8_activations(16, 30, (N, n))
    W = workloads.int8_matrix(16, 31, (m, n))
    table = workloads.noise_table(16, 14)
    L = egr.Layer(n, m, N, 1, 1, layer_id=7, seed=3, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
    Y = torch.zeros((N, m), dtype=torch.int8, device="cuda")
    egr.egr_perturbed_linear_i8(L, to_dev(X), to_dev(W), 6, 7, to_dev(table), Y, ws)
    want = oracle.perturbed_linear_i8(X, W, np.arange(N), 1, 7, 3, 0, 6, 7, table)
    assert np.array_equal(Y.cpu().numpy(), want)


def test_member_base_selects_a_shard_of_the_population(egr, ws):
    """A forward over members [base, base+count) with member_base = base equals those rows of the full forward."""
    import torch
    N, T, m, n, r = 24, 3, 264, 136, 4
    W, X = workloads.linear_layer(17, m, n, N * T, bf16=True)
    Xd, Wd = to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16)
    full = torch.zeros((N * T, m), dtype=torch.bfloat16, device="cuda")
    egr.egr_perturbed_linear(egr.Layer(n, m, N, T, r, seed=9, flags=egr.ANTITHETIC), Xd, Wd, 0.1, full, ws)
    for base, cnt in ((0, 10), (10, 14)):
        part = torch.zeros((cnt * T, m), dtype=torch.bfloat16, device="cuda")
        L = egr.Layer(n, m, cnt, T, r, seed=9, flags=egr.ANTITHETIC, member_base=base)
        egr.egr_perturbed_linear(L, Xd[base * T:(base + cnt) * T].contiguous(), Wd, 0.1, part, ws)
        assert torch.equal(part, full[base * T:(base + cnt) * T])
    Xi = workloads.int8_activations(17, 30, (N, 256))
    Wi = workloads.int8_matrix(17, 31, (256, 256))
    table = to_dev(workloads.noise_table(17, 14))
    fulli = torch.zeros((N, 256), dtype=torch.int8, device="cuda")
    Li = lambda cnt, base: egr.Layer(256, 256, cnt, 1, 1, seed=9, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8, member_base=base)
    egr.egr_perturbed_linear_i8(Li(N, 0), to_dev(Xi), to_dev(Wi), 8, 8, table, fulli, ws)
    parti = torch.zeros((8, 256), dtype=torch.int8, device="cuda")
    egr.egr_perturbed_linear_i8(Li(8, 16), to_dev(Xi[16:24]), to_dev(Wi), 8, 8, table, parti, ws)
    assert torch.equal(parti, fulli[16:24])


@pytest.mark.parametrize("dtype,r,anti,T", [("bf16", 1, False, 1), ("bf16", 4, True, 3), ("f32", 2, True, 2), ("bf16", 2, True, 16)])
def test_a_population_shard_matches_the_oracle(egr, ws, dtype, r, anti, T):
    """Algorithm 1's workers each evaluate their own members: a call over members [base, base + count) with
    member_base = base must regenerate exactly the noise the oracle uses for those population indices."""
    import torch
    pop, m, n = 300, 264, 136
    bf = dtype == "bf16"
    code, tdt = (egr.BF16, torch.bfloat16) if bf else (egr.F32, torch.float32)
    flags = egr.ANTITHETIC if anti else 0
    W, X = workloads.linear_layer(43, m, n, pop * T, bf16=bf)
    Wd = to_dev(W, tdt)
    for base, cnt in ((0, 34), (34, 130), (164, 136), (298, 2)):
        members = np.arange(base, base + cnt)
        Xs = X[base * T:(base + cnt) * T]
        Y = torch.zeros((cnt * T, m), dtype=torch.float32, device="cuda")
        L = egr.Layer(n, m, cnt, T, r, layer_id=8, seed=2 ** 33 + 1, flags=flags, member_base=base, x_dtype=code, w_dtype=code,
                      y_dtype=egr.F32)
        egr.egr_perturbed_linear(L, to_dev(Xs, tdt), Wd, 0.3, Y, ws)
        _check_status(egr, ws)
        want = oracle.perturbed_linear(Xs, W, members, T, r, 8, 2 ** 33 + 1, flags, 0.3)
        base_prod = Xs.astype(np.float64) @ W.astype(np.float64).T
        got = Y.cpu().numpy().astype(np.float64)
        assert rel_fro(got, want) < (1e-4 if bf else TOL_F32)
        assert rel_fro(got - base_prod, want - base_prod) < 1e-3          # the shard's own perturbations, not another shard's


def test_an_integer_population_shard_matches_the_oracle(egr, ws):
    import torch
    pop, m, n = 96, 256, 256
    X = workloads.int8_activations(44, 30, (pop, n))
    W = workloads.int8_matrix(44, 31, (m, n))
    table = workloads.noise_table(44, 14)
    for base, cnt in ((0, 16), (16, 50), (66, 30)):
        L = egr.Layer(n, m, cnt, 1, 1, layer_id=3, seed=12, flags=egr.ANTITHETIC, member_base=base, x_dtype=egr.I8,
                      w_dtype=egr.I8, y_dtype=egr.I8)
        Y = torch.zeros((cnt, m), dtype=torch.int8, device="cuda")
        egr.egr_perturbed_linear_i8(L, to_dev(X[base:base + cnt]), to_dev(W), 6, 8, to_dev(table), Y, ws)
        want = oracle.perturbed_linear_i8(X[base:base + cnt], W, np.arange(base, base + cnt), 1, 3, 12, oracle.ANTITHETIC, 6, 8, table)
        assert np.array_equal(Y.cpu().numpy(), want)


@pytest.mark.parametrize("N,Q", [(64, 1), (1000, 37), (4096, 300)])
def test_per_question_shaping(egr, ws, N, Q):
    import torch
    S = (workloads.rng(N, 8).standard_normal((N, Q)) * 2 + np.arange(Q)).astype(np.float32)
    out = torch.zeros(N, dtype=torch.float32, device="cuda")
    egr.egr_fitness_shape_questions(to_dev(S), out, ws)
    assert rel_fro(out.cpu().numpy(), oracle.fitness_shape_questions(S)) < TOL_F32


@pytest.mark.parametrize("dtype,r,anti", [("bf16", 1, False), ("bf16", 4, True), ("f32", 2, True)])
def test_forward_with_explicit_row_to_member_map(egr, ws, dtype, r, anti):
    """Ragged, interleaved rows: every row names the member whose perturbation it sees."""
    import torch
    R, m, n, pop = 333, 264, 136, 40
    bf = dtype == "bf16"
    W, X = workloads.linear_layer(18, m, n, R, bf16=bf)
    rowmap = workloads.rng(18, 4).integers(0, pop, size=R).astype(np.int32)
    rowmap[:7] = 3                                   # a run of rows of one member
    flags = egr.ANTITHETIC if anti else 0
    code = egr.BF16 if bf else egr.F32
    tdt = torch.bfloat16 if bf else torch.float32
    L = egr.Layer(n, m, R, 1, r, layer_id=2, seed=77, flags=flags, x_dtype=code, w_dtype=code, y_dtype=egr.F32)
    Y = torch.zeros((R, m), dtype=torch.float32, device="cuda")
    egr.egr_perturbed_linear_rows(L, to_dev(X, tdt), to_dev(W, tdt), to_dev(rowmap), 0.2, Y, ws)
    _check_status(egr, ws)
    want = oracle.perturbed_linear(X, W, rowmap, 1, r, 2, 77, flags, 0.2)
    assert rel_fro(Y.cpu().numpy(), want) < (1e-4 if bf else TOL_F32)


@pytest.mark.parametrize("R,r,anti", [(1333, 1, False), (3001, 2, True), (777, 4, False)])
def test_row_map_over_a_long_contraction(egr, ws, R, r, anti):
    """The same with K above 1024, where the products come from the kernel's side warps: single-row claims and four-row
    claims, rows in K-halves, a last band that is not a whole one."""
    import torch
    m, n, pop = 264, 2048, 60
    W, X = workloads.linear_layer(38, m, n, R, bf16=True)
    rowmap = workloads.rng(38, 4).integers(0, pop, size=R).astype(np.int32)
    flags = egr.ANTITHETIC if anti else 0
    L = egr.Layer(n, m, R, 1, r, layer_id=2, seed=78, flags=flags, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.F32)
    Y = torch.zeros((R, m), dtype=torch.float32, device="cuda")
    egr.egr_perturbed_linear_rows(L, to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16), to_dev(rowmap), 0.2, Y, ws)
    _check_status(egr, ws)
    want = oracle.perturbed_linear(X, W, rowmap, 1, r, 2, 78, flags, 0.2)
    assert rel_fro(Y.cpu().numpy(), want) < 1e-4


def test_centred_rank_one_million_members(egr, ws):
    """The paper's largest population (2^20 members): every rank is checked through properties that fix it uniquely
    (ranks follow the stable ascending order of the raw values), plus the oracle's own count on sampled members."""
    import torch
    N = 1 << 20
    raw = workloads.raw_fitness(99, N)
    raw[::1000] = raw[7]                                   # a thousand-fold tie
    out = torch.zeros(N, dtype=torch.float32, device="cuda")
    egr.egr_fitness_shape(to_dev(raw), egr.SHAPE_CENTERED_RANK, out, ws)
    got = out.cpu().numpy()
    order = np.argsort(raw, kind="stable")                # ascending, ties by index: the definition's order
    asc = np.empty(N, dtype=np.int64)
    asc[order] = np.arange(N)
    want = ((2 * asc - (N - 1)).astype(np.float32) / np.float32(2 * (N - 1))).astype(np.float32)
    assert np.array_equal(got, want)
    for i in (0, 7, 1000, 123456, N - 1):                  # the oracle's definition (a count) on single members
        cnt = int(np.sum((raw < raw[i]) | ((raw == raw[i]) & (np.arange(N) < i))))
        assert got[i] == np.float32(np.float32(2 * cnt - (N - 1)) / np.float32(2 * (N - 1)))


def test_forward_one_million_rows_sampled(egr, ws):
    """A long, thin problem (2^20 members x one token, 64 -> 72): row indexing far beyond one wave of tiles."""
    import torch
    N, n, m, r = 1 << 20, 64, 72, 2
    W = workloads.linear_layer(21, m, n, 1, bf16=True)[0]
    gen = torch.Generator().manual_seed(3)
    Xd = torch.randn((N, n), generator=gen, dtype=torch.float32).to(torch.bfloat16).cuda()
    Y = torch.zeros((N, m), dtype=torch.float32, device="cuda")
    L = egr.Layer(n, m, N, 1, r, seed=5, flags=egr.ANTITHETIC, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.F32)
    egr.egr_perturbed_linear(L, Xd, to_dev(W, torch.bfloat16), 0.3, Y, ws)
    _check_status(egr, ws)
    sel = np.array([0, 1, 127, 128, 255, 256, 65535, 65536, 524287, 524288, N - 2, N - 1])
    Xs = Xd[torch.from_numpy(sel).cuda()].float().cpu().numpy()
    want = oracle.perturbed_linear(Xs, W, sel, 1, r, 0, 5, oracle.ANTITHETIC, 0.3)
    assert rel_fro(Y[torch.from_numpy(sel).cuda()].cpu().numpy(), want) < 1e-4


@pytest.mark.parametrize("count", [1, 4, 5, 6, 1003, 1 << 20])
def test_base3_pack_and_unpack_bit_exact(count):
    import torch
    import paper_2511_16652_b200 as egr
    F = workloads.rng(41, count).integers(-1, 2, size=count).astype(np.int8)
    Fd = torch.from_numpy(F).cuda()
    packed = egr.egr_fitness_pack3(Fd)
    if count <= 2000:
        assert np.array_equal(packed.cpu().numpy(), oracle.pack3(F))
    else:
        # vectorised restatement of the byte formula for the large case, plus oracle bytes on a sample
        pad = np.zeros((-count) % 5, np.int8)
        digits = (1 - np.concatenate([F, pad]).astype(np.int64)).reshape(-1, 5)
        assert np.array_equal(packed.cpu().numpy(), (digits * (3 ** np.arange(5))).sum(axis=1).astype(np.uint8))
        for b in (0, 77, count // 5 - 1):
            assert int(packed[b]) == int(oracle.pack3(F[5 * b:5 * b + 5])[0])
    assert packed.numel() == (count + 4) // 5
    back = egr.egr_fitness_unpack3(packed, count)
    assert np.array_equal(back.cpu().numpy(), F)


@pytest.mark.parametrize("table_log2,offset", [(9, 0), (8, 0), (12, 4), (16, 8)])
def test_forward_int8_small_wrapping_and_misaligned_tables(egr, ws, table_log2, offset):
    """The tensor-core kernel stages every row's 256-byte table slice in shared memory with one bulk copy; a 512-byte
    table makes half of the slices wrap round its end (copied byte by byte instead), a 256-byte or a misaligned table
    switches the staging off.  Same bits in every case."""
    import torch
    N, T, m, n = 300, 1, 256, 256
    X = workloads.int8_activations(21, 30, (N * T, n))
    W = workloads.int8_matrix(21, 31, (m, n))
    table = workloads.noise_table(21, table_log2)
    buf = torch.zeros(table.size + 16, dtype=torch.int8, device="cuda")
    buf[offset:offset + table.size] = torch.from_numpy(table).cuda()
    L = egr.Layer(n, m, N, T, 1, layer_id=5, seed=13, flags=egr.ANTITHETIC, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
    Y = torch.zeros((N * T, m), dtype=torch.int8, device="cuda")
    egr.egr_perturbed_linear_i8(L, to_dev(X), to_dev(W), 8, 8, buf[offset:offset + table.size], Y, ws)
    want = oracle.perturbed_linear_i8(X, W, np.arange(N), T, 5, 13, oracle.ANTITHETIC, 8, 8, table)
    assert np.array_equal(Y.cpu().numpy(), want)


def test_a_device_side_wait_that_runs_out_reports_a_timeout_and_leaves_the_context_usable(egr, ws):
    """Every wait in the tensor-core kernels is bounded.  Here the same wait is given a barrier that nothing completes
    and a limit of 50 ms: the kernel returns by itself, the status word says EGR_ERR_TIMEOUT, and the next call works."""
    import time
    import torch
    scratch = egr.Workspace()
    t0 = time.perf_counter()
    egr.egr_debug_bounded_wait(scratch, 50)
    assert egr.egr_workspace_status(scratch) == -6           # EGR_ERR_TIMEOUT
    assert time.perf_counter() - t0 < 5.0
    assert "wait" in egr.egr_strerror(-6)
    W, X = workloads.linear_layer(29, 64, 64, 32, bf16=True)
    L = egr.Layer(64, 64, 32, 1, 1, layer_id=1, seed=2)
    Y = torch.zeros((32, 64), dtype=torch.bfloat16, device="cuda")
    egr.egr_perturbed_linear(L, to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16), 0.1, Y, ws)
    _check_status(egr, ws)
    want = oracle.perturbed_linear(X, W, np.arange(32), 1, 1, 1, 2, 0, 0.1)
    assert rel_fro(Y.float().cpu().numpy(), want) < TOL_BF16


# ------------------------------------------------------------------------------------------ element-wise function after the layer
@pytest.mark.parametrize("act", ["TANH", "RELU", "GELU"])
@pytest.mark.parametrize("dt", ["f32", "bf16", "bf16_f32out"])
def test_forward_with_activation(egr, ws, act, dt):
    """Y = act(perturbed product): several tiles with ragged edges; scaled inputs so that the function is exercised in
    its curved range.  The error is measured on act() itself, so the usual tolerances apply."""
    import torch
    N, T, m, n, r = 300, 2, 328, 200, 2
    W, X = workloads.linear_layer(9, m, n, N * T, bf16=(dt != "f32"))
    flag = getattr(egr, "ACT_" + act)
    oflag = getattr(oracle, "ACT_" + act)
    if dt == "f32":
        xd = wd = yd = egr.F32
        tdt, ydt, tol = torch.float32, torch.float32, TOL_F32
    else:
        xd = wd = egr.BF16
        yd = egr.F32 if dt == "bf16_f32out" else egr.BF16
        tdt, ydt = torch.bfloat16, (torch.float32 if dt == "bf16_f32out" else torch.bfloat16)
        tol = 1e-4 if dt == "bf16_f32out" else TOL_BF16
    L = egr.Layer(n, m, N, T, r, layer_id=6, seed=41, flags=egr.ANTITHETIC | flag, x_dtype=xd, w_dtype=wd, y_dtype=yd)
    Yd = torch.zeros((N * T, m), dtype=ydt, device="cuda")
    egr.egr_perturbed_linear(L, to_dev(X, tdt), to_dev(W, tdt), 0.2, Yd, ws)
    _check_status(egr, ws)
    want = oracle.perturbed_linear(X, W, np.arange(N), T, r, 6, 41, oracle.ANTITHETIC | oflag, 0.2)
    lin = oracle.perturbed_linear(X, W, np.arange(N), T, r, 6, 41, oracle.ANTITHETIC, 0.2)
    assert rel_fro(want, lin) > 0.05                       # the function is not acting as the identity on these inputs
    assert rel_fro(Yd.float().cpu().numpy(), want) < tol


@pytest.mark.parametrize("act", ["TANH", "GELU"])
@pytest.mark.parametrize("y_f32", [False, True])
def test_activation_on_runs_of_rows_that_share_their_noise(egr, ws, act, y_f32):
    """Eight tokens per member with antithetic pairs, rank 4: runs of 16 rows share their factors and the correction is
    added to the accumulator in another register layout than elsewhere; the function after it must see the same sums."""
    import torch
    N, T, m, n, r = 40, 8, 328, 136, 4
    W, X = workloads.linear_layer(19, m, n, N * T, bf16=True)
    L = egr.Layer(n, m, N, T, r, layer_id=8, seed=43, flags=egr.ANTITHETIC | getattr(egr, "ACT_" + act),
                  x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.F32 if y_f32 else egr.BF16)
    Yd = torch.zeros((N * T, m), dtype=torch.float32 if y_f32 else torch.bfloat16, device="cuda")
    egr.egr_perturbed_linear(L, to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16), 0.2, Yd, ws)
    _check_status(egr, ws)
    want = oracle.perturbed_linear(X, W, np.arange(N), T, r, 8, 43, oracle.ANTITHETIC | getattr(oracle, "ACT_" + act), 0.2)
    assert rel_fro(Yd.float().cpu().numpy(), want) < (1e-4 if y_f32 else TOL_BF16)


def test_activation_bits_are_rejected_outside_the_forward(egr, ws):
    import torch
    L = egr.Layer(64, 64, 8, 1, 1, flags=egr.ACT_TANH)
    Wm = torch.zeros((64, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(egr.EgrError):
        egr.egr_es_update(L, Wm, torch.zeros(8, device="cuda"), 0.1, ws)


def test_activation_with_row_map_and_static_entry(egr, ws):
    """The element-wise function goes through every forward entry point: explicit row map and the allocation-free call."""
    import torch
    R, m, n, pop, r = 200, 136, 72, 24, 2
    W, X = workloads.linear_layer(19, m, n, R, bf16=True)
    rowmap = workloads.rng(19, 4).integers(0, pop, size=R).astype(np.int32)
    L = egr.Layer(n, m, R, 1, r, layer_id=3, seed=5, flags=egr.ACT_GELU, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.F32)
    Y = torch.zeros((R, m), dtype=torch.float32, device="cuda")
    egr.egr_perturbed_linear_rows(L, to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16), to_dev(rowmap), 0.3, Y, ws)
    _check_status(egr, ws)
    want = oracle.perturbed_linear(X, W, rowmap, 1, r, 3, 5, oracle.ACT_GELU, 0.3)
    assert rel_fro(Y.cpu().numpy(), want) < 1e-4
    Ls = egr.Layer(n, m, R, 1, r, layer_id=3, seed=5, flags=egr.ACT_TANH, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.F32)
    Y2 = torch.zeros((R, m), dtype=torch.float32, device="cuda")
    egr.egr_perturbed_linear_static(Ls, to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16), 0.3, Y2)
    assert egr.egr_static_status() == 0
    want2 = oracle.perturbed_linear(X, W, np.arange(R), 1, r, 3, 5, oracle.ACT_TANH, 0.3)
    assert rel_fro(Y2.cpu().numpy(), want2) < 1e-4


def test_activation_bits_are_rejected_by_the_integer_forward(egr, ws):
    import torch
    L = egr.Layer(64, 64, 8, 1, 1, flags=egr.ACT_RELU, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
    z = lambda *s: torch.zeros(s, dtype=torch.int8, device="cuda")
    with pytest.raises(egr.EgrError):
        egr.egr_perturbed_linear_i8(L, z(8, 64), z(64, 64), 8, 8, z(1 << 16), z(8, 64), ws)


@pytest.mark.parametrize("N,m,n,r,anti", [(20000, 520, 300, 1, False), (18000, 300, 776, 2, True)])
def test_update_bf16_several_chunks_ragged(egr, ws, N, m, n, r, anti):
    """Contractions of several K-chunks: row counts that are not multiples of the 256-row tile, different tile counts for the
    two factors, a short last chunk, master + shadow + dW together; the same call twice gives the same bits."""
    import torch
    W = workloads.linear_layer(10, m, n, 1, bf16=True)[0]
    f = workloads.raw_fitness(10, N)
    flags = egr.ANTITHETIC if anti else 0
    ldw = (n + 7) // 8 * 8
    L = egr.Layer(n, m, N, 1, r, layer_id=4, seed=321, flags=flags, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16,
                  ldw=ldw)
    Wm = padded(W, ldw)
    Wsh = torch.zeros((m, ldw), dtype=torch.bfloat16, device="cuda")
    dW = torch.zeros((m, n), dtype=torch.float32, device="cuda")
    egr.egr_es_update(L, Wm, to_dev(f), 0.7, ws, W_shadow=Wsh, dW_out=dW)
    _check_status(egr, ws)
    Wn, dWo = oracle.es_update(W, f, r, 4, 321, flags, 0.7)
    assert rel_fro(dW.cpu().numpy(), dWo) < TOL_BF16
    assert rel_fro(Wm.cpu().numpy()[:, :n] - W, dWo) < TOL_BF16
    assert torch.equal(Wsh[:, :n], Wm[:, :n].to(torch.bfloat16))
    # twice the same call gives the same bits (the chunks are added in a fixed order)
    Wm2 = padded(W, ldw)
    dW2 = torch.zeros_like(dW)
    egr.egr_es_update(L, Wm2, to_dev(f), 0.7, ws, dW_out=dW2)
    _check_status(egr, ws)
    assert torch.equal(dW2, dW) and torch.equal(Wm2, Wm)


@pytest.mark.parametrize("N,m,n,r,anti", [(26000, 2100, 4200, 1, False), (29000, 4200, 2100, 2, True), (2500, 2300, 4104, 16, False),
                                          (12000, 2100, 4200, 1, False), (17000, 4200, 2100, 2, True)])
def test_update_bf16_one_launch_ring_of_chunks(egr, ws, N, m, n, r, anti):
    """Long contractions over large matrices (ranks below 4, two tiles and more per CTA pair) run as one launch whose
    side warps stage the factors into a ring of three chunk buffers: more chunks than slots (slots are reused), bands
    that are not multiples of 256 rows, different band counts for the two factors, a short last chunk; contractions of
    two or three full chunks are cut into four shorter ones (the last two cases); the rank-16 case of the same size goes
    launch by launch and must agree all the same.  The form
    with dW_out (register epilogue) and the caller's form (reduce-add stores, shadow in a pass of its own) are both
    compared with the oracle on sampled blocks, and two calls give the same bits (the chunks of a tile are added in a
    fixed order)."""
    import torch
    W = workloads.linear_layer(10, m, n, 1, bf16=True)[0]
    f = workloads.raw_fitness(10, N)
    flags = egr.ANTITHETIC if anti else 0
    ldw = (n + 7) // 8 * 8
    L = egr.Layer(n, m, N, 1, r, layer_id=4, seed=321, flags=flags, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16,
                  ldw=ldw)
    fd = to_dev(f)
    Wm = padded(W, ldw)
    Wsh = torch.zeros((m, ldw), dtype=torch.bfloat16, device="cuda")
    dW = torch.zeros((m, n), dtype=torch.float32, device="cuda")
    egr.egr_es_update(L, Wm, fd, 0.7, ws, W_shadow=Wsh, dW_out=dW)
    _check_status(egr, ws)
    Wc = padded(W, ldw)
    Wc[:, n:] = 5.0
    Wsh_c = torch.full((m, ldw), 9.0, dtype=torch.bfloat16, device="cuda")
    egr.egr_es_update(L, Wc, fd, 0.7, ws, W_shadow=Wsh_c)
    _check_status(egr, ws)
    got_dw = dW.cpu().numpy()
    got_c = (Wc[:, :n] - to_dev(W)).cpu().numpy()
    g = workloads.rng(10, 5)
    blocks = [(0, 0), (m - 32, n - 32), (m - 32, 0), (0, n - 32)] + [(int(g.integers(0, m - 32)), int(g.integers(0, n - 32))) for _ in range(8)]
    for (j0, l0) in blocks:
        want = oracle.es_update_block(f, r, 4, 321, flags, 0.7, j0, j0 + 32, l0, l0 + 32)
        assert rel_fro(got_dw[j0:j0 + 32, l0:l0 + 32], want) < TOL_BF16, (j0, l0)
        assert rel_fro(got_c[j0:j0 + 32, l0:l0 + 32], want) < TOL_BF16, (j0, l0)
    assert rel_fro(Wm.cpu().numpy()[:, :n] - W, got_dw) < 1e-3
    assert torch.equal(Wsh[:, :n], Wm[:, :n].to(torch.bfloat16))
    assert torch.equal(Wsh_c[:, :n], Wc[:, :n].to(torch.bfloat16))
    assert torch.all(Wc[:, n:] == 5.0) and torch.all(Wsh_c[:, n:] == 9.0)
    Wc2 = padded(W, ldw)
    egr.egr_es_update(L, Wc2, fd, 0.7, ws)
    _check_status(egr, ws)
    assert torch.equal(Wc2[:, :n], Wc[:, :n])


@pytest.mark.parametrize("N,T,m,n,r,flags", [(40, 1, 1000, 264, 1, 0), (6, 32, 1500, 136, 1, 0), (10, 3, 32000, 128, 4, 1),
                                             (16, 2, 300, 520, 16, 0), (300, 1, 2048, 256, 2, 2)])
def test_vocabulary_head_ending_in_the_log_likelihood(egr, ws, N, T, m, n, r, flags):
    """egr_perturbed_linear_loglik: the perturbed head's logits never reach memory, only log p(target) per row does.
    Against the oracle's explicit forward followed by the plain definition; ragged vocabularies (a last tile that is
    almost empty), targets at both ends, unscored rows, shared noise inside a member, the unperturbed flag."""
    import torch
    W, X = workloads.linear_layer(45, m, n, N * T, bf16=True, w_std=0.05)
    g = workloads.rng(45, 6)
    targets = g.integers(0, m, size=N * T).astype(np.int32)
    targets[0], targets[1], targets[2], targets[3] = 0, m - 1, -1, m
    oflags = flags & 1
    sigma = 0.2
    L = egr.Layer(n, m, N, T, r, layer_id=1001, seed=8, flags=flags, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16)
    logp = torch.full((N * T,), 7.0, dtype=torch.float32, device="cuda")
    egr.egr_perturbed_linear_loglik(L, to_dev(X, torch.bfloat16), to_dev(W, torch.bfloat16), sigma, to_dev(targets), logp, ws)
    _check_status(egr, ws)
    if flags & 2:
        Z = X.astype(np.float64) @ W.astype(np.float64).T
    else:
        Z = oracle.perturbed_linear(X, W, np.arange(N), T, r, 1001, 8, oflags, sigma)
    want = oracle.token_log_likelihood(Z, targets)
    got = logp.cpu().numpy().astype(np.float64)
    assert got[2] == 0.0 and got[3] == 0.0
    assert np.abs(got - want).max() < 2e-4 * max(1.0, np.abs(want).max())
    # the perturbation matters at this sigma (a head that dropped it would not pass)
    if not flags & 2:
        base = oracle.token_log_likelihood(X.astype(np.float64) @ W.astype(np.float64).T, targets)
        assert np.abs(base - want).max() > 50 * np.abs(got - want).max()

"""Randomised parity (hypothesis): the CUDA path against the oracle on many small, ragged shapes drawn at random --
odd row and column counts, every rank, with and without antithetic pairs, with and without the element-wise function --
for the fp32 and bf16 forward, the update and the integer forward.  Same tolerances as the fixed cases."""
import numpy as np
import pytest
from hypothesis import HealthCheck, given, settings, strategies as st

import oracle
import workloads
from util import padded, rel_fro, to_dev

pytestmark = pytest.mark.gpu

SET = settings(max_examples=40, deadline=None, derandomize=True, database=None,
               suppress_health_check=[HealthCheck.function_scoped_fixture, HealthCheck.too_slow])
ACTS = [0, oracle.ACT_TANH, oracle.ACT_RELU, oracle.ACT_GELU]


@pytest.fixture(scope="module")
def egr():
    import torch
    assert torch.cuda.is_available()
    import paper_2511_16652_b200 as m
    m.load_library()
    return m


@SET
@given(st.integers(1, 9), st.integers(1, 3), st.integers(1, 70), st.integers(1, 70), st.sampled_from([1, 2, 4, 8, 16]),
       st.booleans(), st.sampled_from(ACTS), st.integers(0, 2 ** 31 - 1))
def test_forward_fp32_random_shapes(egr, N, T, m, n, r, anti, act, seed):
    import torch
    N += N & 1 if anti else 0
    g = np.random.default_rng(seed)
    W = (g.standard_normal((m, n)) / np.sqrt(n)).astype(np.float32)
    X = g.standard_normal((N * T, n)).astype(np.float32)
    ldx, ldw, ldy = (n + 3) // 4 * 4, (n + 3) // 4 * 4 + 4, (m + 3) // 4 * 4
    flags = (egr.ANTITHETIC if anti else 0) | act
    L = egr.Layer(n, m, N, T, r, layer_id=seed % 50, seed=seed, flags=flags, x_dtype=egr.F32, w_dtype=egr.F32, y_dtype=egr.F32,
                  ldx=ldx, ldw=ldw, ldy=ldy)
    Y = torch.full((N * T, ldy), -3.0, dtype=torch.float32, device="cuda")
    ws = egr.Workspace()
    egr.egr_perturbed_linear(L, padded(X, ldx), padded(W, ldw), 0.3, Y, ws)
    assert egr.egr_workspace_status(ws) == 0
    want = oracle.perturbed_linear(X, W, np.arange(N), T, r, seed % 50, seed, flags, 0.3)
    got = Y.cpu().numpy()
    assert rel_fro(got[:, :m], want) < 1e-5 or np.linalg.norm(want) < 1e-6
    assert np.all(got[:, m:] == -3.0)


@SET
@given(st.integers(1, 40), st.integers(1, 3), st.integers(1, 300), st.integers(1, 40), st.sampled_from([1, 2, 4, 8, 16]),
       st.booleans(), st.sampled_from(ACTS), st.booleans(), st.integers(0, 2 ** 31 - 1))
def test_forward_bf16_random_shapes(egr, N, T, m, n8, r, anti, act, y_f32, seed):
    import torch
    N += N & 1 if anti else 0
    n = n8 * 8 - int(seed % 8)                       # any d_in >= 1: the pitch is what must be a multiple of 8
    n = max(n, 1)
    g = np.random.default_rng(seed)
    W = workloads.round_to_bf16((g.standard_normal((m, n)) / np.sqrt(n)).astype(np.float32))
    X = workloads.round_to_bf16(g.standard_normal((N * T, n)).astype(np.float32))
    ld = (n + 7) // 8 * 8
    ldy = (m + 7) // 8 * 8
    flags = (egr.ANTITHETIC if anti else 0) | act
    L = egr.Layer(n, m, N, T, r, layer_id=7, seed=seed, flags=flags, x_dtype=egr.BF16, w_dtype=egr.BF16,
                  y_dtype=egr.F32 if y_f32 else egr.BF16, ldx=ld, ldw=ld, ldy=ldy)
    Y = torch.full((N * T, ldy), 2.0, dtype=torch.float32 if y_f32 else torch.bfloat16, device="cuda")
    ws = egr.Workspace()
    egr.egr_perturbed_linear(L, padded(X, ld, torch.bfloat16), padded(W, ld, torch.bfloat16), 0.2, Y, ws)
    assert egr.egr_workspace_status(ws) == 0
    want = oracle.perturbed_linear(X, W, np.arange(N), T, r, 7, seed, flags, 0.2)
    got = Y.float().cpu().numpy()
    assert rel_fro(got[:, :m], want) < (1e-4 if y_f32 else 1e-2) or np.linalg.norm(want) < 1e-3
    assert np.all(got[:, m:] == 2.0)


@SET
@given(st.integers(1, 60), st.integers(1, 90), st.integers(1, 12), st.sampled_from([1, 2, 4, 8, 16]), st.booleans(),
       st.booleans(), st.integers(0, 2 ** 31 - 1))
def test_update_random_shapes(egr, N, m, n8, r, anti, bf16, seed):
    import torch
    N += N & 1 if anti else 0
    n = n8 * 8
    g = np.random.default_rng(seed)
    W = (g.standard_normal((m, n)) / np.sqrt(n)).astype(np.float32)
    if bf16:
        W = workloads.round_to_bf16(W)
    f = g.standard_normal(N).astype(np.float32)
    flags = egr.ANTITHETIC if anti else 0
    code = egr.BF16 if bf16 else egr.F32
    L = egr.Layer(n, m, N, 1, r, layer_id=3, seed=seed, flags=flags, x_dtype=code, w_dtype=code, y_dtype=code)
    Wm = to_dev(W)
    dW = torch.zeros((m, n), dtype=torch.float32, device="cuda")
    ws = egr.Workspace()
    egr.egr_es_update(L, Wm, to_dev(f), 0.5, ws, dW_out=dW)
    assert egr.egr_workspace_status(ws) == 0
    Wn, dWo = oracle.es_update(W, f, r, 3, seed, flags, 0.5)
    tol = 1e-2 if bf16 else 1e-5
    assert rel_fro(dW.cpu().numpy(), dWo) < tol or np.linalg.norm(dWo) < 1e-6
    assert rel_fro(Wm.cpu().numpy() - W, dWo) < max(tol, 1e-4) or np.linalg.norm(dWo) < 1e-4


@SET
@given(st.integers(1, 40), st.integers(1, 3), st.integers(1, 300), st.integers(1, 20), st.booleans(), st.integers(0, 12),
       st.integers(0, 12), st.sampled_from([8, 10, 16]), st.integers(0, 2 ** 31 - 1))
def test_forward_int8_random_shapes_bit_exact(egr, N, T, m, n16, anti, sshift, oshift, table_log2, seed):
    import torch
    N += N & 1 if anti else 0
    n = n16 * 16
    X = workloads.int8_activations(seed % 1000, 30, (N * T, n))
    W = workloads.int8_matrix(seed % 1000, 31, (m, n))
    table = workloads.noise_table(seed % 1000, table_log2)
    flags = egr.ANTITHETIC if anti else 0
    L = egr.Layer(n, m, N, T, 1, layer_id=9, seed=seed, flags=flags, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
    Y = torch.zeros((N * T, m), dtype=torch.int8, device="cuda")
    ws = egr.Workspace()
    egr.egr_perturbed_linear_i8(L, to_dev(X), to_dev(W), sshift, oshift, to_dev(table), Y, ws)
    want = oracle.perturbed_linear_i8(X, W, np.arange(N), T, 9, seed, flags, sshift, oshift, table)
    assert np.array_equal(Y.cpu().numpy(), want)


@settings(max_examples=8, deadline=None, derandomize=True, database=None,
          suppress_health_check=[HealthCheck.function_scoped_fixture, HealthCheck.too_slow])
@given(st.integers(1, 400), st.integers(1, 3), st.integers(2, 6), st.sampled_from(["identity", "hard"]), st.integers(4, 10),
       st.integers(0, 1000))
def test_integer_lm_random_models_bit_exact(egr, pairs, layers, seq_len, lut, sigma_shift, seed):
    """The width-256 model through the one-launch kernel: any even population (row tiles that are partly empty), one to
    three layers, short sequences, both table shapes; fitness and carried state bit for bit."""
    import torch
    N, D = 2 * pairs, 256
    P = workloads.egg_lm_params(seed, D, layers, lut=lut)
    tokens = workloads.markov_bytes(seed, 4, seq_len)
    table = workloads.noise_table(seed, 16)
    member_seq = (np.arange(N) // 2) % 4
    Pd = {k: torch.from_numpy(np.ascontiguousarray(v)).cuda() for k, v in P.items()}
    state = torch.zeros((layers, N, D), dtype=torch.int8, device="cuda")
    fit = torch.zeros(N, dtype=torch.int32, device="cuda")
    egr.egr_i8lm_forward(Pd, N, seed, egr.ANTITHETIC, sigma_shift, torch.from_numpy(table).cuda(), torch.from_numpy(tokens).cuda(),
                         torch.from_numpy(member_seq.astype(np.int32)).cuda(), state, fit, egr.Workspace())
    want_fit, want_st = oracle.i8lm_forward(P, tokens, np.arange(N), member_seq, seed, oracle.ANTITHETIC, sigma_shift, table)
    assert np.array_equal(fit.cpu().numpy(), want_fit)
    assert np.array_equal(state.cpu().numpy().transpose(1, 0, 2), want_st)


@settings(max_examples=20, deadline=None, derandomize=True, database=None,
          suppress_health_check=[HealthCheck.function_scoped_fixture, HealthCheck.too_slow])
@given(st.integers(1, 20), st.integers(1, 3), st.integers(1, 140), st.integers(1, 20), st.sampled_from([1, 2, 4, 8, 16]),
       st.booleans(), st.sampled_from([0.0, 1e-3]), st.booleans(), st.integers(0, 2 ** 31 - 1))
def test_forward_q8_random_shapes(egr, N, T, m, n8, r, anti, sigma_s, y_f32, seed):
    """Per-channel-scaled int8 matrix: codes, channel scales, input scale, low-rank term and (optionally) scale noise."""
    import torch
    from oracle import q8
    N += N & 1 if anti else 0
    n = n8 * 8
    g = np.random.default_rng(seed)
    Qo = g.integers(-127, 128, size=(m, n)).astype(np.int8)
    so = q8.bf16_round((0.01 + 0.01 * g.random(m)).astype(np.float32))
    X = workloads.round_to_bf16(g.standard_normal((N * T, n)).astype(np.float32))
    pitch, ldy = (n + 15) // 16 * 16, (m + 7) // 8 * 8
    Q = torch.zeros((m, pitch), dtype=torch.int8, device="cuda")
    Q[:, :n] = torch.from_numpy(Qo).cuda()
    flags = egr.ANTITHETIC if anti else 0
    Y = torch.zeros((N * T, ldy), dtype=torch.float32 if y_f32 else torch.bfloat16, device="cuda")
    L = egr.Layer(n, m, N, T, r, layer_id=2, seed=seed, flags=flags, x_dtype=egr.BF16, w_dtype=egr.I8,
                  y_dtype=egr.F32 if y_f32 else egr.BF16, ldw=pitch, ldy=ldy)
    ws = egr.Workspace()
    egr.egr_perturbed_linear_q8(L, to_dev(X, torch.bfloat16), Q, to_dev(so, torch.bfloat16), 0.5, 8.0, sigma_s, Y, ws)
    assert egr.egr_workspace_status(ws) == 0
    want = q8.perturbed_linear_q8(X.astype(np.float64), Qo, so, 0.5, np.arange(N), T, r, 2, seed, flags, 8.0, sigma_s)
    assert rel_fro(Y.float().cpu().numpy()[:, :m], want) < (2e-3 if y_f32 else 1e-2)

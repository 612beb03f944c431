"""GPU parity of the integer recurrent LM (config 3 of the benchmark set): bit-exact against the oracle."""
import math

import numpy as np
import pytest

import oracle
import workloads

pytestmark = pytest.mark.gpu


def _dev(params):
    import torch
    return {k: torch.from_numpy(np.ascontiguousarray(v)).cuda() for k, v in params.items()}


def _run_gpu(P, N, seed, flags, sigma_shift, table, tokens, member_seq, state0=None):
    import torch
    import paper_2511_16652_b200 as egr
    egr.load_library()
    Pd = _dev(P)
    l, D = P["ln1"].shape
    state = torch.zeros((l, N, D), dtype=torch.int8, device="cuda") if state0 is None else state0
    fit = torch.zeros(N, dtype=torch.int32, device="cuda")
    ws = egr.Workspace()
    egr.egr_i8lm_forward(Pd, N, seed, flags, sigma_shift, torch.from_numpy(table).cuda(),
                         torch.from_numpy(tokens).cuda(), torch.from_numpy(member_seq.astype(np.int32)).cuda(),
                         state, fit, ws)
    torch.cuda.synchronize()
    return fit.cpu().numpy(), state.cpu().numpy()


# width 256: up to eight layers run as one launch for the whole sequence, more layers launch phase by phase; 600 members
# are three row tiles, the last one ragged
@pytest.mark.parametrize("D,l,N,seq_len,lut", [(16, 2, 8, 24, "hard"), (64, 1, 32, 10, "identity"), (256, 4, 64, 8, "identity"),
                                               (256, 2, 600, 5, "hard"), (256, 9, 40, 4, "identity")])
def test_lm_forward_bit_exact(D, l, N, seq_len, lut):
    P = workloads.egg_lm_params(7, D, l, lut=lut)
    P["bf"] = (workloads.int8_matrix(7, 90, (l, D)) // 4).astype(np.int8)
    P["bh"] = (workloads.int8_matrix(7, 91, (l, D)) // 4).astype(np.int8)
    tokens = workloads.markov_bytes(7, 4, seq_len)
    table = workloads.noise_table(7, 16)
    member_seq = (np.arange(N) // 2) % 4
    fit, st = _run_gpu(P, N, 21, 1, 8, table, tokens, member_seq)
    want_fit, want_st = oracle.i8lm_forward(P, tokens, np.arange(N), member_seq, 21, oracle.ANTITHETIC, 8, table)
    assert np.array_equal(fit, want_fit)
    assert np.array_equal(st.transpose(1, 0, 2), want_st)
    assert st.min() >= -127


def test_config3_shape_sampled_members_and_update():
    """Config 3: D=256, 4 layers, N=16384 antithetic members, 16 Markov byte sequences of 128 tokens, sigma_hat=4.
    The oracle evaluates 12 sampled members (both members of each sampled pair); then pair-sign shaping and the
    integer update of one matrix with the threshold for alpha = 0.5."""
    import torch
    import paper_2511_16652_b200 as egr
    D, l, N, n_seq, seq_len = 256, 4, 16384, 16, 128
    P = workloads.egg_lm_params(0, D, l)
    tokens = workloads.markov_bytes(0, n_seq, seq_len)
    table = workloads.noise_table(0, 24)
    member_seq = (np.arange(N) // 2) % n_seq
    fit, st = _run_gpu(P, N, 0, 1, 8, table, tokens, member_seq)
    sel = np.array([0, 1, 2, 3, 4094, 4095, 9000, 9001, 16382, 16383, 777 * 2, 777 * 2 + 1])
    want_fit, want_st = oracle.i8lm_forward(P, tokens, sel, member_seq[sel], 0, oracle.ANTITHETIC, 8, table)
    assert np.array_equal(fit[sel], want_fit)
    assert np.array_equal(st.transpose(1, 0, 2)[sel], want_st)
    # shaping + update of layer 0's Wf with thr = I32(16 * 0.6745) * I32(16 sqrt(8192)) = 10 * 1448
    F = torch.zeros(N // 2, dtype=torch.int8, device="cuda")
    egr.egr_fitness_shape_i8(torch.from_numpy(fit).cuda(), F)
    assert np.array_equal(F.cpu().numpy(), oracle.fitness_shape_i8(fit))
    thr = int(16 * 0.6745) * int(16 * math.sqrt(N // 2))
    assert thr == 14480
    L = egr.Layer(D, D, N, 1, 1, layer_id=0, seed=0, flags=egr.ANTITHETIC, x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
    W = torch.from_numpy(P["Wf"][0].copy()).cuda()
    egr.egr_es_update_i8(L, W, F, thr, torch.from_numpy(table).cuda(), egr.Workspace())
    Wn, _ = oracle.es_update_i8(P["Wf"][0], F.cpu().numpy(), 0, 0, thr, table)
    assert np.array_equal(W.cpu().numpy(), Wn)
    assert 0.2 < np.mean(Wn != P["Wf"][0]) < 0.8


def test_lm_more_row_tiles_than_cta_pairs_sampled_members():
    """40000 members are 157 row tiles of 256 (the last one ragged) for the 74 CTA pairs of the one-launch kernel: every
    pair walks the whole sequence for two or three tiles in turn.  Members at the seams are checked against the oracle."""
    D, l, N, n_seq, seq_len = 256, 2, 40000, 8, 6
    P = workloads.egg_lm_params(3, D, l, lut="hard")
    tokens = workloads.markov_bytes(3, n_seq, seq_len)
    table = workloads.noise_table(3, 20)
    member_seq = (np.arange(N) // 2) % n_seq
    fit, st = _run_gpu(P, N, 5, 1, 8, table, tokens, member_seq)
    sel = np.array([0, 1, 254, 255, 256, 257, 74 * 256 - 2, 74 * 256 - 1, 74 * 256, 74 * 256 + 1, 148 * 256 - 1, 148 * 256,
                    39998, 39999])
    want_fit, want_st = oracle.i8lm_forward(P, tokens, sel, member_seq[sel], 5, oracle.ANTITHETIC, 8, table)
    assert np.array_equal(fit[sel], want_fit)
    assert np.array_equal(st.transpose(1, 0, 2)[sel], want_st)


# Layer ids of the perturbed matrices, written out here and not taken from the product: 16 layer + slot for the
# four GRU matrices and the two MLP matrices, 1000 for the embedding, 1001 for the head.
_SLOT_OF = {"Wf": 0, "Uf": 1, "Wh": 2, "Uh": 3, "mlp1": 4, "mlp2": 5}


def _threshold(alpha, n_noise):
    """I32(16 Phi^-1(1 - alpha/2)) I32(16 sqrt K) of the integer appendix's "Parameter Update", truncating casts, with
    scipy's quantile function (the product uses the standard library's)."""
    from scipy.stats import norm
    if alpha <= 0.0:
        return 2 ** 31 - 1
    zi = int(16.0 * float(norm.ppf(1.0 - alpha / 2.0)))
    return min(2 ** 31 - 1, zi * int(16.0 * math.sqrt(n_noise)))


def _oracle_egg_step(P, N, seed, sigma_shift, table, tokens, member_seq, state, alpha):
    fit, st = oracle.i8lm_forward(P, tokens, np.arange(N), member_seq, seed, oracle.ANTITHETIC, sigma_shift, table, state=state)
    F = oracle.fitness_shape_i8(fit)
    thr = _threshold(alpha, N // 2)
    newP = dict(P)
    l = P["ln1"].shape[0]
    for name, slot in _SLOT_OF.items():
        newP[name] = np.stack([oracle.es_update_i8(P[name][i], F, 16 * i + slot, seed, thr, table)[0] for i in range(l)])
    newP["emb_t"] = oracle.es_update_i8(P["emb_t"], F, 1000, seed, thr, table)[0]
    newP["head"] = oracle.es_update_i8(P["head"], F, 1001, seed, thr, table)[0]
    return newP, fit, st, F, thr


@pytest.mark.parametrize("D,l,N", [(16, 2, 32), (256, 1, 64)])
def test_egg_training_steps_bit_exact(D, l, N):
    """Three truncated-ES steps with carried state and the alpha schedule: every matrix, the embedding and the head
    stay bit-identical to the oracle's."""
    import torch
    import paper_2511_16652_b200 as egr
    from paper_2511_16652_b200 import egg
    P = workloads.egg_lm_params(11, D, l, lut="hard")
    tokens_all = workloads.markov_bytes(11, 4, 3 * 6 + 1)
    table = workloads.noise_table(11, 16)
    member_seq = ((np.arange(N) // 2) % 4).astype(np.int32)
    Pd = _dev(P)
    state_d = torch.zeros((l, N, D), dtype=torch.int8, device="cuda")
    state_o = np.zeros((N, l, D), dtype=np.int8)
    ws = egr.Workspace()
    changed = 0
    for step in range(3):
        chunk = np.ascontiguousarray(tokens_all[:, step * 6: step * 6 + 7])          # 6 scored positions, overlapping by one byte
        alpha = 1.0 / (0.015 * (step * 40) + 1.0)            # the appendix's schedule, restated
        assert alpha == egg.alpha_schedule(step * 40)
        fit_d, F_d, thr_d = egg.egg_step(Pd, N, 100 + step, 6, torch.from_numpy(table).cuda(), torch.from_numpy(chunk).cuda(),
                                         torch.from_numpy(member_seq).cuda(), state_d, alpha, ws)
        P_new, fit_o, state_o, F_o, thr_o = _oracle_egg_step(P, N, 100 + step, 6, table, chunk, member_seq, state_o, alpha)
        assert thr_d == thr_o
        assert np.array_equal(fit_d.cpu().numpy(), fit_o)
        assert np.array_equal(F_d.cpu().numpy(), F_o)
        assert np.array_equal(state_d.cpu().numpy().transpose(1, 0, 2), state_o)
        for k in list(_SLOT_OF) + ["emb_t", "head"]:
            assert np.array_equal(Pd[k].cpu().numpy(), P_new[k]), k
            changed += int((P_new[k] != P[k]).sum())
        P = P_new
    assert changed > 0


def test_lm_forward_replayed_as_a_cuda_graph_is_bit_exact():
    """The fused LM pass only enqueues work on the caller's stream (memsets, kernel launches), so after one warm-up
    call it can be captured into a CUDA graph; the replay must give the oracle's fitness and state."""
    import torch
    import paper_2511_16652_b200 as egr
    egr.load_library()
    D, l, N, seq_len = 256, 2, 512, 12
    P = workloads.egg_lm_params(9, D, l)
    tokens = workloads.markov_bytes(9, 4, seq_len)
    table = workloads.noise_table(9, 16)
    member_seq = (np.arange(N) // 2) % 4
    Pd = _dev(P)
    td, kd = torch.from_numpy(table).cuda(), torch.from_numpy(tokens).cuda()
    md = torch.from_numpy(member_seq.astype(np.int32)).cuda()
    state = torch.zeros((l, N, D), dtype=torch.int8, device="cuda")
    fit = torch.zeros(N, dtype=torch.int32, device="cuda")
    ws = egr.Workspace()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        egr.egr_i8lm_forward(Pd, N, 33, 1, 8, td, kd, md, state, fit, ws)        # warm-up: attributes, workspace size
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            egr.egr_i8lm_forward(Pd, N, 33, 1, 8, td, kd, md, state, fit, ws)
    torch.cuda.synchronize()
    state.zero_()
    fit.zero_()
    graph.replay()
    torch.cuda.synchronize()
    want_fit, want_st = oracle.i8lm_forward(P, tokens, np.arange(N), member_seq, 33, oracle.ANTITHETIC, 8, table)
    assert np.array_equal(fit.cpu().numpy(), want_fit)
    assert np.array_equal(state.cpu().numpy().transpose(1, 0, 2), want_st)

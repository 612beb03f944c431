"""Pins for the oracle's integer recurrent LM (CPU only)."""
import math
import os

import numpy as np

import oracle
import workloads

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_parameter_count_matches_the_paper():
    for line in open(os.path.join(GOLD, "egg_param_count.txt")):
        if line.startswith("#") or not line.strip():
            continue
        l, D, want = [int(t) for t in line.split()]
        assert workloads.egg_lm_param_count(workloads.egg_lm_params(0, D, l)) == want
        assert want == 513 * D + l * (4 * D + 12 * D * D)


def test_exp2_and_log2_tables_follow_the_printed_formulas():
    e = oracle.exp2_table()
    for i in range(256):
        assert abs(e[i] - 16 * 2 ** (i / 16)) <= 0.5
    assert e[255] < 2 ** 20                                # "at most 20 bits"
    g = workloads.rng(0, 60)
    for S in list(range(1, 600)) + [int(x) for x in g.integers(1, 2 ** 28, size=2000)]:
        assert abs(oracle.log2_int(S) - 16 * math.log2(S / 16)) <= 0.6     # 0.1 from the 8-bit mantissa + rounding
    assert oracle.log2_int(16) == 0 and oracle.log2_int(32) == 16 and oracle.log2_int(1 << 27) == 16 * 23


def _numpy_forward(P, tokens, D, l):
    """Unperturbed model restated with numpy int64 (zero noise table): scaled matmuls are floor shifts."""
    def sat(v):
        return np.clip(v, -127, 127)

    def mm(u, theta):
        n = theta.shape[1]
        shift = 4 + int(round(math.log(n, 4)))
        return sat((theta.astype(np.int64) @ u.astype(np.int64)) >> shift)

    def ln(w, u):
        mav = max(1, int(min(127, int(np.abs(u.astype(np.int64)).sum()) >> (2 * int(round(math.log(D, 4)))))))
        prod = u.astype(np.int64) * w.astype(np.int64)
        return sat(np.sign(prod) * (np.abs(prod) // mav))

    E = oracle.exp2_table().astype(np.int64)
    s = np.zeros((l, D), dtype=np.int64)
    fit = 0
    for pos in range(len(tokens) - 1):
        y = P["emb_t"][:, tokens[pos]].astype(np.int64)
        for i in range(l):
            x = ln(P["ln1"][i], y)
            f = P["lut_sigma"][sat(mm(x, P["Wf"][i]) + mm(s[i], P["Uf"][i]) + P["bf"][i]) + 128].astype(np.int64)
            fh = sat(((f + 127) * s[i]) >> 8)
            hh = P["lut_phi"][sat(mm(x, P["Wh"][i]) + mm(fh, P["Uh"][i]) + P["bh"][i]) + 128].astype(np.int64)
            h = sat(s[i] + sat(((f + 127) * (hh - s[i])) >> 8))
            s[i] = h
            y = sat(h + y)
            x = ln(P["ln2"][i], y)
            y = sat(mm(mm(x, P["mlp1"][i]), P["mlp2"][i]) + y)
        logits = mm(ln(P["ln_out"], y), P["head"])
        z = logits + 128
        fit += int(z[tokens[pos + 1]]) - oracle.log2_int(int(E[z].sum()))
    return fit, s


def test_zero_noise_table_gives_the_unperturbed_model_and_partners_agree():
    D, l = 16, 2
    P = workloads.egg_lm_params(3, D, l, lut="hard")
    P["bf"] = workloads.int8_matrix(3, 90, (l, D)) // 4
    P["ln1"] = (16 + workloads.int8_matrix(3, 91, (l, D)) // 8).astype(np.int8)
    tokens = workloads.markov_bytes(3, 2, 24)
    table0 = np.zeros(1 << 10, np.int8)
    fit, st = oracle.i8lm_forward(P, tokens, [0, 1, 2, 3], [0, 0, 1, 1], 7, oracle.ANTITHETIC, 8, table0)
    assert fit[0] == fit[1] and fit[2] == fit[3]
    for k, seq in ((0, 0), (2, 1)):
        want_fit, want_state = _numpy_forward(P, tokens[seq], D, l)
        assert fit[k] == want_fit
        assert np.array_equal(st[k], want_state)
    assert st.min() >= -127


def test_perturbed_members_differ_and_state_carries_over():
    D, l = 16, 2
    P = workloads.egg_lm_params(4, D, l)
    tokens = workloads.markov_bytes(4, 1, 40)
    table = workloads.noise_table(4, 12)
    fit, st = oracle.i8lm_forward(P, tokens, np.arange(8), np.zeros(8, int), 11, oracle.ANTITHETIC, 6, table)
    assert len(set(fit.tolist())) > 4
    # two half sequences with carried state give the same total as the full sequence, except that the
    # transition between the halves is scored once more in neither: compare position by position instead
    fit_a, st_a = oracle.i8lm_forward(P, tokens[:, :21], np.arange(8), np.zeros(8, int), 11, oracle.ANTITHETIC, 6, table)
    fit_b, st_b = oracle.i8lm_forward(P, tokens[:, 20:], np.arange(8), np.zeros(8, int), 11, oracle.ANTITHETIC, 6, table,
                                      state=st_a)
    assert np.array_equal(fit_a + fit_b, fit)
    assert np.array_equal(st_b, st)


def test_embedding_perturbation_is_rank_one_slice_product():
    # A table that is non-zero only inside the embedding's two slices leaves every matmul unperturbed, so the model
    # must equal the unperturbed one run on embeddings emb[:,t] + ((sign B[t] A[j]) >> shift), saturated.
    D, l, L, shift, seed = 16, 1, 14, 5, 3
    P = workloads.egg_lm_params(5, D, l)
    tokens = workloads.markov_bytes(5, 1, 12)
    mask = (1 << L) - 1
    full = workloads.noise_table(5, L)
    for p in range(4):
        offa, offb = oracle.i8_offsets(seed, 1000, p, L)
        keep = np.zeros(1 << L, bool)
        keep[(offa + np.arange(D)) & mask] = True
        keep[(offb + np.arange(256)) & mask] = True
        clash = False
        for layer_id in [0, 1, 2, 3, 4, 5, 1001]:
            oa, ob = oracle.i8_offsets(seed, layer_id, p, L)
            idx = np.concatenate([(oa + np.arange(4 * D + 256)) & mask, (ob + np.arange(4 * D + 256)) & mask])
            clash |= bool(keep[idx].any())
        if clash:
            continue
        table = np.where(keep, full, 0).astype(np.int8)
        A = table[(offa + np.arange(D)) & mask].astype(np.int64)
        B = table[(offb + np.arange(256)) & mask].astype(np.int64)
        for member, sign in ((2 * p, 1), (2 * p + 1, -1)):
            fit, st = oracle.i8lm_forward(P, tokens, [member], [0], seed, oracle.ANTITHETIC, shift, table)
            P2 = dict(P)
            emb = P["emb_t"].astype(np.int64) + ((sign * B[None, :] * A[:, None]) >> shift)
            P2["emb_t"] = np.clip(emb, -127, 127).astype(np.int8)
            want_fit, want_state = _numpy_forward(P2, tokens[0], D, l)
            assert fit[0] == want_fit and np.array_equal(st[0], want_state)
            assert not np.array_equal(P2["emb_t"], P["emb_t"])
        return
    raise AssertionError("no clash-free noise index found")


def _stepwise_forward(P, tokens, D, l, member, seed, flags, sigma_shift, table):
    """The perturbed model rebuilt position by position: every matrix product is one call of the separately pinned
    integer perturbed matmul with the matrix's own id (hard-coded here: 16 layer + {Wf 0, Uf 1, Wh 2, Uh 3, mlp1 4,
    mlp2 5}, head 1001, embedding 1000) and out_shift = 4 + log4(fan_in); everything else is numpy int64."""
    def sat(v):
        return np.clip(v, -127, 127)

    def pm(u, theta, layer_id):
        n = theta.shape[1]
        out_shift = 4 + int(round(math.log(n, 4)))
        y = oracle.perturbed_linear_i8(u.astype(np.int8)[None, :], theta, [member], 1, layer_id, seed, flags, sigma_shift,
                                       out_shift, table)
        return y[0].astype(np.int64)

    def ln(w, u):
        mav = max(1, int(min(127, int(np.abs(u.astype(np.int64)).sum()) >> (2 * int(round(math.log(D, 4)))))))
        prod = u.astype(np.int64) * w.astype(np.int64)
        return sat(np.sign(prod) * (np.abs(prod) // mav))

    Lg = int(np.log2(len(table)))
    mask = (1 << Lg) - 1
    p, sign = (member >> 1, 1 - 2 * (member & 1)) if flags & oracle.ANTITHETIC else (member, 1)
    offa, offb = oracle.i8_offsets(seed, 1000, p, Lg)
    A = table[(offa + np.arange(D)) & mask].astype(np.int64)
    B = table[(offb + np.arange(256)) & mask].astype(np.int64)
    E = oracle.exp2_table().astype(np.int64)
    s = np.zeros((l, D), dtype=np.int64)
    fit = 0
    for pos in range(len(tokens) - 1):
        t = int(tokens[pos])
        y = sat(P["emb_t"][:, t].astype(np.int64) + ((sign * B[t] * A) >> sigma_shift))
        for i in range(l):
            x = ln(P["ln1"][i], y)
            f = P["lut_sigma"][sat(pm(x, P["Wf"][i], 16 * i + 0) + pm(s[i], P["Uf"][i], 16 * i + 1) + P["bf"][i]) + 128].astype(np.int64)
            fh = sat(((f + 127) * s[i]) >> 8)
            hh = P["lut_phi"][sat(pm(x, P["Wh"][i], 16 * i + 2) + pm(fh, P["Uh"][i], 16 * i + 3) + P["bh"][i]) + 128].astype(np.int64)
            h = sat(s[i] + sat(((f + 127) * (hh - s[i])) >> 8))
            s[i] = h
            y = sat(h + y)
            x = ln(P["ln2"][i], y)
            y = sat(pm(pm(x, P["mlp1"][i], 16 * i + 4), P["mlp2"][i], 16 * i + 5) + y)
        logits = pm(ln(P["ln_out"], y), P["head"], 1001)
        z = logits + 128
        fit += int(z[tokens[pos + 1]]) - oracle.log2_int(int(E[z].sum()))
    return fit, s


def test_every_matrix_product_of_the_model_is_the_pinned_perturbed_matmul_with_its_own_id():
    # The model's inner perturbed product restates the formula of "Adding EGGROLL Perturbations"; this rebuilds a whole
    # forward from single calls of the stand-alone integer perturbed matmul (pinned in test_oracle_int8.py against a
    # big-integer restatement), so a wrong slice, sign, shift or matrix id inside the model changes fitness or state.
    D, l = 16, 2
    P = workloads.egg_lm_params(6, D, l, lut="hard")
    P["bf"] = workloads.int8_matrix(6, 90, (l, D)) // 4
    P["bh"] = workloads.int8_matrix(6, 92, (l, D)) // 4
    tokens = workloads.markov_bytes(6, 2, 14)
    table = workloads.noise_table(6, 13)
    for flags, members in ((oracle.ANTITHETIC, [0, 1, 6, 7]), (0, [0, 3])):
        seqs = [k % 2 for k in range(len(members))]
        fit, st = oracle.i8lm_forward(P, tokens, members, seqs, 21, flags, 4, table)
        assert len(set(fit.tolist())) == len(members)                 # the perturbations matter at this shift
        for k, member in enumerate(members):
            want_fit, want_state = _stepwise_forward(P, tokens[seqs[k]], D, l, member, 21, flags, 4, table)
            assert fit[k] == want_fit
            assert np.array_equal(st[k], want_state)


def test_matrix_ids_are_not_interchangeable():
    # the check above would be blind to a swap of two ids if both gave the same slices: they do not
    offs = {lid: oracle.i8_offsets(21, lid, 0, 13) for lid in [0, 1, 2, 3, 4, 5, 16, 17, 18, 19, 20, 21, 1000, 1001]}
    assert len(set(offs.values())) == len(offs)

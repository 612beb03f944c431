"""Pins for the oracle's fitness shaping (CPU only)."""
import numpy as np
from scipy import stats

import oracle
import workloads


def test_centred_rank_matches_the_printed_formula_with_a_library_ranking():
    # F_i = 1/2 - rank_i/(M-1), rank 0 = best (HFT appendix); scipy ranks ascending from 1.
    raw = workloads.raw_fitness(3, 257).astype(np.float64)
    got = oracle.fitness_shape(raw, oracle.SHAPE_CENTERED_RANK)
    desc_rank = len(raw) - stats.rankdata(raw, method="ordinal")          # 0 = best
    want = 0.5 - desc_rank / (len(raw) - 1)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-7)
    assert got.max() == 0.5 and got.min() == -0.5
    assert abs(got.sum()) < 1e-4
    assert got[np.argmax(raw)] == 0.5 and got[np.argmin(raw)] == -0.5


def test_centred_rank_brute_force_with_ties_and_nan():
    raw = np.array([1.0, 3.0, 1.0, np.nan, -2.0, 3.0, 0.0])
    got = oracle.fitness_shape(raw, oracle.SHAPE_CENTERED_RANK)
    # ascending order with ties by index and NaN worst: nan(3), -2(4), 0(6), 1(0), 1(2), 3(1), 3(5)
    order = [3, 4, 6, 0, 2, 1, 5]
    want = np.zeros(7)
    for asc, i in enumerate(order):
        want[i] = np.float32((2 * asc - 6) / 12.0)
    assert np.array_equal(got, want)


def test_centred_rank_values_are_fp32_of_one_division():
    raw = workloads.raw_fitness(9, 1000).astype(np.float64)
    got = oracle.fitness_shape(raw, oracle.SHAPE_CENTERED_RANK)
    asc = stats.rankdata(raw, method="ordinal") - 1
    want = (np.float32(2 * asc - 999) / np.float32(2 * 999)).astype(np.float64)   # IEEE fp32 division
    assert np.array_equal(got, want)


def test_zscore_against_library():
    raw = workloads.raw_fitness(4, 500).astype(np.float64) * 3 + 2
    got = oracle.fitness_shape(raw, oracle.SHAPE_ZSCORE)
    np.testing.assert_allclose(got, stats.zscore(raw), rtol=1e-6)
    assert abs(got.mean()) < 1e-12 and abs(got.std() - 1) < 1e-6
    assert np.all(oracle.fitness_shape(np.full(8, 2.0), oracle.SHAPE_ZSCORE) == 0.0)


def test_antithetic_sign_range_and_symmetry():
    raw = np.array([1.0, 0.5, 2.0, 2.0, -1.0, 3.0])
    got = oracle.fitness_shape(raw, oracle.SHAPE_ANTITHETIC_SIGN)
    assert list(got) == [1, -1, 0, 0, -1, 1]
    raw_i = np.array([10, 3, 5, 5, -7, 9, -2**31 + 1, 2**31 - 1], dtype=np.int32)
    assert list(oracle.fitness_shape_i8(raw_i)) == [1, 0, -1, -1]


def test_identity_mode():
    raw = workloads.raw_fitness(1, 10)
    assert np.array_equal(oracle.fitness_shape(raw, oracle.SHAPE_NONE), raw.astype(np.float64))


def test_per_question_scores_against_numpy():
    g = workloads.rng(5, 9)
    S = g.standard_normal((37, 11)) * np.linspace(0.5, 3, 11) + np.arange(11)
    got = oracle.fitness_shape_questions(S)
    c = S - S.mean(axis=0, keepdims=True)
    want = (c / (np.sqrt((c ** 2).mean()) + 1e-8)).mean(axis=1)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-14)
    assert abs(got.sum()) < 1e-9                                  # every question is centred over the members
    # one question: reduces to the plain z-score
    one = oracle.fitness_shape_questions(S[:, :1])
    np.testing.assert_allclose(one, oracle.fitness_shape(S[:, 0], oracle.SHAPE_ZSCORE), rtol=1e-9)
    # adding a per-question constant changes nothing
    np.testing.assert_allclose(oracle.fitness_shape_questions(S + 100 * np.arange(11)), got, rtol=1e-9, atol=1e-12)


def test_base3_packing_formula_round_trip_and_payload():
    """"Base-3 Fitness Packing": +1, 0, -1 -> 0, 1, 2 and byte = sum v_i 3^i; 1.6 bit per value."""
    # worked by hand from the formula: digits (0, 1, 2, 0, 1) -> 0 + 3 + 18 + 0 + 81 = 102
    assert oracle.pack3([1, 0, -1, 1, 0]).tolist() == [102]
    assert oracle.pack3([1, 1, 1, 1, 1]).tolist() == [0]
    assert oracle.pack3([-1] * 5).tolist() == [242]                    # the largest byte: 2 (1+3+9+27+81)
    assert oracle.pack3([-1]).tolist() == [2 + 3 + 9 + 27 + 81]        # the tail packs as zeros (digit 1)
    g = workloads.rng(41, 0)
    for count in (0, 1, 4, 5, 6, 1003):
        F = g.integers(-1, 2, size=count).astype(np.int8)
        packed = oracle.pack3(F)
        assert len(packed) == (count + 4) // 5 and (packed.max(initial=0) <= 242)
        assert np.array_equal(oracle.unpack3(packed, count), F)
    # all 243 digit combinations are distinct bytes
    import itertools
    seen = {int(oracle.pack3(list(c))[0]) for c in itertools.product((-1, 0, 1), repeat=5)}
    assert seen == set(range(243))
    # payload: N members -> N/2 pair signs -> N/10 bytes (the paper's chunk_size / 10)
    assert len(oracle.pack3(np.zeros(65536 // 2, np.int8))) == -(-65536 // 10)

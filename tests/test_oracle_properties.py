"""Property tests of the oracle (hypothesis): invariances that follow from the definitions in the paper and that a
dropped term, a wrong sign or a transposed operand would break."""
import numpy as np
from hypothesis import given, settings, strategies as st

import oracle
from oracle import q8

SET = settings(max_examples=25, deadline=None, derandomize=True, database=None)


@SET
@given(st.integers(1, 5), st.integers(1, 6), st.sampled_from([1, 2, 4]), st.booleans(), st.integers(0, 2 ** 31 - 1),
       st.floats(-2, 2), st.floats(-2, 2))
def test_forward_is_linear_in_the_input_for_a_fixed_member(m, n, r, anti, seed, a, b):
    """y = x (W + sigma E_i)^T is linear in x: the perturbation depends on the member, not on the data."""
    g = np.random.default_rng(seed)
    W = g.standard_normal((m, n))
    N = 4
    x1, x2 = g.standard_normal((N, n)), g.standard_normal((N, n))
    flags = oracle.ANTITHETIC if anti else 0
    f = lambda X: oracle.perturbed_linear_factored(X, W, np.arange(N), 1, r, 3, seed, flags, 0.4)
    np.testing.assert_allclose(f(a * x1 + b * x2), a * f(x1) + b * f(x2), rtol=1e-9, atol=1e-9)


@SET
@given(st.integers(2, 6), st.integers(2, 6), st.sampled_from([1, 2, 4]), st.booleans(), st.integers(0, 2 ** 31 - 1))
def test_update_is_linear_in_the_fitness_and_ignores_a_constant_under_pairs(m, n, r, anti, seed):
    """dW = (alpha/N) sum_i f_i E_i: additive in f; with antithetic pairs a constant added to every f_i changes nothing."""
    g = np.random.default_rng(seed)
    N = 8
    f1, f2 = g.standard_normal(N), g.standard_normal(N)
    flags = oracle.ANTITHETIC if anti else 0
    d = lambda f: oracle.es_update_block(f, r, 1, seed, flags, 0.3, 0, m, 0, n)
    np.testing.assert_allclose(d(f1 + f2), d(f1) + d(f2), rtol=1e-10, atol=1e-12)
    if anti:
        np.testing.assert_allclose(d(f1 + 7.5), d(f1), rtol=1e-9, atol=1e-10)


@SET
@given(st.lists(st.floats(-1e3, 1e3, allow_nan=False), min_size=2, max_size=40), st.integers(0, 2 ** 31 - 1))
def test_centred_rank_depends_only_on_the_order(values, seed):
    raw = np.array(values, dtype=np.float32)
    out = oracle.fitness_shape(raw, oracle.SHAPE_CENTERED_RANK)
    assert out.min() >= -0.5 and out.max() <= 0.5 and abs(out.sum()) < 1e-9
    # a strictly increasing map of the values leaves the ranks alone (ties stay ties: broken by index on both sides)
    mono = np.float32(3.0) * raw.astype(np.float64) ** 3 + 2.0 * raw.astype(np.float64)
    if len(np.unique(mono.astype(np.float32))) == len(np.unique(raw)):
        assert np.array_equal(oracle.fitness_shape(mono.astype(np.float32), oracle.SHAPE_CENTERED_RANK), out)
    # permuting members of distinct fitness permutes their ranks
    if len(np.unique(raw)) == len(raw):
        perm = np.random.default_rng(seed).permutation(len(raw))
        assert np.array_equal(oracle.fitness_shape(raw[perm], oracle.SHAPE_CENTERED_RANK), out[perm])


@SET
@given(st.lists(st.floats(-100, 100, allow_nan=False), min_size=3, max_size=40), st.floats(0.5, 20), st.floats(-50, 50))
def test_zscore_is_invariant_to_positive_affine_maps(values, scale, shift):
    raw = np.array(values, dtype=np.float64)
    if raw.std() < 1e-3:
        return
    a = oracle.fitness_shape(raw.astype(np.float32), oracle.SHAPE_ZSCORE)
    b = oracle.fitness_shape((scale * raw + shift).astype(np.float32), oracle.SHAPE_ZSCORE)
    np.testing.assert_allclose(a, b, rtol=2e-3, atol=2e-3)
    assert abs(a.mean()) < 1e-4


@SET
@given(st.lists(st.sampled_from([-1, 0, 1]), min_size=0, max_size=64))
def test_base3_packing_round_trips(trits):
    F = np.array(trits, dtype=np.int8)
    packed = oracle.pack3(F)
    assert len(packed) == (len(F) + 4) // 5
    assert np.array_equal(oracle.unpack3(packed, len(F)), F)


@SET
@given(st.integers(1, 6), st.sampled_from([4, 8, 16]), st.integers(0, 2 ** 31 - 1), st.integers(0, 6), st.integers(2, 8))
def test_int8_forward_is_mirrored_by_the_antithetic_partner(m, n, seed, sshift, oshift):
    """Partners share (A_p, B_p) with opposite signs: with W = 0 and no output shift loss, y_- = -y_+ up to the floor."""
    g = np.random.default_rng(seed)
    X = g.integers(-20, 21, size=(2, n)).astype(np.int8)
    X[1] = X[0]
    W = np.zeros((m, n), np.int8)
    table = g.integers(-60, 61, size=256).astype(np.int8)
    y = oracle.perturbed_linear_i8(X, W, np.arange(2), 1, 4, seed, oracle.ANTITHETIC, sshift, 0, table).astype(int)
    # floor shifts: -floor(v) = floor(-v) or floor(-v) + 1, so the mirrored outputs differ by at most one
    assert np.all(np.abs(y[0] + y[1]) <= 1)


@SET
@given(st.integers(1, 6), st.integers(1, 12), st.integers(0, 2 ** 31 - 1), st.floats(0.01, 10))
def test_per_channel_quantisation_commutes_with_row_scaling(m, n, seed, scale):
    """Scaling a whole channel by a power of two scales its scale and leaves its codes alone."""
    g = np.random.default_rng(seed)
    W = g.standard_normal((m, n)).astype(np.float32)
    Q, s = q8.quantize_per_channel(W)
    k = 2.0 ** round(np.log2(scale))
    Q2, s2 = q8.quantize_per_channel((W * np.float32(k)).astype(np.float32))
    assert np.array_equal(Q, Q2) and np.array_equal(s2, s * np.float32(k))
    assert np.all(np.abs(q8.dequantize(Q, s) - W) <= 0.5 * s[:, None] * (1 + 1e-6))

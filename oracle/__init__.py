"""CPU oracle for the EGGROLL hot path -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end over ``egr_oracle.c`` (plain C, fp64 / exact integer).  Only the tests,
the smoke check and the bench's CPU-baseline / reference arm may import this package; the CUDA
library and its Python binding never do, and nothing here imports them.

Every function names the passage of the paper it follows; the arithmetic itself lives in the C file.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "egr_oracle.c")
_SO = os.path.join(_HERE, "libegr_oracle.so")

ANTITHETIC = 1
# element-wise function applied to the output of the perturbed product (bits 2..3 of the flags)
ACT_MASK, ACT_TANH, ACT_RELU, ACT_GELU = 12, 4, 8, 12
SHAPE_NONE, SHAPE_CENTERED_RANK, SHAPE_ZSCORE, SHAPE_ANTITHETIC_SIGN = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no BLAS, no fast-math, no contraction)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-std=c11", "-shared", "-fPIC",
             "-o", _SO, _SRC, "-lm"])
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_normal.restype = ctypes.c_double
        _lib.orc_normal.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                                    ctypes.c_uint64]
        _lib.orc_perturbed_linear_i8.restype = ctypes.c_int
        _lib.orc_es_update_i8.restype = ctypes.c_int
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def threads() -> int:
    """Number of host threads the OpenMP loops will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0))


# ----------------------------------------------------------------------------- noise
def philox4x32_10(ctr, key) -> np.ndarray:
    """Philox4x32-10 block function (Salmon et al. 2011; the paper's counter-based RNG citation)."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c, ctypes.c_uint32), _p(k, ctypes.c_uint32), _p(out, ctypes.c_uint32))
    return out


def noise_factor(seed: int, layer_id: int, p: int, which: int, rows: int, r: int) -> np.ndarray:
    """A_p (which=0, m x r) or B_p (which=1, n x r) of Algorithm 1, as fp64 holding fp32-rounded normals."""
    out = np.zeros((rows, r), dtype=np.float64)
    lib().orc_noise_factor(ctypes.c_uint64(seed), ctypes.c_uint32(layer_id), ctypes.c_uint32(p),
                           ctypes.c_uint32(which), ctypes.c_int(rows), ctypes.c_int(r),
                           _p(out, ctypes.c_double))
    return out


# ----------------------------------------------------------------------------- forward
def activation(Y, flags: int) -> np.ndarray:
    """The element-wise function that follows a perturbed layer in the experiments' networks (tanh and relu in the
    hyperparameter tables of the reinforcement-learning appendix; GELU, in its exact form x Phi(x) with Phi the standard
    normal distribution function, for the transformer workload).  Applied in fp64 to the fp64 product."""
    import math
    act = flags & ACT_MASK
    Y = np.asarray(Y, dtype=np.float64)
    if act == 0:
        return Y
    if act == ACT_TANH:
        return np.tanh(Y)
    if act == ACT_RELU:
        return np.maximum(Y, 0.0)
    erf = np.vectorize(math.erf, otypes=[np.float64])
    return 0.5 * Y * (1.0 + erf(Y / math.sqrt(2.0)))


def _forward(fn, X, W, members, T, r, layer_id, seed, flags, sigma):
    act, flags = flags & ACT_MASK, flags & ~ACT_MASK
    return activation(_forward_linear(fn, X, W, members, T, r, layer_id, seed, flags, sigma), act)


def _forward_linear(fn, X, W, members, T, r, layer_id, seed, flags, sigma):
    W = _f64(W)
    m, n = W.shape
    members = np.ascontiguousarray(members, dtype=np.int32)
    X = _f64(X)
    assert X.shape == (len(members) * T, n), (X.shape, len(members), T, n)
    Y = np.zeros((len(members) * T, m), dtype=np.float64)
    fn(_p(X, ctypes.c_double), _p(W, ctypes.c_double), _p(members, ctypes.c_int32),
       ctypes.c_int(len(members)), ctypes.c_int(T), ctypes.c_int(m), ctypes.c_int(n), ctypes.c_int(r),
       ctypes.c_uint32(layer_id), ctypes.c_uint64(seed), ctypes.c_uint32(flags), ctypes.c_double(sigma),
       _p(Y, ctypes.c_double))
    return Y


def perturbed_linear(X, W, members, T, r, layer_id, seed, flags, sigma) -> np.ndarray:
    """y = x (W + sigma E_i)^T with E_i formed explicitly (Algorithm 1; Section 4.2, left-hand side).

    ``X`` holds the rows of the selected ``members`` only, member-major, ``T`` rows each."""
    return _forward(lib().orc_perturbed_linear_explicit, X, W, members, T, r, layer_id, seed, flags, sigma)


def perturbed_linear_factored(X, W, members, T, r, layer_id, seed, flags, sigma) -> np.ndarray:
    """Same through u M^T + (sigma/sqrt r)(u B) A^T (Section 4.2, right-hand side)."""
    return _forward(lib().orc_perturbed_linear_factored, X, W, members, T, r, layer_id, seed, flags, sigma)


def perturbed_linear_blas(X, W, members, T, r, layer_id, seed, flags, sigma) -> np.ndarray:
    """The explicit form once more, for layers too large for the plain loops: every selected member's
    W_i = W + sigma sign_i A_p B_p^T / sqrt(r) is formed in fp64 (factors from ``noise_factor``) and applied with the
    library matrix product, y = x W_i^T (Algorithm 1; Section 4.2, left-hand side).  Nothing is blocked or fused; the
    only difference from ``perturbed_linear`` is who runs the inner loops."""
    act, flags = flags & ACT_MASK, flags & ~ACT_MASK
    W = _f64(W)
    X = _f64(X)
    m, n = W.shape
    assert X.shape == (len(members) * T, n)
    Y = np.zeros((len(members) * T, m), dtype=np.float64)
    for k, i in enumerate(members):
        i = int(i)
        p, sign = ((i >> 1), (1.0 - 2.0 * (i & 1))) if flags & ANTITHETIC else (i, 1.0)
        A = noise_factor(seed, layer_id, p, 0, m, r)
        B = noise_factor(seed, layer_id, p, 1, n, r)
        Wi = W + (sigma * sign / math.sqrt(r)) * (A @ B.T)
        Y[k * T:(k + 1) * T] = X[k * T:(k + 1) * T] @ Wi.T
    return activation(Y, act)


def token_log_likelihood(logits, targets) -> np.ndarray:
    """log p(target) = z[target] - log sum_j exp(z[j]) per row (the fitness of the LLM fine-tuning experiments is the
    log-likelihood of the tokens); rows whose target lies outside [0, V) are not scored and give 0."""
    z = _f64(logits)
    targets = np.asarray(targets, dtype=np.int64)
    out = np.zeros(z.shape[0], dtype=np.float64)
    for i in range(z.shape[0]):
        t = int(targets[i])
        if 0 <= t < z.shape[1]:
            m = z[i].max()
            out[i] = z[i, t] - (m + math.log(np.exp(z[i] - m).sum()))
    return out


# ----------------------------------------------------------------------------- update
def es_update_block(fitness, r, layer_id, seed, flags, alpha, j0, j1, l0, l1) -> np.ndarray:
    """Block [j0:j1, l0:l1] of dW = (alpha/N) sum_i f_i E_i (boxed EGGROLL update), explicit outer products."""
    f = _f64(fitness)
    out = np.zeros((j1 - j0, l1 - l0), dtype=np.float64)
    lib().orc_es_update_block(_p(f, ctypes.c_double), ctypes.c_int(len(f)), ctypes.c_int(r),
                              ctypes.c_uint32(layer_id), ctypes.c_uint64(seed), ctypes.c_uint32(flags),
                              ctypes.c_double(alpha), ctypes.c_int(j0), ctypes.c_int(j1), ctypes.c_int(l0),
                              ctypes.c_int(l1), _p(out, ctypes.c_double))
    return out


def es_update(W, fitness, r, layer_id, seed, flags, alpha):
    """Full update: returns (W + dW, dW)."""
    W = _f64(W)
    m, n = W.shape
    dW = es_update_block(fitness, r, layer_id, seed, flags, alpha, 0, m, 0, n)
    return W + dW, dW


# ----------------------------------------------------------------------------- shaping
def fitness_shape(raw, mode: int) -> np.ndarray:
    """Centred rank (HFT appendix), z-score, or antithetic sign (integer appendix, Fitness Shaping)."""
    raw = _f64(raw)
    out = np.zeros_like(raw)
    lib().orc_fitness_shape(_p(raw, ctypes.c_double), ctypes.c_int(len(raw)), ctypes.c_int(mode),
                            _p(out, ctypes.c_double))
    return out


def fitness_shape_questions(S) -> np.ndarray:
    """Per-question centred, globally scaled scores averaged over questions (LLM fine-tuning section)."""
    S = _f64(S)
    N, Q = S.shape
    out = np.zeros(N, dtype=np.float64)
    lib().orc_fitness_shape_questions(_p(S, ctypes.c_double), ctypes.c_int(N), ctypes.c_int(Q), _p(out, ctypes.c_double))
    return out


# ----------------------------------------------------------------------------- integer path
def i8_offsets(seed, layer_id, p, table_log2):
    a, b = ctypes.c_uint32(0), ctypes.c_uint32(0)
    lib().orc_i8_offsets(ctypes.c_uint64(seed), ctypes.c_uint32(layer_id), ctypes.c_uint32(p),
                         ctypes.c_uint32(table_log2), ctypes.byref(a), ctypes.byref(b))
    return a.value, b.value


def perturbed_linear_i8(X, W, members, T, layer_id, seed, flags, sigma_shift, out_shift, table) -> np.ndarray:
    """I8((u theta^T + ((u.B) I32(A) >> (4+sigma_hat))) / (16 sqrt n)) (Adding EGGROLL Perturbations)."""
    X = np.ascontiguousarray(X, dtype=np.int8)
    W = np.ascontiguousarray(W, dtype=np.int8)
    table = np.ascontiguousarray(table, dtype=np.int8)
    L = int(np.log2(len(table)))
    assert 1 << L == len(table)
    m, n = W.shape
    members = np.ascontiguousarray(members, dtype=np.int32)
    assert X.shape == (len(members) * T, n)
    Y = np.zeros((len(members) * T, m), dtype=np.int8)
    ovf = lib().orc_perturbed_linear_i8(
        _p(X, ctypes.c_int8), _p(W, ctypes.c_int8), _p(members, ctypes.c_int32), ctypes.c_int(len(members)),
        ctypes.c_int(T), ctypes.c_int(m), ctypes.c_int(n), ctypes.c_uint32(layer_id), ctypes.c_uint64(seed),
        ctypes.c_uint32(flags), ctypes.c_int(sigma_shift), ctypes.c_int(out_shift), _p(table, ctypes.c_int8),
        ctypes.c_uint32(L), _p(Y, ctypes.c_int8))
    if ovf:
        raise OverflowError("int32 range exceeded in the integer perturbed matmul")
    return Y


def fitness_shape_i8(raw) -> np.ndarray:
    """sign(s+ - s-) per antithetic pair (integer appendix, Fitness Shaping)."""
    raw = np.ascontiguousarray(raw, dtype=np.int32)
    out = np.zeros(len(raw) // 2, dtype=np.int8)
    lib().orc_fitness_shape_i8(_p(raw, ctypes.c_int32), ctypes.c_int(len(raw)), _p(out, ctypes.c_int8))
    return out


def es_update_i8(W, F, layer_id, seed, threshold, table):
    """E = (diag(F) A)^T B, one-bin move where |E| >= threshold (integer appendix, Parameter Update).

    Returns (W_new, E)."""
    Wn = np.array(W, dtype=np.int8, order="C", copy=True)
    F = np.ascontiguousarray(F, dtype=np.int8)
    table = np.ascontiguousarray(table, dtype=np.int8)
    L = int(np.log2(len(table)))
    assert 1 << L == len(table)
    m, n = Wn.shape
    E = np.zeros((m, n), dtype=np.int32)
    ovf = lib().orc_es_update_i8(_p(Wn, ctypes.c_int8), _p(F, ctypes.c_int8), ctypes.c_int(len(F)),
                                 ctypes.c_int(m), ctypes.c_int(n), ctypes.c_uint32(layer_id),
                                 ctypes.c_uint64(seed), ctypes.c_int32(threshold), _p(table, ctypes.c_int8),
                                 ctypes.c_uint32(L), _p(E, ctypes.c_int32))
    if ovf:
        raise OverflowError("int32 range exceeded in the integer update")
    return Wn, E


# ----------------------------------------------------------------------------- integer recurrent LM
def pack3(F) -> np.ndarray:
    """Base-3 packing of ternary pair signs ("Base-3 Fitness Packing"): +1, 0, -1 -> digits 0, 1, 2;
    byte = sum_{i<5} digit_i 3^i.  Missing trailing values count as 0 (digit 1)."""
    F = np.asarray(F, dtype=np.int64)
    digit = {1: 0, 0: 1, -1: 2}
    out = np.zeros((len(F) + 4) // 5, dtype=np.uint8)
    for b in range(len(out)):
        byte = 0
        for i in range(5):
            e = 5 * b + i
            byte += digit[int(F[e]) if e < len(F) else 0] * 3 ** i
        out[b] = byte
    return out


def unpack3(packed, count: int) -> np.ndarray:
    """Inverse of pack3: the first ``count`` ternary values."""
    value = {0: 1, 1: 0, 2: -1}
    out = np.zeros(count, dtype=np.int8)
    for e in range(count):
        out[e] = value[(int(packed[e // 5]) // 3 ** (e % 5)) % 3]
    return out


class _OrcLM(ctypes.Structure):
    _fields_ = [("D", ctypes.c_int), ("n_layers", ctypes.c_int)] + \
               [(k, ctypes.c_void_p) for k in ("emb_t", "head", "ln_out", "ln1", "ln2", "Wf", "Uf", "Wh", "Uh",
                                               "bf", "bh", "mlp1", "mlp2", "lut_sigma", "lut_phi", "table")] + \
               [("table_log2", ctypes.c_uint32), ("seed", ctypes.c_uint64), ("flags", ctypes.c_uint32),
                ("sigma_shift", ctypes.c_int)]


def exp2_table() -> np.ndarray:
    """EXP2[i] = 16 * 2^(i/16) rounded (Fitness Calculation in Integer Types)."""
    lib().orc_exp2_table.restype = ctypes.c_int32
    return np.array([lib().orc_exp2_table(ctypes.c_int(i)) for i in range(256)], dtype=np.int32)


def log2_int(S: int) -> int:
    """Integer LOG2(S) ~ 16 log2(S/16)."""
    lib().orc_log2_int.restype = ctypes.c_int32
    return int(lib().orc_log2_int(ctypes.c_int64(S)))


def i8lm_forward(params: dict, tokens, members, member_seq, seed, flags, sigma_shift, table, state=None):
    """EGG forward pass (Algorithm "EGG forward pass") under per-member integer perturbations.

    ``params``: emb_t [D,256], head [256,D], ln_out [D], ln1/ln2 [l,D], Wf/Uf/Wh/Uh [l,D,D], bf/bh [l,D],
    mlp1 [l,4D,D], mlp2 [l,D,4D], lut_sigma/lut_phi [256].  Returns (fitness int32 [n_sel], state int8 [n_sel,l,D])."""
    keep = {k: np.ascontiguousarray(v, dtype=np.int8) for k, v in params.items()}
    table = np.ascontiguousarray(table, dtype=np.int8)
    L = int(np.log2(len(table)))
    l, D = keep["ln1"].shape
    tokens = np.ascontiguousarray(tokens, dtype=np.uint8)
    members = np.ascontiguousarray(members, dtype=np.int32)
    member_seq = np.ascontiguousarray(member_seq, dtype=np.int32)
    n_sel = len(members)
    st = np.zeros((n_sel, l, D), dtype=np.int8) if state is None else np.array(state, dtype=np.int8, order="C", copy=True)
    fit = np.zeros(n_sel, dtype=np.int32)
    M = _OrcLM(D, l, *[keep[k].ctypes.data for k in ("emb_t", "head", "ln_out", "ln1", "ln2", "Wf", "Uf", "Wh", "Uh",
                                                     "bf", "bh", "mlp1", "mlp2", "lut_sigma", "lut_phi")],
               table.ctypes.data, L, seed, flags, sigma_shift)
    lib().orc_i8lm_forward.restype = ctypes.c_int
    ovf = lib().orc_i8lm_forward(ctypes.byref(M), _p(tokens, ctypes.c_uint8), ctypes.c_int(tokens.shape[1]),
                                 _p(members, ctypes.c_int32), _p(member_seq, ctypes.c_int32), ctypes.c_int(n_sel),
                                 _p(st, ctypes.c_int8), _p(fit, ctypes.c_int32))
    if ovf:
        raise OverflowError("int32 range exceeded in the integer LM")
    return fit, st

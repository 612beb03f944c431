"""TEST INFRASTRUCTURE -- CPU oracle for the per-channel int8 fine-tuning path (appendix "Fine-tuning of Integer
Quantised Models": "Quantisation Procedure" and "Integrating integer-quantised EGGROLL with Adam").

Plain numpy, written from the paper's equations; shares no code with the CUDA path.  Only tests, the smoke check and
the CPU-baseline leg of the benchmark may import it.

Precision.  The paper fixes bf16 storage for the channel scales, for Adam's proposal u and for both moments, and an
int8 lattice for Q; everything that decides an integer (the quantised code, the unit step) is therefore evaluated
here in fp32 with one rounding per operation, in the order written below, which a kernel can follow bit for bit.
The forward is a real-valued function and is evaluated in fp64.  The mean and deviation of u are taken in fp64 and
rounded once to fp32 before the comparison.

Readings of what the appendix leaves open (each is also listed in the design notes):
  * layout: Q is [d_out][d_in], one scale per output channel (row); round = round-half-to-even; Q is computed with
    the stored (bf16-rounded) scale, so that Q * s reproduces W to within s/2;
  * the forward applies the scales to the accumulated sum: y_j = s_x s_j (sum_l x_l Q_jl + low-rank term);
  * "explicit scale perturbations" are additive Gaussian: member i sees s_j + sign_i sigma_s e_p[j] and
    s_x + sign_i sigma_s e_p[d_out], e_p = noise factor with tag 3 (d_out + 1 elements, rank 1) of its noise index;
  * the ES gradient estimates are (1/N) sum_i f_i E_i for Q (the boxed update without the step size) and
    (1/N) sum_i f_i sign_i e_p(i) for the scales;
  * Adam is the textbook rule with bias correction and epsilon outside the square root, ascending the fitness:
    u = +lr m_hat / (sqrt(v_hat) + eps), evaluated as (lr / (1 - b1^t)) m / (sqrt(v) / sqrt(1 - b2^t) + eps) with the
    two scalar factors formed once; the proposal uses the fp32 moments of this step, which are then stored rounded
    to bf16; sigma(u) is the population deviation (divide by the count).
"""
from __future__ import annotations

import math

import numpy as np

from . import ANTITHETIC, es_update_block, noise_factor, perturbed_linear_factored

TAG_SCALE = 3
F32 = np.float32


def bf16_round(a) -> np.ndarray:
    """Nearest-even rounding of fp32 values to bf16, returned as fp32 (NaN stays NaN)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    rounded = ((bits + 0x7FFF + ((bits >> 16) & 1)) >> 16) << 16
    out = (rounded & 0xFFFFFFFF).astype(np.uint32).view(np.float32).reshape(a.shape)
    return np.where(np.isnan(a), a, out)


# ----------------------------------------------------------------------------- quantisation ("Quantisation Procedure")
def quantize_per_channel(W, eps: float = 1e-8):
    """s_i = bf16(max(max_j |W_ij| / 127, eps)); Q_ij = clip(round(W_ij / s_i), -127, 127).  Returns (Q int8, s fp32)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    absmax = np.max(np.abs(W), axis=1).astype(F32) if W.shape[1] else np.zeros(W.shape[0], F32)
    s = bf16_round(np.maximum(absmax / F32(127.0), F32(eps)).astype(F32))
    q = np.rint((W / s[:, None]).astype(F32))
    return np.clip(q, -127, 127).astype(np.int8), s


def dequantize(Q, s) -> np.ndarray:
    return Q.astype(np.float64) * np.asarray(s, dtype=np.float64)[:, None]


# ----------------------------------------------------------------------------- forward
def _member_noise(member: int, flags: int):
    if flags & ANTITHETIC:
        return member >> 1, (-1.0 if member & 1 else 1.0)
    return member, 1.0


def scale_noise(seed: int, layer_id: int, p: int, d_out: int) -> np.ndarray:
    """e_p: d_out channel-scale normals followed by the one for the input scale."""
    return noise_factor(seed, layer_id, p, TAG_SCALE, d_out + 1, 1)[:, 0]


def perturbed_linear_q8(X, Q, s, s_x, members, T, r, layer_id, seed, flags, sigma, sigma_s=0.0) -> np.ndarray:
    """y_j = (s_x + sign sigma_s e[m]) (s_j + sign sigma_s e[j]) (sum_l x_l Q_jl + sign (sigma/sqrt r) (x B_p) A_p[j]^T)."""
    Q = np.asarray(Q)
    m = Q.shape[0]
    assert flags & ~(ANTITHETIC | 2) == 0, "no element-wise function is defined for the scaled forward"
    core = perturbed_linear_factored(X, Q.astype(np.float64), members, T, r, layer_id, seed, flags, sigma)
    s = np.asarray(s, dtype=np.float64)
    out = np.empty_like(core)
    for idx, member in enumerate(np.asarray(members)):
        p, sign = _member_noise(int(member), flags)
        if sigma_s != 0.0:
            e = scale_noise(seed, layer_id, p, m)
            col = (float(s_x) + sign * sigma_s * e[m]) * (s + sign * sigma_s * e[:m])
        else:
            col = float(s_x) * s
        out[idx * T:(idx + 1) * T] = core[idx * T:(idx + 1) * T] * col[None, :]
    return out


# ----------------------------------------------------------------------------- ES gradient estimates ("ES gradients")
def es_gradient_block(fitness, r, layer_id, seed, flags, j0, j1, l0, l1) -> np.ndarray:
    """Block of G = (1/N) sum_i f_i E_i for the quantised matrix (low-rank pathway)."""
    return es_update_block(fitness, r, layer_id, seed, flags, 1.0, j0, j1, l0, l1)


def es_scale_gradient(fitness, d_out, layer_id, seed, flags) -> np.ndarray:
    """g[j] = (1/N) sum_i f_i sign_i e_p(i)[j], j = 0 .. d_out (the last entry belongs to s_x)."""
    f = np.asarray(fitness, dtype=np.float64)
    N = len(f)
    g = np.zeros(d_out + 1)
    for i in range(N):
        p, sign = _member_noise(i, flags)
        g += f[i] * sign * scale_noise(seed, layer_id, p, d_out)
    return g / N


# ----------------------------------------------------------------------------- Adam ("Adam updates for int8 tensors")
def adam_proposal(g, mom1, mom2, t: int, lr, b1, b2, eps):
    """One Adam step in fp32 on bf16-stored moments.  Returns (u bf16-valued fp32, mom1', mom2' bf16-valued fp32)."""
    g = np.asarray(g, dtype=F32)
    m0, v0 = np.asarray(mom1, dtype=F32), np.asarray(mom2, dtype=F32)
    b1, b2, lr, eps = F32(b1), F32(b2), F32(lr), F32(eps)
    c1, c2 = F32(1.0) - b1, F32(1.0) - b2
    # bias corrections folded into two scalars, evaluated in double and rounded once:
    # u = (lr / (1 - b1^t)) m' / (sqrt(v') / sqrt(1 - b2^t) + eps)
    step = F32(float(lr) / (1.0 - float(b1) ** t))
    rsb2 = F32(1.0 / math.sqrt(1.0 - float(b2) ** t))
    m1 = (b1 * m0).astype(F32) + (c1 * g).astype(F32)
    v1 = (b2 * v0).astype(F32) + (c2 * (g * g).astype(F32)).astype(F32)
    den = (np.sqrt(v1).astype(F32) * rsb2).astype(F32) + eps
    u = ((step * m1).astype(F32) / den).astype(F32)
    return bf16_round(u), bf16_round(m1), bf16_round(v1)


def unit_step(u, tau):
    """Delta = sign(z) 1{|z| >= tau}, z = (u - mean(u)) / (std(u) + 1e-8), evaluated as |u - mean| >= tau (std + 1e-8)."""
    u = np.asarray(u, dtype=F32)
    u64 = u.astype(np.float64)
    mu = F32(u64.mean()) if u.size else F32(0)
    thr = F32(float(tau) * (u64.std() + 1e-8)) if u.size else F32(0)
    d = (u - mu).astype(F32)
    return (np.sign(d) * (np.abs(d) >= thr)).astype(np.int8)


def adam_step_q8(Q, g, mom1, mom2, t, lr, b1, b2, eps, tau):
    """Discretised Adam on an int8 tensor: Q <- clip(Q + Delta, -127, 127).  Returns (Q', mom1', mom2', u, Delta)."""
    u, m1, v1 = adam_proposal(g, mom1, mom2, t, lr, b1, b2, eps)
    delta = unit_step(u, tau)
    Qn = np.clip(np.asarray(Q, dtype=np.int16) + delta, -127, 127).astype(np.int8)
    return Qn, m1, v1, u, delta


def adam_step_bf16(param, g, mom1, mom2, t, lr, b1, b2, eps):
    """Adam on a bf16 floating-point leaf (the scales): param <- bf16(param + u).  Returns (param', mom1', mom2')."""
    u, m1, v1 = adam_proposal(g, mom1, mom2, t, lr, b1, b2, eps)
    return bf16_round(np.asarray(param, dtype=F32) + u), m1, v1

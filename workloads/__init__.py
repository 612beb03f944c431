"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds data recipes only (numpy's PCG64 streams, rounding of stored values to the storage
dtype).  It contains none of the method's arithmetic: no perturbation noise, no forward, no update.
Both the CPU oracle's tests and the CUDA path's tests / bench draw their inputs from here.
"""
from __future__ import annotations

import numpy as np


def rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed), int(stream)]))


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result kept as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """Upper 16 bits of fp32 values that are already exactly representable in bf16."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


def linear_layer(seed: int, m: int, n: int, rows: int, *, bf16: bool, w_std=None):
    """One linear layer W[m,n] ~ N(0, w_std^2) (default 1/n variance) and inputs X[rows,n] ~ N(0,1)."""
    g = rng(seed, 1)
    std = (1.0 / np.sqrt(n)) if w_std is None else w_std
    W = (g.standard_normal((m, n)) * std).astype(np.float32)
    X = g.standard_normal((rows, n)).astype(np.float32)
    if bf16:
        W, X = round_to_bf16(W), round_to_bf16(X)
    return W, X


def pair_shared_rows(X: np.ndarray, T: int) -> np.ndarray:
    """Make antithetic partners (members 2p, 2p+1) see identical inputs: copy member 2p's T rows."""
    X = X.copy()
    R, n = X.shape
    Xm = X.reshape(R // T, T, n)
    Xm[1::2] = Xm[0::2]
    return Xm.reshape(R, n)


def raw_fitness(seed: int, N: int) -> np.ndarray:
    return rng(seed, 2).standard_normal(N).astype(np.float32)


def int8_matrix(seed: int, stream: int, shape) -> np.ndarray:
    """round(16 z) clipped to [-127,127]: the integer model's standard initialisation / noise table law."""
    z = rng(seed, stream).standard_normal(shape)
    return np.clip(np.rint(16.0 * z), -127, 127).astype(np.int8)


def int8_activations(seed: int, stream: int, shape) -> np.ndarray:
    return int8_matrix(seed, stream, shape)


def noise_table(seed: int, table_log2: int) -> np.ndarray:
    """Pre-generated table of round(16 z) int8 values the integer path slices its perturbations from."""
    return int8_matrix(seed, 7, (1 << table_log2,))


def markov_bytes(seed: int, n_seq: int, length: int) -> np.ndarray:
    """Byte sequences from a first-order Markov chain with transition matrix softmax(2 G), G ~ N(0,1)."""
    g = rng(seed, 20)
    G = g.standard_normal((256, 256))
    P = np.exp(2.0 * G - (2.0 * G).max(axis=1, keepdims=True))
    P /= P.sum(axis=1, keepdims=True)
    cdf = np.cumsum(P, axis=1)
    out = np.zeros((n_seq, length), dtype=np.uint8)
    out[:, 0] = g.integers(0, 256, size=n_seq)
    u = g.random((n_seq, length))
    for t in range(1, length):
        rows = cdf[out[:, t - 1]]
        out[:, t] = np.minimum((rows < u[:, t:t + 1]).sum(axis=1), 255)
    return out


# ----------------------------------------------------------------------------- named configurations
def config1():
    """Single fp32 linear layer m=n=64, 16 antithetic pairs, r=1."""
    W, X = linear_layer(0, 64, 64, 32, bf16=False)
    X = pair_shared_rows(X, 1)
    t = rng(0, 3).standard_normal(64).astype(np.float32)
    return dict(W=W, X=X, target=t, N=32, T=1, r=1, sigma=0.1, alpha=0.01, steps=10, seed=0,
                antithetic=True)


def config5(N: int, r: int, seed: int = 0):
    """One 4096x4096 bf16 layer, one token per member."""
    W, X = linear_layer(seed, 4096, 4096, N, bf16=True)
    return dict(W=W, X=X, N=N, T=1, r=r, sigma=0.01, alpha=0.01, seed=seed, antithetic=False,
                raw=raw_fitness(seed, N))


def egg_lm_params(seed: int, D: int = 256, n_layers: int = 4, lut: str = "identity"):
    """Parameters of the integer recurrent LM with the paper's initialisation: matrices round(16 z), layer-norm
    weights 16, biases 0.  The embedding is stored transposed ([D,256], column t = byte t).  ``lut`` selects the
    256-entry gate tables: "identity" (the paper's choice) or "hard" (a hard-tanh-like clamp to +-64)."""
    g = lambda i, shape: int8_matrix(seed, 100 + i, shape)
    v = np.arange(-128, 128)
    if lut == "identity":
        t = np.clip(v, -127, 127)
    else:
        t = np.clip(v, -64, 64)
    return dict(
        emb_t=g(0, (D, 256)), head=g(1, (256, D)), ln_out=np.full(D, 16, np.int8),
        ln1=np.full((n_layers, D), 16, np.int8), ln2=np.full((n_layers, D), 16, np.int8),
        Wf=g(2, (n_layers, D, D)), Uf=g(3, (n_layers, D, D)), Wh=g(4, (n_layers, D, D)), Uh=g(5, (n_layers, D, D)),
        bf=np.zeros((n_layers, D), np.int8), bh=np.zeros((n_layers, D), np.int8),
        mlp1=g(6, (n_layers, 4 * D, D)), mlp2=g(7, (n_layers, D, 4 * D)),
        lut_sigma=t.astype(np.int8), lut_phi=t.astype(np.int8))


def egg_lm_param_count(params: dict) -> int:
    return int(sum(v.size for k, v in params.items() if not k.startswith("lut_")))


def bf16_normal_matrix_torch(seed: int, stream: int, m: int, n: int, std: float, device):
    """A bf16 matrix ~ N(0, std^2) drawn on ``device`` from torch's seeded generator, for models too large to draw with
    numpy in a test's time (the 1.3 B-parameter decoder).  Both sides of a parity test read the same tensor: the
    oracle takes ``.float().cpu().numpy()`` of it, so the generator's device does not matter to the comparison."""
    import torch
    g = torch.Generator(device=device).manual_seed(int(seed) * 100003 + int(stream))
    return (torch.randn((m, n), device=device, generator=g, dtype=torch.float32) * std).to(torch.bfloat16)

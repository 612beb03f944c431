"""One integer-EGGROLL training step of the recurrent byte-level LM ("EGG Pretraining with Integer EGGROLL").

Plumbing only: it chains the library's entry points -- population forward with carried state, pair-sign fitness
shaping, and the one-bin integer update of every perturbed matrix (the four GRU matrices and the two MLP matrices of
each layer, the embedding and the head).  Layer-norm weights and biases are neither perturbed nor updated.
"""
from __future__ import annotations

import math

from . import api as egr

# layer ids of the perturbed matrices: 16*layer + slot; embedding 1000, head 1001
SLOTS = {"Wf": 0, "Uf": 1, "Wh": 2, "Uh": 3, "mlp1": 4, "mlp2": 5}


def alpha_schedule(step: int) -> float:
    """alpha_t = 1 / (0.015 t + 1) ("Parameter Update", last paragraph)."""
    return 1.0 / (0.015 * step + 1.0)


def update_threshold(alpha: float, n_noise: int) -> int:
    """I32(16 Phi^-1(1 - alpha/2)) * I32(16 sqrt(K)) with truncating casts; K = number of distinct noise vectors.

    (The printed argument (1 - alpha)/2 gives a negative quantile and contradicts "alpha is about the fraction of
    parameters updated"; this is the reading under which that sentence holds.)"""
    from statistics import NormalDist
    q = 1.0 - alpha / 2.0
    z = NormalDist().inv_cdf(q) if q < 1.0 else float("inf")
    zi = int(16.0 * z) if math.isfinite(z) else 2 ** 20
    return max(0, min(2 ** 31 - 1, zi * int(16.0 * math.sqrt(n_noise))))


def perturbed_matrices(params: dict):
    """(tensor view, layer_id) of every matrix the update touches, in a fixed order."""
    n_layers = params["ln1"].shape[0]
    out = []
    for i in range(n_layers):
        for name, slot in SLOTS.items():
            out.append((params[name][i], 16 * i + slot))
    out.append((params["emb_t"], 1000))
    out.append((params["head"], 1001))
    return out


def egg_step(params: dict, n_members: int, seed: int, sigma_shift: int, noise_table, tokens, member_seq, state, alpha: float,
             ws: "egr.Workspace"):
    """Forward over ``tokens`` (state carried in ``state``), sign(s+ - s-) per antithetic pair, then the integer update
    of every matrix in place.  Returns (raw fitness [N] int32, shaped fitness [N/2] int8, threshold)."""
    import torch
    dev = noise_table.device
    fitness = torch.zeros(n_members, dtype=torch.int32, device=dev)
    egr.egr_i8lm_forward(params, n_members, seed, egr.ANTITHETIC, sigma_shift, noise_table, tokens, member_seq, state,
                         fitness, ws)
    F = torch.empty(n_members // 2, dtype=torch.int8, device=dev)
    egr.egr_fitness_shape_i8(fitness, F)
    thr = update_threshold(alpha, n_members // 2)
    for W, layer_id in perturbed_matrices(params):
        m, n = W.shape
        L = egr.Layer(n, m, n_members, 1, 1, layer_id=layer_id, seed=seed, flags=egr.ANTITHETIC,
                      x_dtype=egr.I8, w_dtype=egr.I8, y_dtype=egr.I8)
        egr.egr_es_update_i8(L, W, F, thr, noise_table, ws)
    return fitness, F, thr

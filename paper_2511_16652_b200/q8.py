"""One EGGROLL step on a per-channel-scaled int8 matrix with the discretised Adam update ("Fine-tuning of Integer
Quantised Models").

Plumbing only: it holds the tensors of one quantised matrix parameter (codes, channel scales, input scale, Adam
moments) and chains the library's entry points -- quantisation, the scaled perturbed forward, the two gradient
estimates, Adam on the bf16 leaves and the thresholded unit step on the codes.  All arithmetic runs in the kernels
behind the C ABI (`include/egr_q8.h`).
"""
from __future__ import annotations

from . import api as egr


class Q8Matrix:
    """Q [m, n] int8 codes, scales [m] bf16, s_x (one bf16 value kept in a 1-element tensor), and the Adam state."""

    def __init__(self, W, eps: float = 1e-8, s_x: float = 1.0, layer_id: int = 0):
        import torch
        m, n = W.shape
        if n % 16:
            raise ValueError("d_in must be a multiple of 16 (pitch of the int8 codes)")
        dev = W.device
        self.layer_id = layer_id
        self.Q = torch.empty((m, n), dtype=torch.int8, device=dev)
        # one leaf of m + 1 bf16 values: the channel scales followed by the input scale (the order of the scale noise)
        self.leaf = torch.empty(m + 1, dtype=torch.bfloat16, device=dev)
        egr.egr_q8_quantize(W.float().contiguous(), eps, self.Q, self.leaf[:m])
        self.leaf[m] = s_x
        self._s_x_host = None                # host copy of the (bf16-rounded) input scale: the forward takes it by value
        self.mom1 = torch.zeros((m, n), dtype=torch.bfloat16, device=dev)
        self.mom2 = torch.zeros((m, n), dtype=torch.bfloat16, device=dev)
        self.leaf_mom1 = torch.zeros(m + 1, dtype=torch.bfloat16, device=dev)
        self.leaf_mom2 = torch.zeros(m + 1, dtype=torch.bfloat16, device=dev)
        self.G = torch.empty((m, n), dtype=torch.float32, device=dev)
        self.g_leaf = torch.empty(m + 1, dtype=torch.float32, device=dev)
        self.n_changed = torch.zeros(1, dtype=torch.int64, device=dev)
        self.t = 0

    @property
    def shape(self):
        return tuple(self.Q.shape)

    @property
    def scales(self):
        return self.leaf[: self.Q.shape[0]]

    @property
    def s_x(self) -> float:
        if self._s_x_host is None:           # refreshed once after the scales moved
            self._s_x_host = float(self.leaf[self.Q.shape[0]].item())
        return self._s_x_host

    def layer(self, n_members: int, rows_per_member: int, rank: int, seed: int, flags: int, y_dtype=egr.BF16):
        m, n = self.Q.shape
        return egr.Layer(n, m, n_members, rows_per_member, rank, layer_id=self.layer_id, seed=seed, flags=flags,
                         x_dtype=egr.BF16, w_dtype=egr.I8, y_dtype=y_dtype)

    def forward(self, X, Y, n_members: int, rows_per_member: int, rank: int, seed: int, flags: int, sigma: float,
                sigma_s: float, ws: "egr.Workspace"):
        """Y = population forward of X through this matrix under the members' perturbations."""
        y_dtype = egr.F32 if Y.dtype.is_floating_point and Y.element_size() == 4 else egr.BF16
        L = self.layer(n_members, rows_per_member, rank, seed, flags, y_dtype)
        return egr.egr_perturbed_linear_q8(L, X, self.Q, self.scales, self.s_x, sigma, sigma_s, Y, ws)

    def update(self, shaped_fitness, n_members: int, rank: int, seed: int, flags: int, lr: float, tau: float,
               ws: "egr.Workspace", lr_scales: float = 0.0, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8):
        """Gradient estimates from the shaped fitness, then Adam: unit steps on the codes (threshold tau) and, when
        ``lr_scales`` is not zero, a plain Adam step on the scales.  Returns the number of codes that moved."""
        self.t += 1
        L = self.layer(n_members, 1, rank, seed, flags)
        egr.egr_es_gradient(L, shaped_fitness, self.G, ws)
        egr.egr_adam_step_q8(self.Q, self.G, self.mom1, self.mom2, self.t, lr, beta1, beta2, eps, tau, ws,
                             n_changed=self.n_changed)
        if lr_scales != 0.0:
            egr.egr_es_scale_gradient(L, shaped_fitness, self.g_leaf, ws)
            egr.egr_adam_step_bf16(self.leaf, self.g_leaf, self.leaf_mom1, self.leaf_mom2, self.t, lr_scales, beta1, beta2, eps)
            self._s_x_host = None
        return self.n_changed

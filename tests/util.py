"""Shared helpers for the parity tests (no arithmetic of the method lives here)."""
import numpy as np


def rel_fro(got, want) -> float:
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    den = np.linalg.norm(want)
    return float(np.linalg.norm(got - want) / (den if den > 0 else 1.0))


def to_dev(a, dtype=None):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t if dtype is None else t.to(dtype)


def padded(a, ld, dtype=None):
    """Device copy of a 2-D array inside a buffer with row pitch ld (elements); returns (buffer, view)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    buf = torch.zeros((a.shape[0], ld), dtype=t.dtype, device="cuda")
    buf[:, : a.shape[1]] = t.cuda()
    return buf

"""The allocation-free forward entry point, for hosts that cannot hand the library a workspace.

Some users of this library live inside a memory plan they do not control (a plug-in that only receives its
input and output buffers, a process whose device memory was partitioned before the library was loaded, code
that must not call cudaMalloc because it would synchronise the device).  For them
``egr_perturbed_linear_static`` keeps its scratch in a fixed array of about 1 MiB inside the library.  This file checks
it against the regular entry point, twice in a row (the array is shared and keeps the previous call's
contents), and is named so that pytest collects it last.
"""
import ctypes

import numpy as np
import pytest

import workloads


def _rel(a, b):
    a = a.astype(np.float64)
    b = b.astype(np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


@pytest.mark.gpu
def test_static_forward_matches_workspace_forward_twice():
    import torch
    import paper_2511_16652_b200 as egr
    egr.load_library()
    ws = egr.Workspace()
    cases = [
        # N, T, m, n, r, flags, dtype code
        (300, 1, 520, 200, 4, egr.ANTITHETIC, egr.BF16),
        (64, 8, 264, 784, 16, 0, egr.BF16),
        (70, 1, 12, 784, 2, 0, egr.F32),
    ]
    for call in range(2):                       # two calls in a row share the same built-in scratch
        for (N, T, m, n, r, flags, dt) in cases:
            bf16 = dt == egr.BF16
            W, X = workloads.linear_layer(20 + call, m, n, N * T, bf16=bf16)
            tdt = torch.bfloat16 if bf16 else torch.float32
            Xd = torch.from_numpy(X).cuda().to(tdt)
            Wd = torch.from_numpy(W).cuda().to(tdt)
            L = egr.Layer(n, m, N, T, r, layer_id=3, seed=100 + call, flags=flags, x_dtype=dt, w_dtype=dt, y_dtype=dt)
            Y_ref = torch.zeros((N * T, m), dtype=tdt, device="cuda")
            Y_new = torch.zeros_like(Y_ref)
            egr.egr_perturbed_linear(L, Xd, Wd, 0.05, Y_ref, ws)
            assert egr.egr_workspace_status(ws) == 0
            egr.egr_perturbed_linear_static(L, Xd, Wd, 0.05, Y_new)
            assert egr.egr_static_status() == 0
            torch.cuda.synchronize()
            tol = 1e-2 if bf16 else 1e-5
            assert _rel(Y_new.float().cpu().numpy(), Y_ref.float().cpu().numpy()) < tol
            assert torch.equal(Y_new, Y_ref)    # same kernels, same inputs: identical bits


@pytest.mark.gpu
def test_static_forward_refuses_problems_beyond_its_scratch():
    import torch
    import paper_2511_16652_b200 as egr
    egr.load_library()
    N, r = egr.STATIC_MAX_S_FLOATS // 4 + 1, 4            # one row too many
    L = egr.Layer(64, 64, N, 1, r, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16)
    X = torch.zeros((N, 64), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    Y = torch.full((N, 64), 5.0, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(egr.EgrError) as e:
        egr.egr_perturbed_linear_static(L, X, W, 0.1, Y)
    assert e.value.code == -7 and "scratch" in str(e.value)
    assert bool((Y == 5.0).all())                          # nothing was launched
    L_ok = egr.Layer(64, 64, N - 1, 1, r, x_dtype=egr.BF16, w_dtype=egr.BF16, y_dtype=egr.BF16)
    egr.egr_perturbed_linear_static(L_ok, X, W, 0.1, Y)    # exactly at the limit is accepted
    assert egr.egr_static_status() == 0


def test_static_entry_point_validates_on_the_host():
    import paper_2511_16652_b200 as egr
    from paper_2511_16652_b200 import build
    build.build()
    lib = egr.load_library()
    fake = ctypes.c_void_p(4096)
    L = egr.Layer(64, 64, 1 << 20, 1, 1)                   # 2^20 floats of s > 262144
    assert lib.egr_perturbed_linear_static(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, None) == -7
    assert lib.egr_perturbed_linear_static(None, fake, fake, ctypes.c_float(0.1), fake, None) == -1
    L = egr.Layer(64, 64, 32, 1, 3)                        # bad rank is still a bad argument
    assert lib.egr_perturbed_linear_static(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, None) == -1
    L = egr.Layer(64, 64, 1 << 20, 1, 3)                   # invalid and too large: the argument error wins
    assert lib.egr_perturbed_linear_static(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, None) == -1
    L = egr.Layer(64, 64, 1 << 20, 1, 1, ldx=68)           # misaligned pitch and too large
    assert lib.egr_perturbed_linear_static(ctypes.byref(L.c), fake, fake, ctypes.c_float(0.1), fake, None) == -2

"""ctypes binding of libegr.so: same names as the C ABI, argument marshalling only."""
from __future__ import annotations

import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(HERE, "libegr.so")

F32, BF16, I8 = 0, 1, 2
ANTITHETIC, NO_PERTURB = 1, 2
ACT_MASK, ACT_TANH, ACT_RELU, ACT_GELU = 12, 4, 8, 12     # forward only: element-wise function after the layer
SHAPE_NONE, SHAPE_CENTERED_RANK, SHAPE_ZSCORE, SHAPE_ANTITHETIC_SIGN = 0, 1, 2, 3
OP_PERTURBED_LINEAR, OP_ES_UPDATE, OP_FITNESS_SHAPE, OP_PERTURBED_LINEAR_I8, OP_ES_UPDATE_I8 = 0, 1, 2, 3, 4
OP_FITNESS_SHAPE_QUESTIONS = 5
OP_PERTURBED_LINEAR_LOGLIK = 10
OP_PERTURBED_LINEAR_Q8, OP_ES_GRADIENT, OP_ES_SCALE_GRADIENT, OP_ADAM_STEP_Q8 = 6, 7, 8, 9

EXPORTS = [
    "egr_perturbed_linear", "egr_es_update", "egr_fitness_shape",
    "egr_perturbed_linear_i8", "egr_es_update_i8", "egr_fitness_shape_i8",
    "egr_philox4x32_10", "egr_philox4x32_10_device", "egr_noise_materialize",
    "egr_workspace_bytes", "egr_workspace_status", "egr_strerror", "egr_version",
    "egr_perturbed_linear_static", "egr_static_status",
    "egr_i8lm_forward", "egr_i8lm_workspace_bytes", "egr_fitness_shape_questions",
    "egr_perturbed_linear_rows", "egr_perturbed_linear_loglik",
    "egr_q8_quantize", "egr_perturbed_linear_q8", "egr_es_gradient", "egr_es_scale_gradient",
    "egr_adam_step_q8", "egr_adam_step_bf16",
    "egr_fitness_pack3", "egr_fitness_unpack3", "egr_q8_expand",
    "egr_debug_bounded_wait",
]


class EgrError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {egr_strerror(code)} ({code})")


class _CLayer(ctypes.Structure):
    _fields_ = [
        ("d_in", ctypes.c_int32), ("d_out", ctypes.c_int32), ("n_members", ctypes.c_int32),
        ("rows_per_member", ctypes.c_int32), ("rank", ctypes.c_int32), ("layer_id", ctypes.c_uint32),
        ("seed", ctypes.c_uint64), ("flags", ctypes.c_uint32),
        ("x_dtype", ctypes.c_int32), ("w_dtype", ctypes.c_int32), ("y_dtype", ctypes.c_int32),
        ("ldx", ctypes.c_int64), ("ldw", ctypes.c_int64), ("ldy", ctypes.c_int64), ("member_base", ctypes.c_int32),
    ]


_lib = None


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libegr.so (built in-tree by ``paper_2511_16652_b200.build``).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2511_16652_b200.build` (nvcc, sm_100a); "
                           "there is no CPU fallback")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, u32, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32, ctypes.c_float, ctypes.c_size_t
    LP = ctypes.POINTER(_CLayer)
    lib.egr_perturbed_linear.argtypes = [LP, vp, vp, f32, vp, vp, sz, vp]
    lib.egr_es_update.argtypes = [LP, vp, vp, f32, vp, vp, vp, sz, vp]
    lib.egr_fitness_shape.argtypes = [vp, i32, i32, vp, vp, sz, vp]
    lib.egr_perturbed_linear_i8.argtypes = [LP, vp, vp, i32, i32, vp, u32, vp, vp, sz, vp]
    lib.egr_es_update_i8.argtypes = [LP, vp, vp, i32, vp, u32, vp, vp, sz, vp]
    lib.egr_fitness_shape_i8.argtypes = [vp, i32, vp, vp]
    lib.egr_philox4x32_10.argtypes = [ctypes.POINTER(u32), ctypes.POINTER(u32), ctypes.POINTER(u32)]
    lib.egr_philox4x32_10_device.argtypes = [vp, ctypes.POINTER(u32), ctypes.c_int64, vp, vp]
    lib.egr_noise_materialize.argtypes = [LP, i32, i32, i32, vp, vp]
    lib.egr_workspace_bytes.argtypes = [LP, i32]
    lib.egr_workspace_bytes.restype = sz
    lib.egr_workspace_status.argtypes = [vp, vp]
    lib.egr_perturbed_linear_static.argtypes = [LP, vp, vp, f32, vp, vp]
    lib.egr_static_status.argtypes = [vp]
    i64 = ctypes.c_int64
    lib.egr_q8_quantize.argtypes = [vp, i32, i32, i64, f32, vp, i64, vp, vp]
    lib.egr_perturbed_linear_q8.argtypes = [LP, vp, vp, vp, f32, f32, f32, vp, vp, sz, vp]
    lib.egr_q8_expand.argtypes = [vp, i32, i32, i64, vp, i64, vp]
    lib.egr_debug_bounded_wait.argtypes = [vp, sz, u32, vp]
    lib.egr_es_gradient.argtypes = [LP, vp, vp, vp, sz, vp]
    lib.egr_es_scale_gradient.argtypes = [LP, vp, vp, vp, sz, vp]
    lib.egr_adam_step_q8.argtypes = [vp, i64, i32, i32, vp, i64, vp, vp, i32, f32, f32, f32, f32, f32, vp, vp, sz, vp]
    lib.egr_adam_step_bf16.argtypes = [vp, i64, vp, vp, vp, i32, f32, f32, f32, f32, vp]
    lib.egr_fitness_pack3.argtypes = [vp, i64, vp, vp]
    lib.egr_fitness_unpack3.argtypes = [vp, i64, vp, vp]
    lib.egr_strerror.argtypes = [ctypes.c_int]
    lib.egr_strerror.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("egr_workspace_bytes", "egr_strerror", "egr_i8lm_workspace_bytes"):
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def _dtype_code(t) -> int:
    import torch
    return {torch.float32: F32, torch.bfloat16: BF16, torch.int8: I8}[t.dtype]


class Layer:
    """Python mirror of ``egr_layer``: one perturbed matrix W[d_out, d_in] and its population layout."""

    def __init__(self, d_in, d_out, n_members, rows_per_member=1, rank=1, layer_id=0, seed=0, flags=0,
                 x_dtype=BF16, w_dtype=BF16, y_dtype=BF16, ldx=None, ldw=None, ldy=None, member_base=0):
        self.c = _CLayer(d_in, d_out, n_members, rows_per_member, rank, layer_id, seed, flags,
                         x_dtype, w_dtype, y_dtype,
                         d_in if ldx is None else ldx, d_in if ldw is None else ldw, d_out if ldy is None else ldy,
                         member_base)

    def __getattr__(self, k):
        return getattr(self.__dict__["c"], k)

    def with_seed(self, seed):
        c = self.c
        return Layer(c.d_in, c.d_out, c.n_members, c.rows_per_member, c.rank, c.layer_id, seed, c.flags,
                     c.x_dtype, c.w_dtype, c.y_dtype, c.ldx, c.ldw, c.ldy, c.member_base)


class Workspace:
    """Caller-owned scratch: a torch uint8 buffer on the device, grown on demand."""

    def __init__(self, device="cuda"):
        self.device = device
        self.buf = None

    def ensure(self, nbytes: int):
        import torch
        if self.buf is None or self.buf.numel() < nbytes:
            self.buf = torch.empty(max(int(nbytes), 4096), dtype=torch.uint8, device=self.device)
        return self.buf

    def ptr(self):
        return self.buf.data_ptr()

    def nbytes(self):
        return self.buf.numel()


def _stream():
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _check(rc, where):
    if rc != 0:
        raise EgrError(rc, where)


def _ws(layer, op, ws: Workspace):
    need = egr_workspace_bytes(layer, op)
    ws.ensure(need)
    return ctypes.c_void_p(ws.ptr()), ctypes.c_size_t(ws.nbytes())


def egr_version() -> int:
    return load_library().egr_version()


def egr_strerror(code: int) -> str:
    try:
        return load_library().egr_strerror(code).decode()
    except Exception:
        return f"error {code}"


def egr_workspace_bytes(layer, op: int) -> int:
    lp = ctypes.byref(layer.c) if layer is not None else None
    return int(load_library().egr_workspace_bytes(lp, op))


def egr_workspace_status(ws: Workspace) -> int:
    return load_library().egr_workspace_status(ctypes.c_void_p(ws.ptr()), _stream())


def egr_philox4x32_10(ctr, key):
    c = (ctypes.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (ctypes.c_uint32 * 4)()
    _check(load_library().egr_philox4x32_10(c, k, o), "egr_philox4x32_10")
    return [int(x) for x in o]


def egr_philox4x32_10_device(ctr, key, out):
    k = (ctypes.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    _check(load_library().egr_philox4x32_10_device(_ptr(ctr), k, ctr.shape[0], _ptr(out), _stream()),
           "egr_philox4x32_10_device")
    return out


def egr_noise_materialize(layer: Layer, member: int, which: int, precise: bool, out):
    _check(load_library().egr_noise_materialize(ctypes.byref(layer.c), member, which, int(precise), _ptr(out),
                                                _stream()), "egr_noise_materialize")
    return out


def egr_perturbed_linear(layer: Layer, X, W, sigma: float, Y, ws: Workspace):
    wp, wn = _ws(layer, OP_PERTURBED_LINEAR, ws)
    _check(load_library().egr_perturbed_linear(ctypes.byref(layer.c), _ptr(X), _ptr(W), ctypes.c_float(sigma),
                                               _ptr(Y), wp, wn, _stream()), "egr_perturbed_linear")
    return Y


def egr_perturbed_linear_rows(layer: Layer, X, W, member_of_row, sigma: float, Y, ws: Workspace):
    """Forward with an explicit int32 row -> member map (ragged / interleaved populations)."""
    lib = load_library()
    lib.egr_perturbed_linear_rows.argtypes = [ctypes.POINTER(_CLayer), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                              ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                                              ctypes.c_void_p]
    wp, wn = _ws(layer, OP_PERTURBED_LINEAR, ws)
    _check(lib.egr_perturbed_linear_rows(ctypes.byref(layer.c), _ptr(X), _ptr(W), _ptr(member_of_row), ctypes.c_float(sigma),
                                         _ptr(Y), wp, wn, _stream()), "egr_perturbed_linear_rows")
    return Y


def egr_perturbed_linear_loglik(layer: Layer, X, W, sigma: float, targets, logp, ws: Workspace):
    """Perturbed vocabulary head ending in the log-likelihood of ``targets`` (int32 [R]); no logits are written."""
    lib = load_library()
    lib.egr_perturbed_linear_loglik.argtypes = [ctypes.POINTER(_CLayer), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float,
                                                ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
    wp, wn = _ws(layer, OP_PERTURBED_LINEAR_LOGLIK, ws)
    _check(lib.egr_perturbed_linear_loglik(ctypes.byref(layer.c), _ptr(X), _ptr(W), ctypes.c_float(sigma), _ptr(targets),
                                           _ptr(logp), wp, wn, _stream()), "egr_perturbed_linear_loglik")
    return logp


def egr_es_update(layer: Layer, W_master, shaped_fitness, alpha: float, ws: Workspace, W_shadow=None, dW_out=None):
    wp, wn = _ws(layer, OP_ES_UPDATE, ws)
    _check(load_library().egr_es_update(ctypes.byref(layer.c), _ptr(W_master), _ptr(shaped_fitness),
                                        ctypes.c_float(alpha), _ptr(W_shadow), _ptr(dW_out), wp, wn, _stream()),
           "egr_es_update")
    return W_master


def egr_fitness_shape(raw, mode: int, out, ws: Workspace):
    wp, wn = _ws(Layer(1, 1, raw.numel()), OP_FITNESS_SHAPE, ws)
    _check(load_library().egr_fitness_shape(_ptr(raw), raw.numel(), mode, _ptr(out), wp, wn, _stream()),
           "egr_fitness_shape")
    return out


def egr_fitness_shape_questions(S, out, ws: Workspace):
    """Per-question centred, globally scaled scores averaged over the questions; S is [N, Q] fp32."""
    N, Q = S.shape
    lib = load_library()
    lib.egr_fitness_shape_questions.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                                ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
    wp, wn = _ws(Layer(Q, 1, N), OP_FITNESS_SHAPE_QUESTIONS, ws)
    _check(lib.egr_fitness_shape_questions(_ptr(S), N, Q, _ptr(out), wp, wn, _stream()), "egr_fitness_shape_questions")
    return out


def egr_perturbed_linear_i8(layer: Layer, X, W, sigma_shift: int, out_shift: int, noise_table, Y, ws: Workspace):
    wp, wn = _ws(layer, OP_PERTURBED_LINEAR_I8, ws)
    log2 = noise_table.numel().bit_length() - 1
    assert 1 << log2 == noise_table.numel()
    _check(load_library().egr_perturbed_linear_i8(ctypes.byref(layer.c), _ptr(X), _ptr(W), sigma_shift, out_shift,
                                                  _ptr(noise_table), log2, _ptr(Y), wp, wn, _stream()),
           "egr_perturbed_linear_i8")
    return Y


def egr_es_update_i8(layer: Layer, W, F, threshold: int, noise_table, ws: Workspace, E_out=None):
    wp, wn = _ws(layer, OP_ES_UPDATE_I8, ws)
    log2 = noise_table.numel().bit_length() - 1
    assert 1 << log2 == noise_table.numel()
    _check(load_library().egr_es_update_i8(ctypes.byref(layer.c), _ptr(W), _ptr(F), threshold, _ptr(noise_table),
                                           log2, _ptr(E_out), wp, wn, _stream()), "egr_es_update_i8")
    return W


def egr_fitness_shape_i8(raw, out):
    _check(load_library().egr_fitness_shape_i8(_ptr(raw), raw.numel(), _ptr(out), _stream()),
           "egr_fitness_shape_i8")
    return out


def egr_debug_bounded_wait(ws: Workspace, limit_ms: int):
    """Runs the kernels' bounded wait on a barrier nothing completes; the status word of ``ws`` then holds the time-out."""
    ws.ensure(4096)
    _check(load_library().egr_debug_bounded_wait(ctypes.c_void_p(ws.ptr()), ctypes.c_size_t(ws.nbytes()), limit_ms, _stream()),
           "egr_debug_bounded_wait")


def egr_fitness_pack3(F, packed=None):
    """int8 pair signs in {-1,0,1} -> base-3 bytes, five values per byte."""
    import torch
    if packed is None:
        packed = torch.empty((F.numel() + 4) // 5, dtype=torch.uint8, device=F.device)
    _check(load_library().egr_fitness_pack3(_ptr(F), F.numel(), _ptr(packed), _stream()), "egr_fitness_pack3")
    return packed


def egr_fitness_unpack3(packed, count: int, F=None):
    import torch
    if F is None:
        F = torch.empty(count, dtype=torch.int8, device=packed.device)
    _check(load_library().egr_fitness_unpack3(_ptr(packed), count, _ptr(F), _stream()), "egr_fitness_unpack3")
    return F


STATIC_MAX_S_FLOATS = 262144


def egr_perturbed_linear_static(layer: Layer, X, W, sigma: float, Y):
    """Forward without a workspace: the scratch is a fixed array of about 1 MiB inside the library, for callers that
    cannot allocate device memory.  Needs N*T*r <= STATIC_MAX_S_FLOATS; calls on one device must not overlap."""
    _check(load_library().egr_perturbed_linear_static(ctypes.byref(layer.c), _ptr(X), _ptr(W), ctypes.c_float(sigma),
                                                      _ptr(Y), _stream()), "egr_perturbed_linear_static")
    return Y


def egr_static_status() -> int:
    return load_library().egr_static_status(_stream())


# ----------------------------------------------------------------------------------------------- integer LM
class _CI8LM(ctypes.Structure):
    _fields_ = [("D", ctypes.c_int32), ("n_layers", ctypes.c_int32), ("n_members", ctypes.c_int32),
                ("seed", ctypes.c_uint64), ("flags", ctypes.c_uint32), ("sigma_shift", ctypes.c_int32)] + \
               [(k, ctypes.c_void_p) for k in ("emb_t", "head", "ln_out", "ln1", "ln2", "Wf", "Uf", "Wh", "Uh", "bf", "bh",
                                               "mlp1", "mlp2", "lut_sigma", "lut_phi", "noise_table")] + \
               [("table_log2", ctypes.c_uint32)]


I8LM_MATRICES = ("Wf", "Uf", "Wh", "Uh", "mlp1", "mlp2")


def _i8lm_struct(params: dict, n_members: int, seed: int, flags: int, sigma_shift: int, noise_table):
    l, D = params["ln1"].shape
    log2 = noise_table.numel().bit_length() - 1
    assert 1 << log2 == noise_table.numel()
    ptrs = [params[k].data_ptr() for k in ("emb_t", "head", "ln_out", "ln1", "ln2", "Wf", "Uf", "Wh", "Uh", "bf", "bh",
                                           "mlp1", "mlp2", "lut_sigma", "lut_phi")]
    return _CI8LM(D, l, n_members, seed, flags, sigma_shift, *ptrs, noise_table.data_ptr(), log2)


def egr_i8lm_workspace_bytes(params: dict, n_members: int) -> int:
    lib = load_library()
    lib.egr_i8lm_workspace_bytes.restype = ctypes.c_size_t
    import torch
    dummy = torch.zeros(4, dtype=torch.int8, device=params["ln1"].device)
    c = _i8lm_struct(params, n_members, 0, 0, 8, dummy)
    return int(lib.egr_i8lm_workspace_bytes(ctypes.byref(c)))


def egr_i8lm_forward(params: dict, n_members: int, seed: int, flags: int, sigma_shift: int, noise_table,
                     tokens, member_seq, state, fitness, ws: Workspace):
    """Population forward of the integer recurrent LM.  ``params`` maps the field names of ``egr_i8lm`` to int8
    device tensors; ``state`` [l, N, D] and ``fitness`` [N] are updated in place."""
    lib = load_library()
    lib.egr_i8lm_forward.restype = ctypes.c_int
    lib.egr_i8lm_forward.argtypes = [ctypes.POINTER(_CI8LM), ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.c_size_t, ctypes.c_void_p]
    c = _i8lm_struct(params, n_members, seed, flags, sigma_shift, noise_table)
    need = egr_i8lm_workspace_bytes(params, n_members)
    ws.ensure(need)
    _check(lib.egr_i8lm_forward(ctypes.byref(c), _ptr(tokens), tokens.shape[0], tokens.shape[1], _ptr(member_seq),
                                _ptr(state), _ptr(fitness), ctypes.c_void_p(ws.ptr()), ctypes.c_size_t(ws.nbytes()),
                                _stream()), "egr_i8lm_forward")
    return fitness


# ----------------------------------------------------------------------------- per-channel int8 weights, discretised Adam
def egr_q8_quantize(W, eps: float, Q, scales):
    """W [m, n] fp32 -> Q [m, n] int8 codes and scales [m] bf16 (declared in include/egr_q8.h)."""
    m, n = W.shape
    _check(load_library().egr_q8_quantize(_ptr(W), m, n, W.stride(0), ctypes.c_float(eps), _ptr(Q), Q.stride(0),
                                          _ptr(scales), _stream()), "egr_q8_quantize")
    return Q, scales


def egr_q8_expand(Q, Q_bf16):
    """int8 codes -> bf16 (exact), for forwards that reuse one expansion (pass it with w_dtype = BF16)."""
    m, n = Q.shape
    _check(load_library().egr_q8_expand(_ptr(Q), m, n, Q.stride(0), _ptr(Q_bf16), Q_bf16.stride(0), _stream()), "egr_q8_expand")
    return Q_bf16


def egr_perturbed_linear_q8(layer: Layer, X, Q, scales, s_x: float, sigma: float, sigma_s: float, Y, ws: Workspace):
    wp, wn = _ws(layer, OP_PERTURBED_LINEAR_Q8, ws)
    _check(load_library().egr_perturbed_linear_q8(ctypes.byref(layer.c), _ptr(X), _ptr(Q), _ptr(scales), ctypes.c_float(s_x),
                                                  ctypes.c_float(sigma), ctypes.c_float(sigma_s), _ptr(Y), wp, wn, _stream()),
           "egr_perturbed_linear_q8")
    return Y


def egr_es_gradient(layer: Layer, shaped_fitness, G, ws: Workspace):
    wp, wn = _ws(layer, OP_ES_GRADIENT, ws)
    _check(load_library().egr_es_gradient(ctypes.byref(layer.c), _ptr(shaped_fitness), _ptr(G), wp, wn, _stream()),
           "egr_es_gradient")
    return G


def egr_es_scale_gradient(layer: Layer, shaped_fitness, g, ws: Workspace):
    wp, wn = _ws(layer, OP_ES_SCALE_GRADIENT, ws)
    _check(load_library().egr_es_scale_gradient(ctypes.byref(layer.c), _ptr(shaped_fitness), _ptr(g), wp, wn, _stream()),
           "egr_es_scale_gradient")
    return g


def egr_adam_step_q8(Q, G, mom1, mom2, t: int, lr: float, beta1: float, beta2: float, eps: float, tau: float,
                     ws: Workspace, n_changed=None):
    m, n = Q.shape
    layer = Layer(n, m, 1)
    wp, wn = _ws(layer, OP_ADAM_STEP_Q8, ws)
    _check(load_library().egr_adam_step_q8(_ptr(Q), Q.stride(0), m, n, _ptr(G), G.stride(0), _ptr(mom1), _ptr(mom2), t,
                                           ctypes.c_float(lr), ctypes.c_float(beta1), ctypes.c_float(beta2),
                                           ctypes.c_float(eps), ctypes.c_float(tau), _ptr(n_changed), wp, wn, _stream()),
           "egr_adam_step_q8")
    return Q


def egr_adam_step_bf16(param, g, mom1, mom2, t: int, lr: float, beta1: float, beta2: float, eps: float):
    _check(load_library().egr_adam_step_bf16(_ptr(param), param.numel(), _ptr(g), _ptr(mom1), _ptr(mom2), t,
                                             ctypes.c_float(lr), ctypes.c_float(beta1), ctypes.c_float(beta2),
                                             ctypes.c_float(eps), _stream()), "egr_adam_step_bf16")
    return param

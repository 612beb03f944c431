"""EGGROLL hot path on B200: thin Python binding over the C-ABI library ``libegr.so``.

Every function here only marshals arguments (torch tensors -> raw device pointers, current stream) and
calls the entry point of the same name declared in ``include/egr.h``; all arithmetic runs in the CUDA
kernels.  There is no CPU fallback: if the library is missing or no CUDA device is present, calls raise.
"""
from .api import (  # noqa: F401
    ANTITHETIC, NO_PERTURB, ACT_MASK, ACT_TANH, ACT_RELU, ACT_GELU, F32, BF16, I8,
    SHAPE_NONE, SHAPE_CENTERED_RANK, SHAPE_ZSCORE, SHAPE_ANTITHETIC_SIGN,
    OP_PERTURBED_LINEAR, OP_ES_UPDATE, OP_FITNESS_SHAPE, OP_PERTURBED_LINEAR_I8, OP_ES_UPDATE_I8,
    EgrError, Layer, Workspace,
    egr_perturbed_linear, egr_es_update, egr_fitness_shape,
    egr_perturbed_linear_i8, egr_es_update_i8, egr_fitness_shape_i8,
    egr_philox4x32_10, egr_philox4x32_10_device, egr_noise_materialize,
    egr_workspace_bytes, egr_workspace_status, egr_strerror, egr_version,
    library_path, load_library,
    egr_perturbed_linear_static, egr_static_status, STATIC_MAX_S_FLOATS,
    egr_i8lm_forward, egr_i8lm_workspace_bytes, I8LM_MATRICES, egr_fitness_shape_questions,
    egr_perturbed_linear_rows, egr_perturbed_linear_loglik, OP_PERTURBED_LINEAR_LOGLIK,
    OP_PERTURBED_LINEAR_Q8, OP_ES_GRADIENT, OP_ES_SCALE_GRADIENT, OP_ADAM_STEP_Q8,
    egr_q8_quantize, egr_perturbed_linear_q8, egr_es_gradient, egr_es_scale_gradient,
    egr_adam_step_q8, egr_adam_step_bf16, egr_fitness_pack3, egr_fitness_unpack3, egr_q8_expand, egr_debug_bounded_wait,
)

// C ABI of the per-channel int8 / discretised-Adam entry points: argument validation and dispatch only.
#include <cmath>

#include "../../include/egr_q8.h"
#include "egr_internal.h"

using namespace egr;

namespace {

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
bool rank_ok(int r) { return r == 1 || r == 2 || r == 4 || r == 8 || r == 16; }
bool have_device()
{
    int n = 0;
    return cudaGetDeviceCount(&n) == cudaSuccess && n > 0;
}

int check_population(const egr_layer *L)
{
    if (!L) return EGR_ERR_BADARG;
    if (L->d_in <= 0 || L->d_out <= 0 || L->n_members <= 0 || !rank_ok(L->rank)) return EGR_ERR_BADARG;
    if ((L->flags & EGR_ANTITHETIC) && (L->n_members & 1)) return EGR_ERR_BADARG;
    if (L->flags & ~(EGR_ANTITHETIC | EGR_NO_PERTURB)) return EGR_ERR_BADARG;
    if (L->member_base < 0 || ((L->flags & EGR_ANTITHETIC) && (L->member_base & 1))) return EGR_ERR_BADARG;
    return EGR_OK;
}

// pitch (elements) of the bf16 expansion of Q inside the forward workspace
int64_t expand_pitch(const egr_layer &L) { return ((int64_t)L.d_in + 63) / 64 * 64; }

egr_layer as_bf16_layer(const egr_layer &L)
{
    egr_layer B = L;
    B.w_dtype = EGR_BF16; B.x_dtype = EGR_BF16;
    B.ldw = expand_pitch(L);
    return B;
}

size_t forward_part_bytes(const egr_layer &L)
{
    const egr_layer B = as_bf16_layer(L);
    return align_up(gemm_sm100_workspace(B, EGR_OP_PERTURBED_LINEAR), 1024);
}

bool adam_scalars_ok(int32_t t, float lr, float b1, float b2, float eps)
{
    return t >= 1 && lr == lr && b1 >= 0.f && b1 < 1.f && b2 >= 0.f && b2 < 1.f && eps >= 0.f;
}

// step = lr / (1 - b1^t), rsb2 = 1 / sqrt(1 - b2^t): evaluated in double, rounded once to fp32
void adam_step_scalars(int32_t t, float lr, float b1, float b2, float &step, float &rsb2)
{
    step = (float)((double)lr / (1.0 - std::pow((double)b1, (double)t)));
    rsb2 = (float)(1.0 / std::sqrt(1.0 - std::pow((double)b2, (double)t)));
}

}  // namespace

namespace egr {

size_t q8_workspace_bytes(const egr_layer *L, int op)
{
    if (!L) return 0;
    switch (op) {
        case EGR_OP_PERTURBED_LINEAR_Q8:
            return forward_part_bytes(*L) + align_up((size_t)L->d_out * expand_pitch(*L) * 2, 256);
        case EGR_OP_ES_GRADIENT: {
            egr_layer B = *L;
            B.w_dtype = EGR_BF16;
            return gemm_sm100_workspace(B, EGR_OP_ES_UPDATE);
        }
        case EGR_OP_ES_SCALE_GRADIENT:
            return scale_gradient_ws(L->d_out, (L->flags & EGR_ANTITHETIC) ? L->n_members / 2 : L->n_members);
        case EGR_OP_ADAM_STEP_Q8:
            return adam_q8_ws(L->d_out, L->d_in);
    }
    return 0;
}

}  // namespace egr

extern "C" {

int egr_q8_quantize(const float *W, int32_t d_out, int32_t d_in, int64_t ldw, float eps, int8_t *Q, int64_t ldq,
                    void *scales_bf16, void *stream)
{
    if (!W || !Q || !scales_bf16 || d_out <= 0 || d_in <= 0 || ldw < d_in || ldq < d_in || !(eps > 0.f)) return EGR_ERR_BADARG;
    if (!aligned(W, 4) || !aligned(scales_bf16, 2)) return EGR_ERR_ALIGN;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_q8_quantize(W, d_out, d_in, ldw, eps, Q, ldq, scales_bf16, (cudaStream_t)stream);
}

int egr_q8_expand(const int8_t *Q, int32_t d_out, int32_t d_in, int64_t ldq, void *Q_bf16, int64_t ld_out, void *stream)
{
    if (!Q || !Q_bf16 || d_out <= 0 || d_in <= 0 || ldq < d_in || ld_out < ((int64_t)d_in + 15) / 16 * 16) return EGR_ERR_BADARG;
    if (!aligned(Q, 16) || !aligned(Q_bf16, 16) || (ldq & 15) || (ld_out & 15)) return EGR_ERR_ALIGN;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_q8_expand(Q, d_out, d_in, ldq, Q_bf16, ld_out, (cudaStream_t)stream);
}

int egr_perturbed_linear_q8(const egr_layer *L, const void *X, const int8_t *Q, const void *scales_bf16, float s_x,
                            float sigma, float sigma_s, void *Y, void *ws, size_t ws_bytes, void *stream)
{
    int rc = check_population(L);
    if (rc != EGR_OK) return rc;
    if (!X || !Q || !scales_bf16 || !Y || L->rows_per_member <= 0) return EGR_ERR_BADARG;
    if (L->ldx < L->d_in || L->ldw < L->d_in || L->ldy < L->d_out) return EGR_ERR_BADARG;
    const bool expanded = (L->w_dtype == EGR_BF16);                  // Q already holds the bf16 expansion
    if (L->x_dtype != EGR_BF16 || (L->w_dtype != EGR_I8 && !expanded) || (L->y_dtype != EGR_BF16 && L->y_dtype != EGR_F32))
        return EGR_ERR_UNSUPPORTED;
    if (!aligned(X, 16) || !aligned(Q, 16) || !aligned(Y, 16) || !aligned(scales_bf16, 2)) return EGR_ERR_ALIGN;
    if ((L->ldx & 7) || (L->ldw & (expanded ? 7 : 15))) return EGR_ERR_ALIGN;
    if (L->y_dtype == EGR_BF16 ? (L->ldy & 7) : (L->ldy & 3)) return EGR_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < q8_workspace_bytes(L, EGR_OP_PERTURBED_LINEAR_Q8)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    egr_layer B = as_bf16_layer(*L);
    const void *Qb = Q;
    if (expanded) {
        B.ldw = L->ldw;
    } else {
        void *dst = reinterpret_cast<unsigned char *>(ws) + forward_part_bytes(*L);
        rc = launch_q8_expand(Q, L->d_out, L->d_in, L->ldw, dst, B.ldw, st);
        if (rc != EGR_OK) return rc;
        Qb = dst;
    }
    const ColScales cs = {scales_bf16, s_x, sigma_s};
    const float coef = (float)((double)sigma / std::sqrt((double)L->rank));
    return launch_forward_bf16(B, X, Qb, coef, nullptr, Y, ws, ws_bytes, st, &cs);
}

int egr_es_gradient(const egr_layer *L, const float *fitness, float *G, void *ws, size_t ws_bytes, void *stream)
{
    int rc = check_population(L);
    if (rc != EGR_OK) return rc;
    if (!fitness || !G) return EGR_ERR_BADARG;
    if (!aligned(fitness, 4) || !aligned(G, 16)) return EGR_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < q8_workspace_bytes(L, EGR_OP_ES_GRADIENT)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    egr_layer B = *L;
    B.w_dtype = EGR_BF16;
    const float scale = (float)(1.0 / ((double)L->n_members * std::sqrt((double)L->rank)));
    return launch_update_bf16(B, nullptr, fitness, scale, nullptr, G, ws, ws_bytes, (cudaStream_t)stream);
}

int egr_es_scale_gradient(const egr_layer *L, const float *fitness, float *g, void *ws, size_t ws_bytes, void *stream)
{
    int rc = check_population(L);
    if (rc != EGR_OK) return rc;
    if (!fitness || !g) return EGR_ERR_BADARG;
    if (!aligned(fitness, 4) || !aligned(g, 4)) return EGR_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < q8_workspace_bytes(L, EGR_OP_ES_SCALE_GRADIENT)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_scale_gradient(*L, fitness, g, ws, (cudaStream_t)stream);
}

int egr_adam_step_q8(int8_t *Q, int64_t ldq, int32_t d_out, int32_t d_in, const float *G, int64_t ldg, void *mom1,
                     void *mom2, int32_t t, float lr, float beta1, float beta2, float eps, float tau, int64_t *n_changed,
                     void *ws, size_t ws_bytes, void *stream)
{
    if (!Q || !G || !mom1 || !mom2 || d_out <= 0 || d_in <= 0 || ldq < d_in || ldg < d_in) return EGR_ERR_BADARG;
    if (!adam_scalars_ok(t, lr, beta1, beta2, eps) || !(tau >= 0.f)) return EGR_ERR_BADARG;
    if ((d_in & 7) || (ldq & 7) || (ldg & 3)) return EGR_ERR_ALIGN;
    if (!aligned(Q, 8) || !aligned(G, 16) || !aligned(mom1, 16) || !aligned(mom2, 16)) return EGR_ERR_ALIGN;
    if (n_changed && !aligned(n_changed, 8)) return EGR_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < adam_q8_ws(d_out, d_in)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    float step, rsb2;
    adam_step_scalars(t, lr, beta1, beta2, step, rsb2);
    return launch_adam_step_q8(Q, ldq, d_out, d_in, G, ldg, mom1, mom2, beta1, beta2, eps, step, rsb2, tau, n_changed, ws,
                               (cudaStream_t)stream);
}

int egr_adam_step_bf16(void *param, int64_t len, const float *g, void *mom1, void *mom2, int32_t t, float lr, float beta1,
                       float beta2, float eps, void *stream)
{
    if (!param || !g || !mom1 || !mom2 || len <= 0) return EGR_ERR_BADARG;
    if (!adam_scalars_ok(t, lr, beta1, beta2, eps)) return EGR_ERR_BADARG;
    if (!aligned(param, 2) || !aligned(g, 4) || !aligned(mom1, 2) || !aligned(mom2, 2)) return EGR_ERR_ALIGN;
    if (!have_device()) return EGR_ERR_CUDA;
    float step, rsb2;
    adam_step_scalars(t, lr, beta1, beta2, step, rsb2);
    return launch_adam_step_bf16(param, len, g, mom1, mom2, beta1, beta2, eps, step, rsb2, (cudaStream_t)stream);
}

}  // extern "C"

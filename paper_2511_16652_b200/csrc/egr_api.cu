// C ABI: argument validation and dispatch.  No kernel lives here.
#include <climits>
#include <cmath>

#include "egr_device.cuh"
#include "egr_internal.h"

using namespace egr;

namespace {

bool rank_ok(int r) { return r == 1 || r == 2 || r == 4 || r == 8 || r == 16; }
bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// `forward`: the entry point applies the element-wise function bits; everybody else rejects them
int check_layer_common(const egr_layer *L, bool forward = false)
{
    if (!L) return EGR_ERR_BADARG;
    if (!forward && (L->flags & EGR_ACT_MASK)) return EGR_ERR_BADARG;
    if (L->d_in <= 0 || L->d_out <= 0 || L->n_members <= 0) return EGR_ERR_BADARG;
    if (!rank_ok(L->rank)) return EGR_ERR_BADARG;
    if ((L->flags & EGR_ANTITHETIC) && (L->n_members & 1)) return EGR_ERR_BADARG;
    if (L->flags & ~(EGR_ANTITHETIC | EGR_NO_PERTURB | EGR_ACT_MASK)) return EGR_ERR_BADARG;
    if (L->member_base < 0 || ((L->flags & EGR_ANTITHETIC) && (L->member_base & 1))) return EGR_ERR_BADARG;
    return EGR_OK;
}

bool have_device()
{
    int n = 0;
    return cudaGetDeviceCount(&n) == cudaSuccess && n > 0;
}

}  // namespace

// Everything egr_perturbed_linear checks about the layer and its three buffers, without touching a device.
int egr::perturbed_linear_check(const egr_layer *L, const void *X, const void *W, const int32_t *rowmap, const void *Y)
{
    if (!L) return EGR_ERR_BADARG;
    egr_layer chk = *L;
    if (rowmap) { chk.n_members += chk.n_members & 1; chk.member_base = 0; }   // with a row map, n_members only counts rows
    int rc = check_layer_common(&chk, true);
    if (rc != EGR_OK) return rc;
    if (!X || !W || !Y || L->rows_per_member <= 0) return EGR_ERR_BADARG;
    if (L->ldx < L->d_in || L->ldw < L->d_in || L->ldy < L->d_out) return EGR_ERR_BADARG;
    const bool f32 = (L->x_dtype == EGR_F32 && L->w_dtype == EGR_F32 && L->y_dtype == EGR_F32);
    const bool b16 = (L->x_dtype == EGR_BF16 && L->w_dtype == EGR_BF16 && (L->y_dtype == EGR_BF16 || L->y_dtype == EGR_F32));
    if (!f32 && !b16) return EGR_ERR_UNSUPPORTED;
    // the tensor-core kernel addresses rows with 32-bit tile coordinates and claims them through a 32-bit counter
    if (b16 && (int64_t)L->n_members * L->rows_per_member > (int64_t)INT32_MAX - 512) return EGR_ERR_UNSUPPORTED;
    if (!aligned(X, 16) || !aligned(W, 16) || !aligned(Y, 16)) return EGR_ERR_ALIGN;
    if (f32) {
        if ((L->ldx & 3) || (L->ldw & 3) || (L->ldy & 3)) return EGR_ERR_ALIGN;
    } else {
        if ((L->ldx & 7) || (L->ldw & 7)) return EGR_ERR_ALIGN;
        if (L->y_dtype == EGR_BF16 ? (L->ldy & 7) : (L->ldy & 3)) return EGR_ERR_ALIGN;
    }
    return EGR_OK;
}

extern "C" {

int egr_version(void) { return 100; }

const char *egr_strerror(int code)
{
    switch (code) {
        case EGR_OK:              return "ok";
        case EGR_ERR_BADARG:      return "bad argument";
        case EGR_ERR_ALIGN:       return "pointer or pitch violates the alignment rules";
        case EGR_ERR_UNSUPPORTED: return "unsupported dtype combination or size";
        case EGR_ERR_WORKSPACE:   return "workspace missing or too small";
        case EGR_ERR_CUDA:        return "CUDA runtime error (no device, or a launch failed)";
        case EGR_ERR_TIMEOUT:     return "a bounded device-side wait ran out";
        case EGR_ERR_CAPACITY:    return "problem exceeds the built-in scratch of the allocation-free entry point";
    }
    return "unknown error code";
}

int egr_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    if (!ctr || !key || !out) return EGR_ERR_BADARG;
    const uint4 r = philox4x32_10(ctr[0], ctr[1], ctr[2], ctr[3], key[0], key[1]);
    out[0] = r.x; out[1] = r.y; out[2] = r.z; out[3] = r.w;
    return EGR_OK;
}

int egr_philox4x32_10_device(const uint32_t *ctr, const uint32_t key[2], int64_t count, uint32_t *out, void *stream)
{
    if (!ctr || !key || !out || count < 0) return EGR_ERR_BADARG;
    if (!aligned(ctr, 16) || !aligned(out, 16)) return EGR_ERR_ALIGN;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_philox_device(ctr, key[0], key[1], count, out, (cudaStream_t)stream);
}

int egr_noise_materialize(const egr_layer *L, int32_t member, int32_t which, int32_t precise, float *out, void *stream)
{
    int rc = check_layer_common(L);
    if (rc != EGR_OK) return rc;
    if (!out || member < 0 || member >= L->n_members || (which != 0 && which != 1)) return EGR_ERR_BADARG;
    if (!have_device()) return EGR_ERR_CUDA;
    const uint32_t p = (L->flags & EGR_ANTITHETIC) ? (uint32_t)(member >> 1) : (uint32_t)member;
    return launch_noise_materialize(*L, p, which, precise, out, (cudaStream_t)stream);
}

size_t egr_workspace_bytes(const egr_layer *L, int32_t op)
{
    switch (op) {
        case EGR_OP_FITNESS_SHAPE:
            return fitness_shape_workspace(L ? L->n_members : 0);
        case EGR_OP_PERTURBED_LINEAR: {
            if (!L) return 0;
            const size_t R = (size_t)L->n_members * (size_t)L->rows_per_member;
            return kWsHeader + forward_ready_bytes(R) + align_up(R * (size_t)L->rank * sizeof(float), 256);
        }
        case EGR_OP_ES_UPDATE:
            if (!L) return 0;
            if (L->w_dtype == EGR_BF16) return gemm_sm100_workspace(*L, op);
            return kWsHeader;
        case EGR_OP_PERTURBED_LINEAR_I8: {
            if (!L) return 0;
            const size_t R = (size_t)L->n_members * (size_t)L->rows_per_member;
            return kWsHeader + align_up(R * 8, 256);
        }
        case EGR_OP_ES_UPDATE_I8:
            return L ? update_i8_workspace(*L) : 0;
        case EGR_OP_FITNESS_SHAPE_QUESTIONS:
            return L ? fitness_shape_questions_ws(L->d_in) : 0;
        case EGR_OP_PERTURBED_LINEAR_LOGLIK: {
            if (!L) return 0;
            const size_t R = (size_t)L->n_members * (size_t)L->rows_per_member;
            return kWsHeader + forward_ready_bytes(R) + align_up(R * (size_t)L->rank * sizeof(float), 256) + forward_loglik_extra_bytes(*L);
        }
    }
    return q8_workspace_bytes(L, op);      // operations of egr_q8.h, 0 for anything unknown
}

int egr_workspace_status(const void *ws, void *stream)
{
    if (!ws) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    int host[2] = {0, 0};
    if (cudaMemcpyAsync(host, ws, sizeof(host), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
        return EGR_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return EGR_ERR_CUDA;
    return host[0] == 0 ? EGR_OK : host[0];
}

static int perturbed_linear_impl(const egr_layer *L, const void *X, const void *W, const int32_t *rowmap, float sigma,
                                 void *Y, void *ws, size_t ws_bytes, void *stream)
{
    int rc = perturbed_linear_check(L, X, W, rowmap, Y);
    if (rc != EGR_OK) return rc;
    const bool f32 = (L->x_dtype == EGR_F32);
    if (!ws || !aligned(ws, 256) || ws_bytes < egr_workspace_bytes(L, EGR_OP_PERTURBED_LINEAR)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const float coef = (float)((double)sigma / std::sqrt((double)L->rank));
    if (f32) {
        const size_t R = (size_t)L->n_members * (size_t)L->rows_per_member;
        float *s = reinterpret_cast<float *>((unsigned char *)ws + kWsHeader + forward_ready_bytes(R));
        if (cudaMemsetAsync(ws, 0, 8, st) != cudaSuccess) return EGR_ERR_CUDA;
        if (!(L->flags & EGR_NO_PERTURB)) {
            rc = launch_skinny_xb(*L, X, rowmap, s, true, st);
            if (rc != EGR_OK) return rc;
        }
        return launch_forward_f32(*L, (const float *)X, (const float *)W, coef, s, rowmap, (float *)Y, st);
    }
    return launch_forward_bf16(*L, X, W, coef, rowmap, Y, ws, ws_bytes, st);
}

int egr_perturbed_linear(const egr_layer *L, const void *X, const void *W, float sigma, void *Y, void *ws,
                         size_t ws_bytes, void *stream)
{
    return perturbed_linear_impl(L, X, W, nullptr, sigma, Y, ws, ws_bytes, stream);
}

int egr_perturbed_linear_rows(const egr_layer *L, const void *X, const void *W, const int32_t *member_of_row, float sigma,
                              void *Y, void *ws, size_t ws_bytes, void *stream)
{
    if (!member_of_row) return EGR_ERR_BADARG;
    if (reinterpret_cast<uintptr_t>(member_of_row) & 3) return EGR_ERR_ALIGN;
    return perturbed_linear_impl(L, X, W, member_of_row, sigma, Y, ws, ws_bytes, stream);
}

int egr_perturbed_linear_loglik(const egr_layer *L, const void *X, const void *W, float sigma, const int32_t *targets,
                                float *logp, void *ws, size_t ws_bytes, void *stream)
{
    if (!L) return EGR_ERR_BADARG;
    if (L->flags & EGR_ACT_MASK) return EGR_ERR_BADARG;
    if (!targets || !logp) return EGR_ERR_BADARG;
    if (L->x_dtype != EGR_BF16 || L->w_dtype != EGR_BF16) return EGR_ERR_UNSUPPORTED;
    // the buffers' rules are those of the forward; there is no output matrix, so the check sees a stand-in for Y
    egr_layer chk = *L;
    chk.y_dtype = EGR_F32; chk.ldy = (chk.d_out + 3) / 4 * 4;
    int rc = perturbed_linear_check(&chk, X, W, nullptr, X);
    if (rc != EGR_OK) return rc;
    if ((reinterpret_cast<uintptr_t>(targets) & 3) || (reinterpret_cast<uintptr_t>(logp) & 3)) return EGR_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < egr_workspace_bytes(L, EGR_OP_PERTURBED_LINEAR_LOGLIK)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    const float coef = (float)((double)sigma / std::sqrt((double)L->rank));
    return launch_forward_bf16(*L, X, W, coef, nullptr, nullptr, ws, ws_bytes, (cudaStream_t)stream, nullptr, targets, logp);
}

int egr_es_update(const egr_layer *L, float *W_master, const float *fitness, float alpha, void *W_shadow_bf16,
                  float *dW_out, void *ws, size_t ws_bytes, void *stream)
{
    int rc = check_layer_common(L);
    if (rc != EGR_OK) return rc;
    if (!W_master || !fitness || L->ldw < L->d_in) return EGR_ERR_BADARG;
    if (L->w_dtype != EGR_F32 && L->w_dtype != EGR_BF16) return EGR_ERR_UNSUPPORTED;
    if (!aligned(W_master, 16) || !aligned(fitness, 4) || (L->ldw & 3)) return EGR_ERR_ALIGN;
    if (dW_out && !aligned(dW_out, 16)) return EGR_ERR_ALIGN;
    if (W_shadow_bf16 && (!aligned(W_shadow_bf16, 16) || (L->ldw & 7))) return EGR_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < egr_workspace_bytes(L, EGR_OP_ES_UPDATE)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const float scale = (float)((double)alpha / ((double)L->n_members * std::sqrt((double)L->rank)));
    if (L->w_dtype == EGR_F32) {
        if (W_shadow_bf16) return EGR_ERR_UNSUPPORTED;
        if (cudaMemsetAsync(ws, 0, 8, st) != cudaSuccess) return EGR_ERR_CUDA;
        return launch_update_f32(*L, W_master, fitness, scale, dW_out, st);
    }
    return launch_update_bf16(*L, W_master, fitness, scale, W_shadow_bf16, dW_out, ws, ws_bytes, st);
}

int egr_fitness_shape(const float *raw, int32_t N, int32_t mode, float *out, void *ws, size_t ws_bytes, void *stream)
{
    if (!raw || !out || N <= 0 || raw == out) return EGR_ERR_BADARG;
    if (mode < EGR_SHAPE_NONE || mode > EGR_SHAPE_ANTITHETIC_SIGN) return EGR_ERR_BADARG;
    if (mode == EGR_SHAPE_ANTITHETIC_SIGN && (N & 1)) return EGR_ERR_BADARG;
    if (!aligned(raw, 16) || !aligned(out, 16)) return EGR_ERR_ALIGN;
    egr_layer sized = {};
    sized.n_members = N;
    if (!ws || !aligned(ws, 256) || ws_bytes < egr_workspace_bytes(&sized, EGR_OP_FITNESS_SHAPE)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_fitness_shape(raw, N, mode, out, ws, (cudaStream_t)stream);
}

int egr_fitness_shape_questions(const float *S, int32_t N, int32_t Q, float *out, void *ws, size_t ws_bytes, void *stream)
{
    if (!S || !out || N <= 0 || Q <= 0) return EGR_ERR_BADARG;
    if (!aligned(S, 4) || !aligned(out, 4)) return EGR_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < fitness_shape_questions_ws(Q)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_fitness_shape_questions(S, N, Q, out, ws, (cudaStream_t)stream);
}

int egr_fitness_shape_i8(const int32_t *raw, int32_t N, int8_t *out, void *stream)
{
    if (!raw || !out || N <= 0 || (N & 1)) return EGR_ERR_BADARG;
    if (!aligned(raw, 16) || !aligned(out, 4)) return EGR_ERR_ALIGN;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_fitness_shape_i8(raw, N, out, (cudaStream_t)stream);
}

int egr_debug_bounded_wait(void *ws, size_t ws_bytes, uint32_t limit_ms, void *stream)
{
    if (!ws || !aligned(ws, 256) || ws_bytes < kWsHeader) return EGR_ERR_WORKSPACE;
    if (limit_ms == 0 || limit_ms > 1000) return EGR_ERR_BADARG;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_bounded_wait_probe(reinterpret_cast<int *>(ws), limit_ms, (cudaStream_t)stream);
}

int egr_fitness_pack3(const int8_t *F, int64_t count, uint8_t *packed, void *stream)
{
    if (count < 0 || (count > 0 && (!F || !packed))) return EGR_ERR_BADARG;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_pack3(F, count, packed, (cudaStream_t)stream);
}

int egr_fitness_unpack3(const uint8_t *packed, int64_t count, int8_t *F, void *stream)
{
    if (count < 0 || (count > 0 && (!F || !packed))) return EGR_ERR_BADARG;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_unpack3(packed, count, F, (cudaStream_t)stream);
}

int egr_perturbed_linear_i8(const egr_layer *L, const int8_t *X, const int8_t *W, int32_t sigma_shift, int32_t out_shift,
                            const int8_t *noise_table, uint32_t table_log2, int8_t *Y, void *ws, size_t ws_bytes,
                            void *stream)
{
    int rc = check_layer_common(L);
    if (rc != EGR_OK) return rc;
    if (!X || !W || !Y || !noise_table || L->rows_per_member <= 0 || L->rank != 1) return EGR_ERR_BADARG;
    if (sigma_shift < 0 || sigma_shift > 31 || out_shift < 0 || out_shift > 31 || table_log2 < 2 || table_log2 > 31)
        return EGR_ERR_BADARG;
    if (L->ldx < L->d_in || L->ldw < L->d_in || L->ldy < L->d_out) return EGR_ERR_BADARG;
    if (L->x_dtype != EGR_I8 || L->w_dtype != EGR_I8 || L->y_dtype != EGR_I8) return EGR_ERR_UNSUPPORTED;
    if ((L->d_in & 3) || (L->ldx & 3) || (L->ldw & 3) || !aligned(X, 4) || !aligned(W, 4)) return EGR_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < egr_workspace_bytes(L, EGR_OP_PERTURBED_LINEAR_I8)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_forward_i8(*L, X, W, sigma_shift, out_shift, noise_table, table_log2, Y, ws, (cudaStream_t)stream);
}

int egr_es_update_i8(const egr_layer *L, int8_t *W, const int8_t *F, int32_t threshold, const int8_t *noise_table,
                     uint32_t table_log2, int32_t *E_out, void *ws, size_t ws_bytes, void *stream)
{
    int rc = check_layer_common(L);
    if (rc != EGR_OK) return rc;
    if (!W || !F || !noise_table || L->rank != 1 || L->ldw < L->d_in) return EGR_ERR_BADARG;
    if (table_log2 < 2 || table_log2 > 31) return EGR_ERR_BADARG;
    if (L->w_dtype != EGR_I8) return EGR_ERR_UNSUPPORTED;
    if (E_out && !aligned(E_out, 4)) return EGR_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < egr_workspace_bytes(L, EGR_OP_ES_UPDATE_I8)) return EGR_ERR_WORKSPACE;
    if (!have_device()) return EGR_ERR_CUDA;
    return launch_update_i8(*L, W, F, threshold, noise_table, table_log2, E_out, ws, (cudaStream_t)stream);
}

}  // extern "C"

/*
 * egr_q8.h -- C ABI for EGGROLL on per-channel-scaled int8 weights with a discretised Adam update
 * (appendix "Fine-tuning of Integer Quantised Models": "Quantisation Procedure" and "Integrating
 * integer-quantised EGGROLL with Adam").  NVIDIA B200 (sm_100a) only; conventions as in egr.h: every pointer
 * is a DEVICE pointer unless stated, nothing is allocated or freed, `stream` is a cudaStream_t passed as void *,
 * the return value is EGR_OK or a negative EGR_ERR_* code, argument errors are detected before any launch.
 *
 * A matrix parameter is (Q, s, s_x): Q [d_out][ldq] int8 codes in [-127, 127], s [d_out] bf16 channel scales,
 * s_x one input scale.  Layout note: the paper writes W as d_in x d_out with one scale per output channel; here
 * a row of Q is an output channel, as for W in egr.h.
 *
 * Readings of what the appendix leaves open:
 *   - round() is round-half-to-even and uses the STORED (bf16) scale;
 *   - the scales multiply the accumulated sum, in fp32: y_j = s_x s_j (sum_l x_l Q_jl + low-rank term);
 *   - "explicit scale perturbations" are additive Gaussian noise with deviation sigma_s, mirrored inside an
 *     antithetic pair: member i sees s_j + sign_i sigma_s e_p[j] and s_x + sign_i sigma_s e_p[d_out], where e_p
 *     is the noise factor with tag 3 (d_out + 1 elements, rank 1) of the member's noise index p;
 *   - gradient estimates carry no step size: G = (1/(N sqrt r)) sum_p g_p A_p B_p^T for Q and
 *     g[j] = (1/N) sum_p g_p e_p[j] for the scales (g_p as in egr_es_update);
 *   - Adam is the textbook rule with bias correction, epsilon outside the square root, ASCENDING the fitness;
 *     its arithmetic is fp32 with one rounding per operation in the order given below, moments stored in bf16.
 */
#ifndef EGR_Q8_H_
#define EGR_Q8_H_

#include "egr.h"

#ifdef __cplusplus
extern "C" {
#endif

/* additional operation ids for egr_workspace_bytes() */
#define EGR_OP_PERTURBED_LINEAR_Q8   6   /* reads d_in, d_out, n_members, rows_per_member, rank, ldw          */
#define EGR_OP_ES_GRADIENT           7   /* as EGR_OP_ES_UPDATE with w_dtype = EGR_BF16                        */
#define EGR_OP_ES_SCALE_GRADIENT     8   /* reads d_out, n_members, flags                                      */
#define EGR_OP_ADAM_STEP_Q8          9   /* reads d_out, d_in                                                  */

/*
 * "Quantisation Procedure": symmetric per-channel absmax quantisation,
 *   s_i  = bf16( max( max_j |W[i][j]| / 127, eps ) )            (fp32 division, then one rounding to bf16)
 *   Q_ij = clip( rint( W[i][j] / s_i ), -127, 127 )             (fp32 division by the stored scale)
 * W [d_out][ldw] fp32 in, Q [d_out][ldq] int8 out, scales_bf16 [d_out] out.  Bit-exact by construction.
 */
int egr_q8_quantize(const float *W, int32_t d_out, int32_t d_in, int64_t ldw, float eps,
                    int8_t *Q, int64_t ldq, void *scales_bf16, void *stream);

/*
 * The codes as bf16 (exact): Q [d_out][ldq] int8 -> Q_bf16 [d_out][ld_out] bf16.  The forward below does this itself on
 * every call; a caller that runs many forwards between two updates can expand once and pass the result instead.
 * ldq a multiple of 16 with Q 16-byte aligned; ld_out a multiple of 16 elements, >= d_in rounded up to 16, Q_bf16
 * 16-byte aligned.
 */
int egr_q8_expand(const int8_t *Q, int32_t d_out, int32_t d_in, int64_t ldq, void *Q_bf16, int64_t ld_out, void *stream);

/*
 * Forward through a quantised matrix under the member's low-rank perturbation of Q and (sigma_s != 0) its
 * perturbation of the scales:
 *   Y[rho][j] = (s_x + sign sigma_s e_p[d_out]) (s_j + sign sigma_s e_p[j])
 *               ( sum_l X[rho][l] Q[j][l] + sign (sigma / sqrt r) sum_k (sum_l X[rho][l] B_p[l][k]) A_p[j][k] )
 * The int8 codes are exact in bf16, so the dense product runs on the bf16 tensor cores (fp32 accumulation) from
 * a bf16 expansion of Q that the call writes into the workspace; the scales are applied in the epilogue.
 * layer: x_dtype = EGR_BF16, w_dtype = EGR_I8, y_dtype = EGR_BF16 or EGR_F32; ldw = pitch of Q in bytes, a multiple
 * of 16, Q 16-byte aligned; X, Y and their pitches as in egr_perturbed_linear; EGR_NO_PERTURB switches off both
 * perturbations.  scales_bf16 [d_out] in, 2-byte aligned.  ws: egr_workspace_bytes(layer, EGR_OP_PERTURBED_LINEAR_Q8).
 * With w_dtype = EGR_BF16 the argument Q is taken to be the expansion written by egr_q8_expand (bf16, pitch ldw in
 * elements, a multiple of 8) and is used as it is.
 */
int egr_perturbed_linear_q8(const egr_layer *layer, const void *X, const int8_t *Q, const void *scales_bf16,
                            float s_x, float sigma, float sigma_s, void *Y, void *ws, size_t ws_bytes, void *stream);

/*
 * "ES gradients", matrix pathway: G = (1 / (N sqrt r)) sum_p g_p A_p B_p^T (the boxed update without the step
 * size), factors rounded to bf16 and contracted on the tensor cores as in egr_es_update with EGR_BF16.
 * G [d_out][d_in] fp32 dense, out, 16-byte aligned.  layer->w_dtype is ignored.
 */
int egr_es_gradient(const egr_layer *layer, const float *shaped_fitness, float *G,
                    void *ws, size_t ws_bytes, void *stream);

/*
 * "ES gradients", scale pathway: g[j] = (1/N) sum_p g_p e_p[j] for j = 0 .. d_out (entry d_out belongs to s_x).
 * g [d_out + 1] fp32 out.  Deterministic (fixed reduction order).
 */
int egr_es_scale_gradient(const egr_layer *layer, const float *shaped_fitness, float *g,
                          void *ws, size_t ws_bytes, void *stream);

/*
 * "Adam updates for int8 tensors (discretised)".  Per element, fp32, one rounding per operation:
 *   m' = b1*m + (1-b1)*g          v' = b2*v + (1-b2)*(g*g)
 *   u  = bf16( (step * m') / (sqrt(v') * rsb2 + eps) )                       m, v <- bf16(m'), bf16(v')
 *   step = lr / (1-b1^t), rsb2 = 1 / sqrt(1-b2^t), each evaluated in double and rounded once to fp32
 * then over the whole tensor (mean and population deviation of u accumulated in fp64, rounded once to fp32)
 *   Delta = sign(u - mu) * [ |u - mu| >= tau * (sigma_u + 1e-8) ],   Q <- clip(Q + Delta, -127, 127).
 * Q [d_out][ldq] int8 in/out; G [d_out][ldg] fp32 in; mom1_bf16, mom2_bf16 [d_out][d_in] bf16 dense in/out;
 * t >= 1 is the step count; n_changed (nullable) receives the number of entries of Q that moved (int64).
 * d_in a multiple of 8; Q 8-byte aligned with ldq a multiple of 8; G 16-byte aligned with ldg a multiple of 4;
 * moments 16-byte aligned.  ws: egr_workspace_bytes(layer, EGR_OP_ADAM_STEP_Q8) (holds u).
 * Bit-exact by construction for identical inputs.
 */
int egr_adam_step_q8(int8_t *Q, int64_t ldq, int32_t d_out, int32_t d_in, const float *G, int64_t ldg,
                     void *mom1_bf16, void *mom2_bf16, int32_t t, float lr, float beta1, float beta2, float eps,
                     float tau, int64_t *n_changed, void *ws, size_t ws_bytes, void *stream);

/*
 * Adam on a bf16 floating-point leaf (the scales): same proposal u, then param <- bf16(param + u).
 * param_bf16, mom1_bf16, mom2_bf16 [len] bf16 in/out; g [len] fp32 in.
 */
int egr_adam_step_bf16(void *param_bf16, int64_t len, const float *g, void *mom1_bf16, void *mom2_bf16,
                       int32_t t, float lr, float beta1, float beta2, float eps, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* EGR_Q8_H_ */

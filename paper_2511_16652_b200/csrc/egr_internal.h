// Host-side declarations of the kernel launchers behind the C ABI.  Every launcher enqueues on `stream`
// and returns a cudaError_t-free int: EGR_OK or EGR_ERR_*.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/egr.h"

namespace egr {

// Workspace layout: [0,256) status block (word 0 = status code, word 1 = detail), then op-specific scratch.
constexpr size_t kWsHeader = 256;

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline int cuda_ok(cudaError_t e) { return e == cudaSuccess ? EGR_OK : EGR_ERR_CUDA; }

// ---- argument rules of egr_perturbed_linear (layer, buffers), checked on the host only
int perturbed_linear_check(const egr_layer *L, const void *X, const void *W, const int32_t *rowmap, const void *Y);

// ---- noise / debug
int launch_philox_device(const uint32_t *ctr, uint32_t k0, uint32_t k1, int64_t count, uint32_t *out,
                         cudaStream_t st);
int launch_noise_materialize(const egr_layer &L, uint32_t p, int which, int precise, float *out, cudaStream_t st);

// ---- skinny reduction s[rho][k] = sum_l X[rho][l] B_p[l][k]  (fp32 out, dense [R][r])
int launch_skinny_xb(const egr_layer &L, const void *X, const int32_t *rowmap, float *s, bool precise, cudaStream_t st);

// ---- fp32 path
int launch_forward_f32(const egr_layer &L, const float *X, const float *W, float coef, const float *s,
                       const int32_t *rowmap, float *Y, cudaStream_t st);
int launch_update_f32(const egr_layer &L, float *W, const float *fitness, float scale, float *dW_out,
                      cudaStream_t st);

// ---- bf16 tensor-core path (tcgen05 + TMA + TMEM)
size_t gemm_sm100_workspace(const egr_layer &L, int op);
size_t forward_ready_bytes(size_t rows);
// per-column scales of a quantised matrix applied in the forward epilogue (scale noise with deviation sigma_s)
struct ColScales { const void *scales_bf16; float s_x; float sigma_s; };
// targets != nullptr: no output matrix; logp [R] receives the log-likelihood of each row's target column
int launch_forward_bf16(const egr_layer &L, const void *X, const void *W, float coef, const int32_t *rowmap, void *Y,
                        void *ws, size_t ws_bytes, cudaStream_t st, const ColScales *cs = nullptr,
                        const int32_t *targets = nullptr, float *logp = nullptr);
size_t forward_loglik_extra_bytes(const egr_layer &L);
// W_master == nullptr: only dW_out is written (gradient estimate)
int launch_update_bf16(const egr_layer &L, float *W_master, const float *fitness, float scale,
                       void *W_shadow, float *dW_out, void *ws, size_t ws_bytes, cudaStream_t st);

// the kernels' bounded wait on a barrier that is never completed (exercises the time-out path; returns normally)
int launch_bounded_wait_probe(int *status, uint32_t limit_ms, cudaStream_t st);

// ---- shaping
size_t fitness_shape_workspace(int N);
int launch_fitness_shape(const float *raw, int N, int mode, float *out, void *ws, cudaStream_t st);
int launch_fitness_shape_i8(const int32_t *raw, int N, int8_t *out, cudaStream_t st);
int launch_fitness_shape_questions(const float *S, int N, int Q, float *out, void *ws, cudaStream_t st);
size_t fitness_shape_questions_ws(int Q);
int launch_pack3(const int8_t *F, int64_t count, uint8_t *packed, cudaStream_t st);
int launch_unpack3(const uint8_t *packed, int64_t count, int8_t *F, cudaStream_t st);

// ---- integer path
int launch_forward_i8(const egr_layer &L, const int8_t *X, const int8_t *W, int sigma_shift, int out_shift,
                      const int8_t *table, uint32_t table_log2, int8_t *Y, void *ws, cudaStream_t st);
int launch_update_i8(const egr_layer &L, int8_t *W, const int8_t *F, int32_t threshold, const int8_t *table,
                     uint32_t table_log2, int32_t *E_out, void *ws, cudaStream_t st);

size_t update_i8_workspace(const egr_layer &L);
// ---- int8 tensor-core path (tcgen05 kind::i8)
// E = At Bt^T over p_pad noise indices (At [d_out][p_pad], Bt [d_in][p_pad], K-major int8), then the one-bin move of W
int launch_update_i8_tc(const egr_layer &L, const int8_t *At, const int8_t *Bt, int64_t p_pad, int8_t *W, int32_t threshold,
                        int32_t *E_out, int *status, cudaStream_t st);
bool i8_tc_eligible(const void *X, int64_t ldx, const void *W, int64_t ldw);
int launch_forward_i8_tc(const egr_layer &L, const int8_t *X, const int8_t *W, int sigma_shift, int out_shift,
                         const int8_t *table, uint32_t table_log2, int8_t *Y, const int2 *aux, int *status, cudaStream_t st);

// one fused step of the width-256 recurrent LM; mode: 0 pm, 1 gate f, 2 gate h (+LN), 3 mlp2 (+residual, LN), 4 head
struct I8LmStep {
    int64_t rows; int cols;
    const int8_t *X0, *W0; int K0; uint32_t layer_id0;
    const int8_t *X1, *W1; int K1; uint32_t layer_id1;       // second GEMM of the gate modes (X1 == nullptr otherwise)
    uint64_t seed; uint32_t flags; int sigma_shift;
    const int8_t *table; uint32_t table_log2;
    int8_t *Y;                                               // mode 0 output [rows][cols]
    const int8_t *bias, *lut, *ln_w;
    int8_t *s, *y, *x, *f, *fh;
    const uint8_t *tokens; const int32_t *member_seq; int seq_len, pos; int32_t *fitness;
    const int *exp2_tab, *frac_tab; int ln_shift;
    int *status;
};
// a step is prepared once (tensor maps, arguments) into lm_plan_bytes() of host memory and launched per position
size_t lm_plan_bytes();
int lm_plan_build(int mode, const I8LmStep &q, void *plan_mem);
int lm_plan_launch(const void *plan_mem, int pos, cudaStream_t st);

// the width-256 recurrent LM over all positions in one launch (each CTA pair walks the sequence for its own rows)
struct I8LmSeq {
    int64_t rows; int n_layers; uint64_t seed; uint32_t flags; int sigma_shift;
    const int8_t *table; uint32_t table_log2;
    int8_t *x, *y, *f, *fh, *h1, *state;                        // work buffers [rows][256] (h1: [rows][1024]); state [n_layers][rows][256]
    const int8_t *Wf, *Uf, *Wh, *Uh, *mlp1, *mlp2, *head;        // stacked per layer as in egr_i8lm
    const int8_t *bf, *bh, *ln1, *ln2, *ln_out, *lut_sigma, *lut_phi, *emb_rows;
    const uint8_t *tokens; const int32_t *member_seq; int seq_len; int32_t *fitness;
    const int *exp2_tab, *frac_tab; int ln_shift;
    int *status;
};
int launch_lm_seq(const I8LmSeq &q, cudaStream_t st);

// ---- per-channel int8 weights with discretised Adam
size_t q8_workspace_bytes(const egr_layer *L, int op);
int launch_q8_quantize(const float *W, int m, int n, int64_t ldw, float eps, int8_t *Q, int64_t ldq, void *scales, cudaStream_t st);
int launch_q8_expand(const int8_t *Q, int m, int n, int64_t ldq, void *out_bf16, int64_t ldo, cudaStream_t st);
size_t scale_gradient_ws(int d_out, int64_t P);
int launch_scale_gradient(const egr_layer &L, const float *fitness, float *g, void *ws, cudaStream_t st);
size_t adam_q8_ws(int m, int n);
int launch_adam_step_q8(int8_t *Q, int64_t ldq, int m, int n, const float *G, int64_t ldg, void *mom1, void *mom2,
                        float b1, float b2, float eps, float step, float rsb2, float tau, int64_t *n_changed,
                        void *ws, cudaStream_t st);
int launch_adam_step_bf16(void *param, int64_t len, const float *g, void *mom1, void *mom2, float b1, float b2,
                          float eps, float step, float rsb2, cudaStream_t st);

}  // namespace egr

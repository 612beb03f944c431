/*
 * egr_i8lm.h -- population forward of the integer-only recurrent byte-level LM under EGGROLL perturbations.
 *
 * The model is the one of the paper's appendix "EGG Architecture" (Algorithm "EGG forward pass"): embedding,
 * n_layers x [LN, GRU, saturating residual, LN, MLP, saturating residual], LN, head, with every weight and
 * activation in int8 (values -127..127), int32 accumulation, and the integer log-likelihood of the appendix's
 * "Fitness Calculation in Integer Types".  Every matrix and the embedding are perturbed per population member
 * with the rank-1 integer perturbation of "Adding EGGROLL Perturbations" (see egr_perturbed_linear_i8 in egr.h
 * for the arithmetic of one perturbed matmul; out_shift = 4 + log4(d_in)).
 *
 * Layer ids of the perturbed matrices: 16*layer + {0: Wf, 1: Uf, 2: Wh, 3: Uh, 4: mlp1, 5: mlp2}, embedding 1000,
 * head 1001.  Vectors (layer-norm weights, biases) are not perturbed.
 *
 * Per position t -> t' (next byte), per member:
 *   y      = sat127(emb[:, t] + ((sign B_p[t] A_p[j]) >> sigma_shift))          embedding: u.B becomes B[t]
 *   LN(w,u)= sat127(trunc((u_j w_j) / max(1, sat127(sum|u| >> 2d))))            D = 4^d
 *   f      = lut_sigma[sat127(pm(x,Wf) + pm(s,Uf) + bf)],  fh = sat127(((f+127) s) >> 8)
 *   hh     = lut_phi[sat127(pm(x,Wh) + pm(fh,Uh) + bh)],   h  = sat127(s + sat127(((f+127)(hh - s)) >> 8))
 *   s <- h,  y <- sat127(h + y),  y <- sat127(pm(pm(LN(ln2,y), mlp1), mlp2) + y)
 *   logits = pm(LN(ln_out, y), head);  z = logits + 128;  fitness += z[t'] - LOG2(sum_v EXP2[z_v])
 * with EXP2[i] = round(16 2^(i/16)) and LOG2(S) = 16 (e - 4) + round(16 log2(1 + mant/256)), e the position of
 * the leading one of S and mant the 8 bits below it.
 *
 * All pointers are device pointers owned by the caller; nothing is allocated; work is enqueued on `stream`.
 */
#ifndef EGR_I8LM_H_
#define EGR_I8LM_H_

#include "egr.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct egr_i8lm {
    int32_t  D;               /* hidden width, a power of 4, multiple of 16 (256 in the paper)                 */
    int32_t  n_layers;
    int32_t  n_members;       /* N                                                                             */
    uint64_t seed;
    uint32_t flags;           /* EGR_ANTITHETIC                                                                */
    int32_t  sigma_shift;     /* 4 + sigma_hat                                                                 */
    const int8_t *emb_t;      /* [D][256]   column t = embedding of byte t (W[m][n] orientation, m = D)        */
    const int8_t *head;       /* [256][D]                                                                      */
    const int8_t *ln_out;     /* [D]                                                                           */
    const int8_t *ln1, *ln2;  /* [n_layers][D]                                                                 */
    const int8_t *Wf, *Uf, *Wh, *Uh;   /* [n_layers][D][D]                                                     */
    const int8_t *bf, *bh;    /* [n_layers][D]                                                                 */
    const int8_t *mlp1;       /* [n_layers][4D][D]                                                             */
    const int8_t *mlp2;       /* [n_layers][D][4D]                                                             */
    const int8_t *lut_sigma;  /* [256] gate non-linearity, indexed by value + 128 (identity in the paper)      */
    const int8_t *lut_phi;    /* [256]                                                                         */
    const int8_t *noise_table;
    uint32_t table_log2;
} egr_i8lm;

/*
 * Runs positions 0 .. seq_len-2 of every member's sequence (member i reads tokens[member_seq[i]]).
 *   tokens      [n_seq][seq_len] uint8
 *   member_seq  [N] int32, values in [0, n_seq)
 *   state       [n_layers][N][D] int8, in-out: the recurrent state carried across calls (zero it to start)
 *   fitness     [N] int32, in-out: the log-likelihood sum is ADDED (zero it to start)
 *   ws          egr_i8lm_workspace_bytes(model) bytes, 256-byte aligned
 * Returns EGR_OK or a negative EGR_ERR_* code.
 * The call only enqueues memsets and kernel launches on `stream` (at D = 256 and up to eight layers one launch for the
 * whole sequence, each CTA pair walking all positions for its own 256 members; 18 launches per position beyond).  After one
 * ordinary call on the device (which sets the kernels' attributes) it can be recorded by stream capture and the
 * whole pass replayed as a CUDA graph, which removes the per-launch host work.
 */
int egr_i8lm_forward(const egr_i8lm *model, const uint8_t *tokens, int32_t n_seq, int32_t seq_len,
                     const int32_t *member_seq, int8_t *state, int32_t *fitness,
                     void *ws, size_t ws_bytes, void *stream);

size_t egr_i8lm_workspace_bytes(const egr_i8lm *model);

#ifdef __cplusplus
}
#endif
#endif /* EGR_I8LM_H_ */

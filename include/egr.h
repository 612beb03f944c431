/*
 * egr.h -- C ABI of the EGGROLL hot path for NVIDIA B200 (sm_100a).
 *
 * EGGROLL ("Evolution Strategies at the Hyperscale") perturbs every weight matrix W[m x n] of a model
 * with a per-member low-rank matrix E_i = A_i B_i^T / sqrt(r) (Algorithm 1), evaluates the population,
 * and moves W along the fitness-weighted sum of the E_i (boxed "EGGROLL UPDATE" equation).  This library
 * implements exactly that path and nothing else:
 *
 *   egr_perturbed_linear      y_i = x_i W^T + (sigma/sqrt r) (x_i B_i) A_i^T            Section 4.2
 *   egr_fitness_shape         raw fitness -> centred ranks / z-scores / pair signs       HFT appendix; integer appendix
 *   egr_es_update             W += (alpha/N) sum_i f_i E_i as one contraction over N*r   boxed update; Section 4.2
 *   egr_*_i8                  the integer-only variants                                  "EGG Pretraining with Integer EGGROLL"
 *
 * The factors A_i (m x r) and B_i (n x r) are never read from memory: they are rebuilt inside the kernels
 * from a counter-based generator ("reconstruct noise on demand", Introduction; Algorithm 1 "reconstruct
 * E_j from the seeds").
 *
 * NOISE DEFINITION (shared by every entry point)
 *   generator  Philox4x32-10, key = (seed & 0xffffffff, seed >> 32), counter = (q, p, layer_id, tag)
 *   p          noise index of member i: i >> 1 with EGR_ANTITHETIC (members 2p and 2p+1 share the noise
 *              with signs +,-), else i
 *   tag        0: factor A (output side, m x r), 1: factor B (input side, n x r), 2: integer table offsets
 *   element    entry (row j, rank column k) of a factor has flat index e = j*r + k, block q = e >> 2,
 *              lane e & 3
 *   normal     words (x0,x1) -> lanes 0,1 and (x2,x3) -> lanes 2,3 by Box-Muller:
 *              u1 = ((xa >> 9) + 1) 2^-23, u2 = (xb >> 9) 2^-23,
 *              even lane sqrt(-2 ln u1) cos(2 pi u2), odd lane sqrt(-2 ln u1) sin(2 pi u2), in fp32
 *
 * CONVENTIONS
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller.  The library
 *     keeps no reference after the call's work has finished on `stream`.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = default stream) and return
 *     without synchronising.  Nothing is allocated: scratch comes from the caller's workspace `ws` of
 *     `ws_bytes` bytes (256-byte aligned), sized by egr_workspace_bytes().
 *   - Matrices are row-major; ld* are row pitches in elements.
 *   - Return value: EGR_OK or a negative EGR_ERR_* code.  Argument errors are detected before any launch
 *     and leave all buffers untouched.  There is no CPU fallback: without a CUDA device the compute entry
 *     points return EGR_ERR_CUDA.
 *   - Device-side waits are bounded.  A kernel that gives up records EGR_ERR_TIMEOUT in the first word
 *     of the workspace; egr_workspace_status() reads it back.
 *   - Host threads: calls may come from several threads when each uses its own workspace and stream.  The
 *     exception is egr_es_update / egr_es_gradient on bf16 layers, which stage the factors of the next
 *     K-chunk on one internal side stream per device: the caller serialises those calls per device.
 */
#ifndef EGR_H_
#define EGR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* element types */
#define EGR_F32   0
#define EGR_BF16  1
#define EGR_I8    2

/* egr_layer.flags */
#define EGR_ANTITHETIC  1u   /* members 2p, 2p+1 share noise index p with signs +, - */
#define EGR_NO_PERTURB  2u   /* forward only: skip the low-rank term entirely (unperturbed inference) */
/* forward only (fp32 and bf16 layers): element-wise function applied to the perturbed product, in fp32, before the
 * one rounding of the output -- the activations of the experiments' networks (tanh, relu) and the exact GELU
 * x Phi(x), Phi the standard normal distribution function.  Every other entry point rejects these bits. */
#define EGR_ACT_MASK   12u
#define EGR_ACT_TANH    4u
#define EGR_ACT_RELU    8u
#define EGR_ACT_GELU   12u

/* egr_fitness_shape modes */
#define EGR_SHAPE_NONE             0
#define EGR_SHAPE_CENTERED_RANK    1
#define EGR_SHAPE_ZSCORE           2
#define EGR_SHAPE_ANTITHETIC_SIGN  3

/* operations, for egr_workspace_bytes */
#define EGR_OP_PERTURBED_LINEAR     0
#define EGR_OP_ES_UPDATE            1
#define EGR_OP_FITNESS_SHAPE        2
#define EGR_OP_PERTURBED_LINEAR_I8  3
#define EGR_OP_ES_UPDATE_I8         4
#define EGR_OP_FITNESS_SHAPE_QUESTIONS 5
#define EGR_OP_PERTURBED_LINEAR_LOGLIK 10   /* 6 .. 9 are the operations of egr_q8.h */

/* return codes */
#define EGR_OK                0
#define EGR_ERR_BADARG       (-1)   /* null pointer, non-positive size, rank not in {1,2,4,8,16}, ...      */
#define EGR_ERR_ALIGN        (-2)   /* pointer or pitch violates the alignment rules below                 */
#define EGR_ERR_UNSUPPORTED  (-3)   /* dtype combination not implemented                                   */
#define EGR_ERR_WORKSPACE    (-4)   /* ws is null or smaller than egr_workspace_bytes()                    */
#define EGR_ERR_CUDA         (-5)   /* a CUDA runtime call failed (no device, launch error)                */
#define EGR_ERR_TIMEOUT      (-6)   /* a bounded device-side wait ran out                                  */
#define EGR_ERR_CAPACITY     (-7)   /* problem larger than the built-in scratch of a *_static entry point  */

/*
 * One perturbed matrix.  W is [d_out][d_in] = [m][n] (Section 4.2: M in R^{d_out x d_in}); X is
 * [n_members * rows_per_member][d_in] with row rho belonging to member member_base + rho / rows_per_member.
 */
typedef struct egr_layer {
    int32_t  d_in;             /* n                                                                       */
    int32_t  d_out;            /* m                                                                       */
    int32_t  n_members;        /* N (even with EGR_ANTITHETIC)                                            */
    int32_t  rows_per_member;  /* T >= 1                                                                  */
    int32_t  rank;             /* r in {1,2,4,8,16}; the integer entry points require r = 1               */
    uint32_t layer_id;         /* distinct per perturbed matrix                                           */
    uint64_t seed;             /* per ES step; the caller passes seed0 + step                             */
    uint32_t flags;            /* EGR_ANTITHETIC | EGR_NO_PERTURB                                         */
    int32_t  x_dtype;          /* EGR_F32 | EGR_BF16 | EGR_I8                                             */
    int32_t  w_dtype;
    int32_t  y_dtype;
    int64_t  ldx, ldw, ldy;    /* row pitches in elements                                                 */
    int32_t  member_base;      /* forward only: population index of the first member in X (0 unless the   */
                               /* population is sharded; even with EGR_ANTITHETIC).  Row rho belongs to   */
                               /* member member_base + rho / rows_per_member.                             */
} egr_layer;

/*
 * Perturbed linear forward (Section 4.2):
 *   Y[rho][j] = sum_l X[rho][l] W[j][l] + sign_i (sigma / sqrt r) sum_k (sum_l X[rho][l] B_p[l][k]) A_p[j][k]
 * Supported dtypes (x, w, y): (F32,F32,F32) fp32 FMA throughout; (BF16,BF16,BF16|F32) bf16 operands on
 * the tcgen05 tensor cores with fp32 accumulation, low-rank term added in fp32 before the one rounding of
 * the output.  bf16 operands: X, W 16-byte aligned, ldx, ldw multiples of 8; Y 16-byte aligned, ldy a
 * multiple of 8.  fp32: 16-byte aligned pointers, pitches multiples of 4.
 * X [R][ldx] in, W [m][ldw] in, Y [R][ldy] out, R = N*T.  ws: egr_workspace_bytes(layer, EGR_OP_PERTURBED_LINEAR).
 * With one of the EGR_ACT_* flags Y = act(the sum above).  fp32 outputs use the fp32 library functions (a few
 * ulp); bf16 outputs use the hardware tanh approximation (relative error 2^-11, below the rounding of the output).
 */
int egr_perturbed_linear(const egr_layer *layer, const void *X, const void *W, float sigma,
                         void *Y, void *ws, size_t ws_bytes, void *stream);

/*
 * Same forward with an explicit row -> member map (batched multi-adapter inference in the style Section 4.2
 * alludes to: rows of different members in any order and in any number per member, e.g. ragged sequences).
 * member_of_row is [R] int32 on the device, R = n_members * rows_per_member rows in X and Y; entry rho is the
 * population index whose perturbation row rho sees (with EGR_ANTITHETIC, indices 2p and 2p+1 share noise p).
 * rows_per_member and member_base only define R here.  Everything else is as in egr_perturbed_linear.
 */
int egr_perturbed_linear_rows(const egr_layer *layer, const void *X, const void *W, const int32_t *member_of_row,
                              float sigma, void *Y, void *ws, size_t ws_bytes, void *stream);

/*
 * Perturbed vocabulary head that ends in the fitness of the LLM fine-tuning experiments, the log-likelihood of given
 * tokens, instead of a matrix of logits: with z[rho][j] the perturbed linear forward of Section 4.2 (fp32, not rounded),
 *   logp[rho] = z[rho][target[rho]] - log sum_j exp(z[rho][j]),        j over the d_out columns.
 * The logits never reach memory: every epilogue warp keeps a running maximum and sum of exponentials over the columns
 * it sees of a row, one (maximum, sum) pair per row and 128-column part goes to the workspace, and a second small kernel
 * adds the parts up in column order.  bf16 X and W only (alignment rules of egr_perturbed_linear); y_dtype, ldy and the
 * EGR_ACT_* flags are not used (the flags are rejected).  targets [R] int32 on the device; a target outside
 * [0, d_out) gives logp = 0 for that row (a position that is not scored).  logp [R] fp32 out.
 * ws: egr_workspace_bytes(layer, EGR_OP_PERTURBED_LINEAR_LOGLIK) (the forward's scratch plus 8 bytes per row and part).
 */
int egr_perturbed_linear_loglik(const egr_layer *layer, const void *X, const void *W, float sigma,
                                const int32_t *targets, float *logp, void *ws, size_t ws_bytes, void *stream);

/*
 * EGGROLL update (boxed update; Algorithm 1 last loop; Section 4.2 "(diag(f) A)^T B"):
 *   dW = (alpha / (N sqrt r)) sum_p g_p A_p B_p^T,   g_p = f_p, or f_2p - f_2p+1 with EGR_ANTITHETIC
 *   W_master += dW   (fp32, in place, [m][ldw])
 * layer->w_dtype selects the arithmetic: EGR_F32 regenerates the factors in fp32 and accumulates with fp32
 * FMA; EGR_BF16 rounds the regenerated factors to bf16 and contracts them on the tensor cores with fp32
 * accumulation.  W_shadow_bf16 (nullable, [m][ldw] bf16) receives the master rounded to nearest-even;
 * dW_out (nullable, [m][d_in] fp32, dense) receives dW.  shaped_fitness is [N] fp32.
 * rows_per_member, x_dtype, y_dtype, ldx, ldy are ignored.
 */
int egr_es_update(const egr_layer *layer, float *W_master, const float *shaped_fitness, float alpha,
                  void *W_shadow_bf16, float *dW_out, void *ws, size_t ws_bytes, void *stream);

/*
 * Fitness shaping of N raw fitness values (fp32 in, fp32 out, out may not alias raw).
 *   EGR_SHAPE_CENTERED_RANK   F_i = 1/2 - rank_i/(N-1), rank 0 = best (HFT appendix), evaluated as
 *                             (2 asc_i - (N-1)) / (2 (N-1)) in fp32; ties: lower index ranks lower;
 *                             NaN ranks worst.
 *   EGR_SHAPE_ZSCORE          (f - mean) / (std + 1e-8), population std.
 *   EGR_SHAPE_ANTITHETIC_SIGN members 2p, 2p+1 get +s, -s with s = sign(f_2p - f_2p+1) (integer appendix,
 *                             Fitness Shaping).
 *   EGR_SHAPE_NONE            copy.
 * ws: egr_workspace_bytes(layer, EGR_OP_FITNESS_SHAPE) with layer->n_members = N (only that field is read).
 */
int egr_fitness_shape(const float *raw, int32_t N, int32_t mode, float *out,
                      void *ws, size_t ws_bytes, void *stream);

/*
 * Per-question fitness shaping (LLM fine-tuning section: scores of N noise directions on Q questions, normalised
 * per question with one global variance and averaged over the questions):
 *   out[i] = (1/Q) sum_j (S[i][j] - mu_j) / (sigma_bar + 1e-8),
 * mu_j = mean of column j over the members, sigma_bar = root mean square of the centred scores over all (i, j).
 * S is [N][Q] fp32 row-major, out [N] fp32.  ws: egr_workspace_bytes(layer, EGR_OP_FITNESS_SHAPE_QUESTIONS) with
 * layer->n_members = N and layer->d_in = Q.
 */
int egr_fitness_shape_questions(const float *S, int32_t N, int32_t Q, float *out,
                                void *ws, size_t ws_bytes, void *stream);

/*
 * Integer perturbed matmul ("Adding EGGROLL Perturbations"), rank 1, exact integer arithmetic:
 *   t      = sign_i * sum_l X[rho][l] B_p[l]                                  (int32)
 *   Y[j]   = sat127( (sum_l X[rho][l] W[j][l] + ((t * A_p[j]) >> sigma_shift)) >> out_shift )
 * Both shifts are arithmetic (floor); sat127 clamps to [-127,127] (the I_8 cast of the paper's notation).
 * sigma_shift = 4 + sigma_hat, out_shift = 4 + d for n = 4^d ("Matrix Multiplication").
 * A_p[j] = noise_table[(off_A + j) mod 2^table_log2], B_p[l] = noise_table[(off_B + l) mod 2^table_log2],
 * (off_A, off_B) = first two words of Philox(counter (0, p, layer_id, 2)) mod 2^table_log2; the table holds
 * the pre-generated round(16 z) values and is an input.  X [R][ldx], W [m][ldw], Y [R][ldy] int8;
 * d_in a multiple of 4, ldx, ldw multiples of 4, X, W 4-byte aligned.  No int32 overflow for d_in <= 1024.
 */
int egr_perturbed_linear_i8(const egr_layer *layer, const int8_t *X, const int8_t *W,
                            int32_t sigma_shift, int32_t out_shift,
                            const int8_t *noise_table, uint32_t table_log2,
                            int8_t *Y, void *ws, size_t ws_bytes, void *stream);

/*
 * Integer update ("Parameter Update"): E = (diag(F) A)^T B in int32 over the P noise vectors (P = N/2 with
 * EGR_ANTITHETIC, else N); where |E[j][l]| >= threshold, W[j][l] moves one bin towards sign(E), saturating
 * at +-127.  F is [P] int8 in {-1,0,1}; E_out (nullable) is [m][d_in] int32, dense.  The signed factors are gathered
 * from the table into the workspace ((d_out + d_in) bytes per noise vector) and contracted on the int8 tensor cores; no
 * int32 overflow for P <= 133000.  ws: egr_workspace_bytes(layer, EGR_OP_ES_UPDATE_I8).
 */
int egr_es_update_i8(const egr_layer *layer, int8_t *W, const int8_t *F, int32_t threshold,
                     const int8_t *noise_table, uint32_t table_log2, int32_t *E_out,
                     void *ws, size_t ws_bytes, void *stream);

/*
 * egr_perturbed_linear without a workspace argument, for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of the call above, same arithmetic, same kernels.)
 *
 * Who needs it: code that runs inside somebody else's memory plan -- a plug-in that is handed only its input and
 * output buffers, a process whose device memory was carved up before this library was loaded, or a region
 * where cudaMalloc is off limits because it synchronises the whole device.  Such callers cannot produce the
 * scratch buffer the regular entry point asks for, so here the scratch (two status words, the counter from which rows
 * are claimed for the skinny products, one ready counter per 128 rows, and the skinny product s = X B_p itself,
 * N*T*r floats) is a fixed array inside the library's device image.
 *
 * Limits and rules:
 *   - N * T * r <= EGR_STATIC_MAX_S_FLOATS (262144, i.e. 1 MiB of skinny products); larger problems are refused with
 *     EGR_ERR_CAPACITY before anything is launched.  All other argument rules are those of egr_perturbed_linear and
 *     are checked first (an invalid layer is reported as invalid whatever its size).
 *   - The array costs 1 MiB + 8.25 KiB of device memory on every GPU that loads the library, until exit.
 *   - The first call on each device looks up the array's device address (a runtime query, no allocation); make
 *     that first call outside of any stream capture.  No call allocates or frees memory.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in it.  The call
 *     clears what it needs cleared, but two calls whose kernels overlap on the GPU (different streams) race on it:
 *     serialise them.  egr_static_status() plays the role of egr_workspace_status() for this array.
 */
#define EGR_STATIC_MAX_S_FLOATS 262144ull
int egr_perturbed_linear_static(const egr_layer *layer, const void *X, const void *W, float sigma,
                                void *Y, void *stream);
int egr_static_status(void *stream);

/* Pair sign shaping of the integer path: out[p] = sign(raw[2p] - raw[2p+1]), p < N/2 ("Fitness Shaping"). */
int egr_fitness_shape_i8(const int32_t *raw, int32_t N, int8_t *out, void *stream);

/*
 * Base-3 packing of pair signs for the fitness exchange between workers ("Base-3 Fitness Packing and Bandwidth
 * Efficiency"): the ternary values {+1, 0, -1} map to the digits {0, 1, 2} and five of them form one byte,
 *   byte = sum_{i=0..4} digit[5 b + i] * 3^i        (at most 242; 1.6 bit per value).
 * F [count] int8 in {-1,0,1}; packed [(count + 4) / 5] bytes; missing trailing values pack as 0 (digit 1).
 * Unpacking writes exactly `count` values; a byte above 242 decodes its digits modulo 3 like any other.
 */
int egr_fitness_pack3(const int8_t *F, int64_t count, uint8_t *packed, void *stream);
int egr_fitness_unpack3(const uint8_t *packed, int64_t count, int8_t *F, void *stream);

/* ---- test / debug surface (the paper has no counterpart; they expose the noise definition above) ---- */

/* Philox4x32-10 block function on the HOST: ctr, key, out are host pointers. */
int egr_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/* Same block function evaluated on the DEVICE for `count` counters: ctr [count][4], out [count][4] (device). */
int egr_philox4x32_10_device(const uint32_t *ctr, const uint32_t key[2] /*host*/, int64_t count,
                             uint32_t *out, void *stream);

/* Writes factor A (which = 0, d_out x r) or B (which = 1, d_in x r) of member `member` as dense fp32
 * [rows][r].  precise != 0 uses the fp32 library log/sin/cos (the fp32 path), 0 the fast hardware
 * approximations (the bf16 path). */
int egr_noise_materialize(const egr_layer *layer, int32_t member, int32_t which, int32_t precise,
                          float *out, void *stream);

/*
 * Time-out path of the device-side waits, on purpose and harmlessly: one warp waits, with the same bounded wait the
 * tensor-core kernels use, on a barrier that nothing completes; after limit_ms (1 .. 1000) it gives up, writes
 * EGR_ERR_TIMEOUT into the status word of `ws` (read it with egr_workspace_status) and the kernel returns.  The
 * context stays usable.  ws: at least 256 bytes, 256-byte aligned.
 */
int egr_debug_bounded_wait(void *ws, size_t ws_bytes, uint32_t limit_ms, void *stream);

/* Bytes of workspace an operation needs for this layer (EGR_OP_FITNESS_SHAPE reads only layer->n_members). */
size_t egr_workspace_bytes(const egr_layer *layer, int32_t op);

/* Synchronises `stream` and returns the status word kernels left in the workspace (EGR_OK or EGR_ERR_TIMEOUT),
 * or EGR_ERR_CUDA if the device reported an error. */
int egr_workspace_status(const void *ws, void *stream);

const char *egr_strerror(int code);
int egr_version(void);

#ifdef __cplusplus
}
#endif
#endif /* EGR_H_ */

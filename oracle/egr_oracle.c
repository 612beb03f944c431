/*
 * egr_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow CPU statement of what the EGGROLL hot path computes, written from the paper:
 * low-rank perturbed linear forward (Section 4.2), the EGGROLL update (Eq. "EGGROLL UPDATE",
 * Algorithm 1), fitness shaping (rank transform of the HFT appendix, antithetic sign of the
 * "EGG Pretraining with Integer EGGROLL" appendix) and the integer variants of that appendix.
 *
 * Floating point is fp64 throughout; integer paths are exact (int64 with an int32 range check).
 * No blocking, fusion or reordering beyond what each cited definition states.  This file shares
 * no code with the CUDA library and is never imported by it: only tests, the smoke check and the
 * bench's cpu_baseline / reference arm may call it.
 *
 * Parity status: every function here is pinned by tests that do not go through this file's own
 * formulas (known-answer vectors, closed forms, brute force, library routines), see tests/test_oracle_*.py.
 * The integer recurrent LM at the end is an encoding rather than a formula with a closed form: it is pinned
 * by the paper's parameter count, by its tables against the printed real-valued formulas, and by a brute-force
 * numpy restatement of the unperturbed model and of the embedding perturbation on tiny widths.
 * Parity unpinned: none.
 */
#define _GNU_SOURCE
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_ANTITHETIC 1u

/* ------------------------------------------------------------------------------------------
 * Counter-based generator: Philox4x32-10 (Salmon et al. 2011, the RNG family the paper cites in
 * its introduction for "reconstruct noise on demand").  Ten rounds; the key is bumped by the Weyl
 * constants before rounds 2..10.
 * ------------------------------------------------------------------------------------------ */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * One standard-normal entry of a perturbation factor (Assumption 1: i.i.d. zero-mean, unit-variance,
 * symmetric; Gaussian as in the paper's experiments).
 *   counter = (e >> 2, p, layer_id, tag), key = (seed low word, seed high word)
 *   e   = flat element index inside the factor, element (row j, rank column k) -> e = j*r + k
 *   tag = 0 for A (output-side factor, m x r), 1 for B (input-side factor, n x r)
 * Box-Muller on word pairs (x0,x1) -> lanes 0,1 and (x2,x3) -> lanes 2,3:
 *   u1 = ((xa >> 9) + 1) / 2^23 in (0,1],  u2 = (xb >> 9) / 2^23 in [0,1)
 *   lane even: sqrt(-2 ln u1) cos(2 pi u2),  lane odd: sqrt(-2 ln u1) sin(2 pi u2)
 * The canonical value is the real-number result rounded to fp32.
 */
double orc_normal(uint64_t seed, uint32_t layer_id, uint32_t p, uint32_t tag, uint64_t e)
{
    uint32_t ctr[4] = { (uint32_t)(e >> 2), p, layer_id, tag };
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    uint32_t x[4];
    orc_philox4x32_10(ctr, key, x);
    int lane = (int)(e & 3u);
    uint32_t xa = x[(lane >> 1) * 2], xb = x[(lane >> 1) * 2 + 1];
    double u1 = ((double)(xa >> 9) + 1.0) / 8388608.0;
    double u2 = (double)(xb >> 9) / 8388608.0;
    double rho = sqrt(-2.0 * log(u1));
    double ang = 2.0 * M_PI * u2;
    double z = (lane & 1) ? rho * sin(ang) : rho * cos(ang);
    return (double)(float)z;
}

/* Whole factor for noise index p: out[rows*r], element (j,k) at out[j*r+k]. */
void orc_noise_factor(uint64_t seed, uint32_t layer_id, uint32_t p, uint32_t tag,
                      int rows, int r, double *out)
{
    for (int64_t e = 0; e < (int64_t)rows * r; ++e)
        out[e] = orc_normal(seed, layer_id, p, tag, (uint64_t)e);
}

/* member i -> (noise index p, sign).  Antithetic pairs are adjacent members 2p, 2p+1 with signs +,-. */
static void member_noise(int member, uint32_t flags, uint32_t *p, double *sign)
{
    if (flags & ORC_ANTITHETIC) { *p = (uint32_t)(member >> 1); *sign = (member & 1) ? -1.0 : 1.0; }
    else                        { *p = (uint32_t)member;        *sign = 1.0; }
}

/* ------------------------------------------------------------------------------------------
 * Perturbed linear forward, plain definition (Algorithm 1 lines "E_i <- A_i B_i^T / sqrt r",
 * "f(W = M + sigma E_i)"; Section 4.2 left-hand side u_i (M + sigma E_i)^T):
 * W_i is formed explicitly, then y = x W_i^T.
 *   X   [n_sel*T][n]   rows of the selected members, member-major
 *   W   [m][n]
 *   members[n_sel]     population index of each selected member
 *   Y   [n_sel*T][m]
 * ------------------------------------------------------------------------------------------ */
void orc_perturbed_linear_explicit(const double *X, const double *W, const int32_t *members,
                                   int n_sel, int T, int m, int n, int r, uint32_t layer_id,
                                   uint64_t seed, uint32_t flags, double sigma, double *Y)
{
    #pragma omp parallel
    {
        double *A  = (double *)malloc(sizeof(double) * (size_t)m * r);
        double *B  = (double *)malloc(sizeof(double) * (size_t)n * r);
        double *Wi = (double *)malloc(sizeof(double) * (size_t)m * n);
        #pragma omp for schedule(dynamic, 1)
        for (int s = 0; s < n_sel; ++s) {
            uint32_t p; double sign;
            member_noise(members[s], flags, &p, &sign);
            orc_noise_factor(seed, layer_id, p, 0u, m, r, A);
            orc_noise_factor(seed, layer_id, p, 1u, n, r, B);
            for (int j = 0; j < m; ++j)
                for (int l = 0; l < n; ++l) {
                    double e = 0.0;
                    for (int k = 0; k < r; ++k) e += A[(size_t)j * r + k] * B[(size_t)l * r + k];
                    e /= sqrt((double)r);
                    Wi[(size_t)j * n + l] = W[(size_t)j * n + l] + sigma * sign * e;
                }
            for (int t = 0; t < T; ++t) {
                const double *x = X + ((size_t)s * T + t) * n;
                double *y = Y + ((size_t)s * T + t) * m;
                for (int j = 0; j < m; ++j) {
                    double acc = 0.0;
                    for (int l = 0; l < n; ++l) acc += x[l] * Wi[(size_t)j * n + l];
                    y[j] = acc;
                }
            }
        }
        free(A); free(B); free(Wi);
    }
}

/* Same quantity through the factored identity of Section 4.2:
 * u (M + sigma E)^T = u M^T + (sigma / sqrt r) (u B) A^T.  Exists to prove the identity on small layers. */
void orc_perturbed_linear_factored(const double *X, const double *W, const int32_t *members,
                                   int n_sel, int T, int m, int n, int r, uint32_t layer_id,
                                   uint64_t seed, uint32_t flags, double sigma, double *Y)
{
    #pragma omp parallel
    {
        double *A  = (double *)malloc(sizeof(double) * (size_t)m * r);
        double *B  = (double *)malloc(sizeof(double) * (size_t)n * r);
        double *ub = (double *)malloc(sizeof(double) * (size_t)r);
        #pragma omp for schedule(dynamic, 1)
        for (int s = 0; s < n_sel; ++s) {
            uint32_t p; double sign;
            member_noise(members[s], flags, &p, &sign);
            orc_noise_factor(seed, layer_id, p, 0u, m, r, A);
            orc_noise_factor(seed, layer_id, p, 1u, n, r, B);
            for (int t = 0; t < T; ++t) {
                const double *x = X + ((size_t)s * T + t) * n;
                double *y = Y + ((size_t)s * T + t) * m;
                for (int k = 0; k < r; ++k) {
                    double acc = 0.0;
                    for (int l = 0; l < n; ++l) acc += x[l] * B[(size_t)l * r + k];
                    ub[k] = acc;
                }
                for (int j = 0; j < m; ++j) {
                    double acc = 0.0;
                    for (int l = 0; l < n; ++l) acc += x[l] * W[(size_t)j * n + l];
                    double low = 0.0;
                    for (int k = 0; k < r; ++k) low += ub[k] * A[(size_t)j * r + k];
                    y[j] = acc + sigma * sign / sqrt((double)r) * low;
                }
            }
        }
        free(A); free(B); free(ub);
    }
}

/* ------------------------------------------------------------------------------------------
 * EGGROLL update, plain definition (boxed "EGGROLL UPDATE" equation and Algorithm 1):
 *   dW = (alpha / N) * sum_i f_i * E_i,   E_i = sign_i * A_p B_p^T / sqrt r
 * as an explicit sum of rank-r outer products, restricted to the block rows [j0,j1) x cols [l0,l1).
 * With antithetic pairs the pair difference g_p = f_{2p} - f_{2p+1} is formed first, so that equal
 * fitness inside a pair contributes exactly nothing.  N is the number of members (not pairs).
 *   dW_block [(j1-j0)][(l1-l0)]
 * ------------------------------------------------------------------------------------------ */
void orc_es_update_block(const double *fitness, int N, int r, uint32_t layer_id, uint64_t seed,
                         uint32_t flags, double alpha, int j0, int j1, int l0, int l1, double *dW_block)
{
    const int bm = j1 - j0, bn = l1 - l0;
    const int P = (flags & ORC_ANTITHETIC) ? N / 2 : N;
    memset(dW_block, 0, sizeof(double) * (size_t)bm * bn);
    /* Members are split into at most 64 contiguous ranges, each summed in order, and the partial sums
     * are then added in range order: the result does not depend on how many threads ran. */
    const int n_parts = P < 64 ? (P > 0 ? P : 1) : 64;
    double *parts = (double *)calloc((size_t)n_parts * bm * bn, sizeof(double));
    #pragma omp parallel
    {
        double *A = (double *)malloc(sizeof(double) * (size_t)bm * r);
        double *B = (double *)malloc(sizeof(double) * (size_t)bn * r);
        #pragma omp for schedule(dynamic, 1)
        for (int part = 0; part < n_parts; ++part) {
            double *acc = parts + (size_t)part * bm * bn;
            int p_lo = (int)((int64_t)P * part / n_parts), p_hi = (int)((int64_t)P * (part + 1) / n_parts);
            for (int p = p_lo; p < p_hi; ++p) {
                double g = (flags & ORC_ANTITHETIC) ? (fitness[2 * p] - fitness[2 * p + 1]) : fitness[p];
                for (int j = 0; j < bm; ++j)
                    for (int k = 0; k < r; ++k)
                        A[(size_t)j * r + k] = orc_normal(seed, layer_id, (uint32_t)p, 0u, (uint64_t)(j0 + j) * r + k);
                for (int l = 0; l < bn; ++l)
                    for (int k = 0; k < r; ++k)
                        B[(size_t)l * r + k] = orc_normal(seed, layer_id, (uint32_t)p, 1u, (uint64_t)(l0 + l) * r + k);
                for (int j = 0; j < bm; ++j)
                    for (int l = 0; l < bn; ++l) {
                        double e = 0.0;
                        for (int k = 0; k < r; ++k) e += A[(size_t)j * r + k] * B[(size_t)l * r + k];
                        acc[(size_t)j * bn + l] += g * (e / sqrt((double)r));
                    }
            }
        }
        free(A); free(B);
    }
    for (int part = 0; part < n_parts; ++part)
        for (size_t q = 0; q < (size_t)bm * bn; ++q) dW_block[q] += parts[(size_t)part * bm * bn + q];
    free(parts);
    for (size_t q = 0; q < (size_t)bm * bn; ++q) dW_block[q] *= alpha / (double)N;
}

/* ------------------------------------------------------------------------------------------
 * Fitness shaping.
 *   mode 0: identity.
 *   mode 1: centred rank, F_i = 1/2 - rank_i/(N-1) with rank 0 = best (HFT appendix), i.e.
 *           F_i = asc_i/(N-1) - 1/2 where asc_i counts the members that sort before i in ascending
 *           order (ties: lower index first; NaN sorts first = worst).  Evaluated as
 *           (2 asc_i - (N-1)) / (2 (N-1)) and rounded to fp32.
 *   mode 2: z-score (f - mean) / (std + 1e-8), population std.
 *   mode 3: antithetic sign: members 2p, 2p+1 receive +s_p, -s_p with s_p = sign(f_2p - f_2p+1)
 *           ("EGG Pretraining with Integer EGGROLL", Fitness Shaping).
 * ------------------------------------------------------------------------------------------ */
static int sorts_before(double a, int ia, double b, int ib)
{
    int na = isnan(a), nb = isnan(b);
    if (na || nb) {
        if (na && nb) return ia < ib;
        return na;                      /* NaN before every number */
    }
    if (a < b) return 1;
    if (a > b) return 0;
    return ia < ib;
}

void orc_fitness_shape(const double *raw, int N, int mode, double *out)
{
    if (mode == 0) { for (int i = 0; i < N; ++i) out[i] = raw[i]; return; }
    if (mode == 1) {
        #pragma omp parallel for schedule(static)
        for (int i = 0; i < N; ++i) {
            long asc = 0;
            for (int j = 0; j < N; ++j) if (j != i && sorts_before(raw[j], j, raw[i], i)) ++asc;
            double v = (N > 1) ? (2.0 * (double)asc - (double)(N - 1)) / (2.0 * (double)(N - 1)) : 0.0;
            out[i] = (double)(float)v;
        }
        return;
    }
    if (mode == 2) {
        double mean = 0.0, var = 0.0;
        for (int i = 0; i < N; ++i) mean += raw[i];
        mean /= (double)N;
        for (int i = 0; i < N; ++i) var += (raw[i] - mean) * (raw[i] - mean);
        var /= (double)N;
        double sd = sqrt(var);
        for (int i = 0; i < N; ++i) out[i] = (raw[i] - mean) / (sd + 1e-8);
        return;
    }
    if (mode == 3) {
        for (int p = 0; p < N / 2; ++p) {
            double d = raw[2 * p] - raw[2 * p + 1];
            double s = (d > 0.0) ? 1.0 : ((d < 0.0) ? -1.0 : 0.0);
            out[2 * p] = s; out[2 * p + 1] = -s;
        }
        return;
    }
}

/* ==========================================================================================
 * Integer path ("EGG Architecture" and "EGG Pretraining with Integer EGGROLL" appendices).
 * ========================================================================================== */

/* I_8 cast: saturating, -128 is not a valid value (Notation and Operations). */
static int64_t sat127(int64_t v) { return v > 127 ? 127 : (v < -127 ? -127 : v); }

/* u >> s for signed u: floor division by 2^s, written without relying on the C shift of negatives. */
static int64_t floor_shift(int64_t v, int s)
{
    int64_t d = (int64_t)1 << s;
    int64_t q = v / d;
    if ((v % d != 0) && (v < 0)) --q;
    return q;
}

static int64_t check_i32(int64_t v, int *overflow)
{
    if (v > 2147483647LL || v < -2147483648LL) *overflow = 1;
    return v;
}

/* Slice offsets into the pre-generated table of round(16 z) values: one Philox call per
 * (matrix, noise index) with tag 2 and block 0; off_A = x0 mod 2^L, off_B = x1 mod 2^L. */
void orc_i8_offsets(uint64_t seed, uint32_t layer_id, uint32_t p, uint32_t table_log2,
                    uint32_t *off_a, uint32_t *off_b)
{
    uint32_t ctr[4] = { 0u, p, layer_id, 2u };
    uint32_t key[2] = { (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32) };
    uint32_t x[4];
    orc_philox4x32_10(ctr, key, x);
    uint32_t mask = (table_log2 >= 32u) ? 0xffffffffu : ((1u << table_log2) - 1u);
    *off_a = x[0] & mask; *off_b = x[1] & mask;
}

/*
 * Integer perturbed matmul (Adding EGGROLL Perturbations):
 *   y = I8( (u theta^T + ((u . B) I32(A) >> (4 + sigma_hat))) / (16 sqrt n) )
 * with the division a right shift by out_shift = 4 + d for n = 4^d (Matrix Multiplication).
 * t = sign * (u . B);  pert_j = (t * A_j) >> sigma_shift;  y_j = sat127((acc_j + pert_j) >> out_shift).
 * Returns 1 if any intermediate left the int32 range (then the result is not meaningful), else 0.
 */
int orc_perturbed_linear_i8(const int8_t *X, const int8_t *W, const int32_t *members, int n_sel,
                            int T, int m, int n, uint32_t layer_id, uint64_t seed, uint32_t flags,
                            int sigma_shift, int out_shift, const int8_t *table, uint32_t table_log2,
                            int8_t *Y)
{
    int overflow = 0;
    const uint32_t mask = (1u << table_log2) - 1u;
    #pragma omp parallel for schedule(dynamic, 1) reduction(|:overflow)
    for (int s = 0; s < n_sel; ++s) {
        uint32_t p; double sign;
        member_noise(members[s], flags, &p, &sign);
        uint32_t offa, offb;
        orc_i8_offsets(seed, layer_id, p, table_log2, &offa, &offb);
        for (int t = 0; t < T; ++t) {
            const int8_t *x = X + ((size_t)s * T + t) * n;
            int8_t *y = Y + ((size_t)s * T + t) * m;
            int64_t ub = 0;
            for (int l = 0; l < n; ++l) ub += (int64_t)x[l] * (int64_t)table[(offb + (uint32_t)l) & mask];
            ub = check_i32(ub, &overflow);
            int64_t tt = (sign < 0) ? -ub : ub;
            for (int j = 0; j < m; ++j) {
                int64_t acc = 0;
                for (int l = 0; l < n; ++l) acc += (int64_t)x[l] * (int64_t)W[(size_t)j * n + l];
                acc = check_i32(acc, &overflow);
                int64_t a = (int64_t)table[(offa + (uint32_t)j) & mask];
                int64_t pert = floor_shift(check_i32(tt * a, &overflow), sigma_shift);
                y[j] = (int8_t)sat127(floor_shift(check_i32(acc + pert, &overflow), out_shift));
            }
        }
    }
    return overflow;
}

/* Pair sign shaping: F_p = sign(s+_p - s-_p) in {-1,0,1} (Fitness Shaping of the integer appendix). */
void orc_fitness_shape_i8(const int32_t *raw, int N, int8_t *out)
{
    for (int p = 0; p < N / 2; ++p) {
        int64_t d = (int64_t)raw[2 * p] - (int64_t)raw[2 * p + 1];
        out[p] = (int8_t)((d > 0) - (d < 0));
    }
}

/*
 * Integer update (Parameter Update): E = (diag(F) A)^T B in int32; where |E| >= threshold the weight
 * moves one bin in the direction of sign(E), saturating at +-127.  P = number of noise vectors.
 * E_out (nullable) receives E.  Returns 1 on int32 overflow of E.
 */
int orc_es_update_i8(int8_t *W, const int8_t *F, int P, int m, int n, uint32_t layer_id,
                     uint64_t seed, int32_t threshold, const int8_t *table, uint32_t table_log2,
                     int32_t *E_out)
{
    int overflow = 0;
    const uint32_t mask = (1u << table_log2) - 1u;
    uint32_t *offa = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)P);
    uint32_t *offb = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)P);
    for (int p = 0; p < P; ++p) orc_i8_offsets(seed, layer_id, (uint32_t)p, table_log2, &offa[p], &offb[p]);
    #pragma omp parallel for schedule(static) reduction(|:overflow)
    for (int j = 0; j < m; ++j)
        for (int l = 0; l < n; ++l) {
            int64_t e = 0;
            for (int p = 0; p < P; ++p)
                e += (int64_t)F[p] * (int64_t)table[(offa[p] + (uint32_t)j) & mask]
                                   * (int64_t)table[(offb[p] + (uint32_t)l) & mask];
            e = check_i32(e, &overflow);
            if (E_out) E_out[(size_t)j * n + l] = (int32_t)e;
            int64_t mag = e < 0 ? -e : e;
            if (mag >= (int64_t)threshold) {
                int64_t sg = (e > 0) - (e < 0);
                W[(size_t)j * n + l] = (int8_t)sat127((int64_t)W[(size_t)j * n + l] + sg);
            }
        }
    free(offa); free(offb);
    return overflow;
}

/* ==========================================================================================
 * Integer recurrent byte-level LM ("EGG Architecture" appendix, Algorithm "EGG forward pass"),
 * evaluated under per-member rank-1 integer perturbations of every matrix and of the embedding.
 * ========================================================================================== */

/* EXP2[i] = 16 * 2^(i/16), rounded to nearest (Fitness Calculation in Integer Types). */
int32_t orc_exp2_table(int i) { return (int32_t)llrint(16.0 * exp2((double)i / 16.0)); }

/* LOG2(S) = 16 * log2(S / 16) evaluated by an integer algorithm instead of the 2^28-entry table the paper
 * mentions: e = position of the leading one, mant = the 8 bits below it,
 * LOG2 = 16 (e - 4) + round(16 log2(1 + mant/256)).  Within 0.1 of the real-valued formula. */
int32_t orc_log2_int(int64_t S)
{
    int e = 0;
    while ((S >> (e + 1)) != 0) ++e;
    int64_t mant = ((S << 8) >> e) & 0xff;
    int32_t frac = (int32_t)llrint(16.0 * log2(1.0 + (double)mant / 256.0));
    return 16 * (e - 4) + frac;
}

typedef struct {
    int D, n_layers;
    const int8_t *emb_t;      /* [D][256]: column t is the embedding of byte t */
    const int8_t *head;       /* [256][D] */
    const int8_t *ln_out;     /* [D] */
    const int8_t *ln1, *ln2;  /* [l][D] */
    const int8_t *Wf, *Uf, *Wh, *Uh;   /* [l][D][D] */
    const int8_t *bf, *bh;    /* [l][D] */
    const int8_t *mlp1;       /* [l][4D][D] */
    const int8_t *mlp2;       /* [l][D][4D] */
    const int8_t *lut_sigma, *lut_phi;   /* [256], indexed by value + 128 */
    const int8_t *table; uint32_t table_log2;
    uint64_t seed; uint32_t flags; int sigma_shift;
} orc_lm;

static int log4_of(int n) { int d = 0; while ((1 << (2 * d)) < n) ++d; return d; }

/* perturbed matmul for one input vector: y[m] = pm(u[n], theta[m][n]) with the member's noise (p, sign) */
static void lm_pm(const orc_lm *M, const int8_t *u, const int8_t *theta, int m, int n, uint32_t layer_id,
                  uint32_t p, int sign, int8_t *y, int *overflow)
{
    const uint32_t mask = (1u << M->table_log2) - 1u;
    uint32_t offa, offb;
    orc_i8_offsets(M->seed, layer_id, p, M->table_log2, &offa, &offb);
    const int out_shift = 4 + log4_of(n);
    int64_t ub = 0;
    for (int l = 0; l < n; ++l) ub += (int64_t)u[l] * (int64_t)M->table[(offb + (uint32_t)l) & mask];
    ub = check_i32(ub, overflow);
    int64_t t = sign < 0 ? -ub : ub;
    for (int j = 0; j < m; ++j) {
        int64_t acc = 0;
        for (int l = 0; l < n; ++l) acc += (int64_t)u[l] * (int64_t)theta[(size_t)j * n + l];
        int64_t a = (int64_t)M->table[(offa + (uint32_t)j) & mask];
        int64_t pert = floor_shift(check_i32(t * a, overflow), M->sigma_shift);
        y[j] = (int8_t)sat127(floor_shift(check_i32(acc + pert, overflow), out_shift));
    }
}

/* Layer normalisation: u_mav = I8(sum|u| >> 2d); out = DIVIDE(I16(u) * I16(w), u_mav), division truncating
 * toward zero, divisor at least 1, result saturated. */
static void lm_ln(int D, const int8_t *w, const int8_t *u, int8_t *out)
{
    int64_t sum = 0;
    for (int j = 0; j < D; ++j) sum += u[j] < 0 ? -(int64_t)u[j] : (int64_t)u[j];
    int64_t mav = sat127(floor_shift(sum, 2 * log4_of(D)));
    if (mav < 1) mav = 1;
    for (int j = 0; j < D; ++j) {
        int64_t prod = (int64_t)u[j] * (int64_t)w[j];
        out[j] = (int8_t)sat127(prod / mav);          /* C division truncates toward zero */
    }
}

/*
 * Forward over one token sequence for each selected member; state[l][D] per member starts from the given
 * values and is updated in place; fitness[s] += sum over positions of (z[t'] - LOG2(sum_v EXP2[z_v])).
 *   tokens      [n_seq][seq_len]
 *   member_seq  [n_sel]   which sequence each selected member reads
 *   state       [n_sel][l][D]
 */
int orc_i8lm_forward(const orc_lm *M, const uint8_t *tokens, int seq_len, const int32_t *members,
                     const int32_t *member_seq, int n_sel, int8_t *state, int32_t *fitness)
{
    int overflow = 0;
    const int D = M->D, L = M->n_layers;
    #pragma omp parallel for schedule(dynamic, 1) reduction(|:overflow)
    for (int s = 0; s < n_sel; ++s) {
        uint32_t p; double dsign;
        member_noise(members[s], M->flags, &p, &dsign);
        const int sign = dsign < 0 ? -1 : 1;
        const uint32_t mask = (1u << M->table_log2) - 1u;
        int8_t *y = (int8_t *)malloc((size_t)D), *x = (int8_t *)malloc((size_t)D);
        int8_t *a = (int8_t *)malloc((size_t)D), *b = (int8_t *)malloc((size_t)D);
        int8_t *f = (int8_t *)malloc((size_t)D), *fh = (int8_t *)malloc((size_t)D), *hh = (int8_t *)malloc((size_t)D);
        int8_t *h1 = (int8_t *)malloc((size_t)4 * D), *y2 = (int8_t *)malloc((size_t)D);
        int8_t logits[256];
        const uint8_t *tok = tokens + (size_t)member_seq[s] * seq_len;
        int8_t *st = state + (size_t)s * L * D;
        int64_t fit = 0;
        for (int pos = 0; pos + 1 < seq_len; ++pos) {
            const int t = tok[pos], tn = tok[pos + 1];
            /* embedding: u.B becomes B[t] (Adding EGGROLL Perturbations, last paragraph); no 16 sqrt(n) division */
            uint32_t offa, offb;
            orc_i8_offsets(M->seed, 1000u, p, M->table_log2, &offa, &offb);
            const int64_t bt = (int64_t)sign * (int64_t)M->table[(offb + (uint32_t)t) & mask];
            for (int j = 0; j < D; ++j) {
                int64_t aj = (int64_t)M->table[(offa + (uint32_t)j) & mask];
                y[j] = (int8_t)sat127((int64_t)M->emb_t[(size_t)j * 256 + t] + floor_shift(bt * aj, M->sigma_shift));
            }
            for (int i = 0; i < L; ++i) {
                int8_t *si = st + (size_t)i * D;
                const uint32_t id = 16u * (uint32_t)i;
                /* GRU */
                lm_ln(D, M->ln1 + (size_t)i * D, y, x);
                lm_pm(M, x, M->Wf + (size_t)i * D * D, D, D, id + 0, p, sign, a, &overflow);
                lm_pm(M, si, M->Uf + (size_t)i * D * D, D, D, id + 1, p, sign, b, &overflow);
                for (int j = 0; j < D; ++j) {
                    int64_t pre = sat127((int64_t)a[j] + (int64_t)b[j] + (int64_t)M->bf[(size_t)i * D + j]);
                    f[j] = M->lut_sigma[pre + 128];
                    fh[j] = (int8_t)sat127(floor_shift(((int64_t)f[j] + 127) * (int64_t)si[j], 8));
                }
                lm_pm(M, x, M->Wh + (size_t)i * D * D, D, D, id + 2, p, sign, a, &overflow);
                lm_pm(M, fh, M->Uh + (size_t)i * D * D, D, D, id + 3, p, sign, b, &overflow);
                for (int j = 0; j < D; ++j) {
                    int64_t pre = sat127((int64_t)a[j] + (int64_t)b[j] + (int64_t)M->bh[(size_t)i * D + j]);
                    hh[j] = M->lut_phi[pre + 128];
                    int64_t delta = sat127(floor_shift(((int64_t)f[j] + 127) * ((int64_t)hh[j] - (int64_t)si[j]), 8));
                    int64_t h = sat127((int64_t)si[j] + delta);
                    si[j] = (int8_t)h;
                    y[j] = (int8_t)sat127(h + (int64_t)y[j]);
                }
                /* MLP */
                lm_ln(D, M->ln2 + (size_t)i * D, y, x);
                lm_pm(M, x, M->mlp1 + (size_t)i * 4 * D * D, 4 * D, D, id + 4, p, sign, h1, &overflow);
                lm_pm(M, h1, M->mlp2 + (size_t)i * 4 * D * D, D, 4 * D, id + 5, p, sign, y2, &overflow);
                for (int j = 0; j < D; ++j) y[j] = (int8_t)sat127((int64_t)y2[j] + (int64_t)y[j]);
            }
            lm_ln(D, M->ln_out, y, x);
            lm_pm(M, x, M->head, 256, D, 1001u, p, sign, logits, &overflow);
            int64_t S = 0;
            for (int v = 0; v < 256; ++v) S += orc_exp2_table((int)logits[v] + 128);
            fit += ((int64_t)logits[tn] + 128) - (int64_t)orc_log2_int(S);
        }
        fitness[s] = (int32_t)check_i32((int64_t)fitness[s] + fit, &overflow);
        free(y); free(x); free(a); free(b); free(f); free(fh); free(hh); free(h1); free(y2);
    }
    return overflow;
}

/*
 * Per-question normalised score ("our scoring function draws parallels to the group relative advantage of GRPO",
 * LLM fine-tuning section): S[i][j] is the score of member i on question j;
 *   out_i = (1/Q) sum_j (S[i][j] - mu_j) / sigma_bar,
 * mu_j the mean of question j over the members and sigma_bar one global standard deviation for all questions.
 * Reading: sigma_bar is the root mean square of the centred scores over all (i, j), plus 1e-8.
 */
void orc_fitness_shape_questions(const double *S, int N, int Q, double *out)
{
    double *mu = (double *)calloc((size_t)Q, sizeof(double));
    for (int i = 0; i < N; ++i) for (int j = 0; j < Q; ++j) mu[j] += S[(size_t)i * Q + j];
    for (int j = 0; j < Q; ++j) mu[j] /= (double)N;
    double var = 0.0;
    for (int i = 0; i < N; ++i) for (int j = 0; j < Q; ++j) { double d = S[(size_t)i * Q + j] - mu[j]; var += d * d; }
    var /= (double)N * (double)Q;
    double sd = sqrt(var) + 1e-8;
    for (int i = 0; i < N; ++i) {
        double acc = 0.0;
        for (int j = 0; j < Q; ++j) acc += (S[(size_t)i * Q + j] - mu[j]) / sd;
        out[i] = acc / (double)Q;
    }
    free(mu);
}

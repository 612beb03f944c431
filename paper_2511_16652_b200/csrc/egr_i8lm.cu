// Integer-only recurrent LM (appendix "EGG Architecture") evaluated for a whole population: a host loop over
// positions and layers.  At the paper's width (D = 256) every layer is one tensor-core tile wide and the
// element-wise steps (GRU gates with 256-entry tables, saturating residuals, layer norms, integer log-likelihood)
// run inside the epilogues of the int8 tcgen05 kernel: one launch for the whole sequence (every CTA pair walks all
// positions for its own 256 members) for up to eight layers, 4 launches per layer and position beyond.  Other widths
// chain the perturbed matmul with small element-wise kernels that move 16 int8 values (128 bits) per thread.
#include <cmath>
#include <vector>

#include "../../include/egr_i8lm.h"
#include "egr_device.cuh"
#include "egr_internal.h"

namespace egr {
namespace {

__device__ __forceinline__ int sat127(int v) { return max(-127, min(127, v)); }

// EXP2[i] = round(16 * 2^(i/16)), FRAC[k] = round(16 * log2(1 + k/256)); filled once per device from the host
static __device__ int g_exp2[256];
static __device__ int g_frac[256];

struct I8x16 { int8_t v[16]; };
__device__ __forceinline__ I8x16 ld16(const int8_t *p) { I8x16 r; *reinterpret_cast<int4 *>(r.v) = *reinterpret_cast<const int4 *>(p); return r; }
__device__ __forceinline__ void st16(int8_t *p, const I8x16 &r) { *reinterpret_cast<int4 *>(p) = *reinterpret_cast<const int4 *>(r.v); }

// y[rho][j] = sat127(emb_t[j][t] + ((sign * B_p[t] * A_p[j]) >> sigma_shift)), 16 values of j per thread
__global__ void __launch_bounds__(256)
lm_embed_kernel(const int8_t *__restrict__ emb_t, const uint8_t *__restrict__ tokens, int seq_len, int pos,
                const int32_t *__restrict__ member_seq, int N, int D, uint32_t flags, NoiseKey key, int sigma_shift,
                const int8_t *__restrict__ table, uint32_t mask, int8_t *__restrict__ y)
{
    const int per_row = D >> 4;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)N * per_row) return;
    const int member = (int)(idx / per_row), j0 = (int)(idx % per_row) * 16;
    uint32_t p; float sign;
    member_noise(member, flags, p, sign);
    const uint4 x = philox4x32_10(0u, p, key.layer_id, kTagI8, key.k0, key.k1);
    const uint32_t off_a = x.x & mask, off_b = x.y & mask;
    const int t = tokens[(int64_t)member_seq[member] * seq_len + pos];
    const int bt = (sign < 0.f ? -1 : 1) * (int)table[(off_b + (uint32_t)t) & mask];
    I8x16 out;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int j = j0 + i;
        const int a = (int)table[(off_a + (uint32_t)j) & mask];
        out.v[i] = (int8_t)sat127((int)emb_t[(int64_t)j * 256 + t] + ((bt * a) >> sigma_shift));
    }
    st16(y + (int64_t)member * D + j0, out);
}

// [D][256] -> [256][D]: the embedding of a token becomes one contiguous row (a column of the stored matrix costs one
// cache line per element)
__global__ void __launch_bounds__(256) lm_transpose_emb_kernel(const int8_t *__restrict__ emb_t, int D, int8_t *__restrict__ rows)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 256 * D) return;
    const int tok = i / D, j = i % D;
    rows[i] = emb_t[(int64_t)j * 256 + tok];
}

// fused path (D = 256): embedding and the first layer norm in one pass, one warp per member (8 values per lane);
// emb_rows is the transposed embedding [256][256]
__global__ void __launch_bounds__(256)
lm_embed_ln256_kernel(const int8_t *__restrict__ emb_rows, const uint8_t *__restrict__ tokens, int seq_len, int pos,
                      const int32_t *__restrict__ member_seq, int N, uint32_t flags, NoiseKey key, int sigma_shift,
                      const int8_t *__restrict__ table, uint32_t mask, const int8_t *__restrict__ ln_w, int ln_shift,
                      int8_t *__restrict__ y, int8_t *__restrict__ x)
{
    const int lane = threadIdx.x & 31;
    const int64_t member = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (member >= N) return;
    lm_embed_ln256_row(emb_rows, tokens, seq_len, pos, member_seq, member, flags, key, sigma_shift, table, mask, ln_w, ln_shift,
                       y, x, lane);
}

// layer norm, one warp per row: mav = sat127(sum|u| >> 2d); out = sat127(trunc(u*w / max(mav,1)))
__global__ void __launch_bounds__(256)
lm_ln_kernel(const int8_t *__restrict__ w, const int8_t *__restrict__ u, int N, int D, int shift2d, int8_t *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= N) return;
    const int8_t *ur = u + row * D;
    int sum = 0;
    for (int j = lane * 16; j < D; j += 512) {
        const I8x16 v = ld16(ur + j);
#pragma unroll
        for (int i = 0; i < 16; ++i) sum += abs((int)v.v[i]);
    }
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    const int mav = max(1, sat127(sum >> shift2d));
    for (int j = lane * 16; j < D; j += 512) {
        const I8x16 v = ld16(ur + j), ww = ld16(w + j);
        I8x16 o;
#pragma unroll
        for (int i = 0; i < 16; ++i) o.v[i] = (int8_t)sat127(((int)v.v[i] * (int)ww.v[i]) / mav);   // C division truncates
        st16(out + row * D + j, o);
    }
}

// f = lut_sigma[sat127(a + b + bf)], fh = sat127(((f + 127) * s) >> 8)
__global__ void __launch_bounds__(256)
lm_gate_f_kernel(const int8_t *__restrict__ a, const int8_t *__restrict__ b, const int8_t *__restrict__ bias,
                 const int8_t *__restrict__ s, const int8_t *__restrict__ lut, int64_t total, int D,
                 int8_t *__restrict__ f, int8_t *__restrict__ fh)
{
    const int64_t e = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 16;
    if (e >= total) return;
    const int j0 = (int)(e % D);
    const I8x16 va = ld16(a + e), vb = ld16(b + e), vs = ld16(s + e), vbias = ld16(bias + j0);
    I8x16 of, ofh;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int pre = sat127((int)va.v[i] + (int)vb.v[i] + (int)vbias.v[i]);
        const int fv = (int)lut[pre + 128];
        of.v[i] = (int8_t)fv;
        ofh.v[i] = (int8_t)sat127(((fv + 127) * (int)vs.v[i]) >> 8);
    }
    st16(f + e, of); st16(fh + e, ofh);
}

// hh = lut_phi[sat127(a + b + bh)], h = sat127(s + sat127(((f + 127)(hh - s)) >> 8)), s <- h, y <- sat127(h + y)
__global__ void __launch_bounds__(256)
lm_gate_h_kernel(const int8_t *__restrict__ a, const int8_t *__restrict__ b, const int8_t *__restrict__ bias,
                 const int8_t *__restrict__ f, const int8_t *__restrict__ lut, int64_t total, int D,
                 int8_t *__restrict__ s, int8_t *__restrict__ y)
{
    const int64_t e = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 16;
    if (e >= total) return;
    const int j0 = (int)(e % D);
    const I8x16 va = ld16(a + e), vb = ld16(b + e), vf = ld16(f + e), vbias = ld16(bias + j0);
    I8x16 vs = ld16(s + e), vy = ld16(y + e);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int pre = sat127((int)va.v[i] + (int)vb.v[i] + (int)vbias.v[i]);
        const int hh = (int)lut[pre + 128];
        const int sv = (int)vs.v[i];
        const int delta = sat127((((int)vf.v[i] + 127) * (hh - sv)) >> 8);
        const int h = sat127(sv + delta);
        vs.v[i] = (int8_t)h;
        vy.v[i] = (int8_t)sat127(h + (int)vy.v[i]);
    }
    st16(s + e, vs); st16(y + e, vy);
}

// y <- sat127(y2 + y)
__global__ void __launch_bounds__(256)
lm_residual_kernel(const int8_t *__restrict__ y2, int64_t total, int8_t *__restrict__ y)
{
    const int64_t e = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 16;
    if (e >= total) return;
    const I8x16 v2 = ld16(y2 + e);
    I8x16 vy = ld16(y + e);
#pragma unroll
    for (int i = 0; i < 16; ++i) vy.v[i] = (int8_t)sat127((int)v2.v[i] + (int)vy.v[i]);
    st16(y + e, vy);
}

// integer log-likelihood of the next byte, one warp per row of 256 logits
__global__ void __launch_bounds__(256)
lm_loglik_kernel(const int8_t *__restrict__ logits, const uint8_t *__restrict__ tokens, int seq_len, int pos,
                 const int32_t *__restrict__ member_seq, int N, int32_t *__restrict__ fitness)
{
    const int lane = threadIdx.x & 31;
    const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= N) return;
    const int8_t *lr = logits + row * 256;
    const int2 v8 = *reinterpret_cast<const int2 *>(lr + lane * 8);
    const int8_t *b = reinterpret_cast<const int8_t *>(&v8);
    int S = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) S += g_exp2[(int)b[i] + 128];
    for (int off = 16; off > 0; off >>= 1) S += __shfl_xor_sync(0xffffffffu, S, off);
    if (lane == 0) {
        const int tn = tokens[(int64_t)member_seq[row] * seq_len + pos + 1];
        const int zt = (int)lr[tn] + 128;
        const int e = 31 - __clz(S);
        const int mant = (int)((((long long)S << 8) >> e) & 0xff);
        fitness[row] += zt - (16 * (e - 4) + g_frac[mant]);
    }
}

const int *g_exp2_ptr[64] = {}, *g_frac_ptr[64] = {};

int tables_ready()
{
    static bool done[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return EGR_ERR_CUDA;
    if (done[dev]) return EGR_OK;
    void *pe = nullptr, *pf = nullptr;
    if (cudaGetSymbolAddress(&pe, g_exp2) != cudaSuccess || cudaGetSymbolAddress(&pf, g_frac) != cudaSuccess) return EGR_ERR_CUDA;
    g_exp2_ptr[dev] = (const int *)pe; g_frac_ptr[dev] = (const int *)pf;
    int e2[256], fr[256];
    for (int i = 0; i < 256; ++i) {
        e2[i] = (int)std::llrint(16.0 * std::exp2((double)i / 16.0));
        fr[i] = (int)std::llrint(16.0 * std::log2(1.0 + (double)i / 256.0));
    }
    if (cudaMemcpyToSymbol(g_exp2, e2, sizeof(e2)) != cudaSuccess) return EGR_ERR_CUDA;
    if (cudaMemcpyToSymbol(g_frac, fr, sizeof(fr)) != cudaSuccess) return EGR_ERR_CUDA;
    done[dev] = true;
    return EGR_OK;
}

int log4_exact(int n)
{
    int d = 0;
    while ((1 << (2 * d)) < n) ++d;
    return ((1 << (2 * d)) == n) ? d : -1;
}

struct Buffers { int8_t *y, *x, *a, *b, *f, *fh, *y2, *h1, *logits; void *pm_ws; int8_t *emb_rows; };

size_t carve(const egr_i8lm &M, unsigned char *base, Buffers *out)
{
    const size_t ND = align_up((size_t)M.n_members * M.D, 256);
    size_t off = 0;
    auto take = [&](size_t bytes) { unsigned char *p = base ? base + off : nullptr; off += align_up(bytes, 256); return p; };
    int8_t *y = (int8_t *)take(ND), *x = (int8_t *)take(ND), *a = (int8_t *)take(ND), *b = (int8_t *)take(ND);
    int8_t *f = (int8_t *)take(ND), *fh = (int8_t *)take(ND), *y2 = (int8_t *)take(ND);
    int8_t *h1 = (int8_t *)take(4 * ND), *logits = (int8_t *)take((size_t)M.n_members * 256);
    void *pm_ws = take(kWsHeader + align_up((size_t)M.n_members * 8, 256));
    int8_t *emb_rows = (int8_t *)take((size_t)256 * M.D);          // the embedding transposed: [256 tokens][D]
    if (out) *out = Buffers{y, x, a, b, f, fh, y2, h1, logits, pm_ws, emb_rows};
    return off;
}

}  // namespace
}  // namespace egr

using namespace egr;

extern "C" size_t egr_i8lm_workspace_bytes(const egr_i8lm *M)
{
    if (!M || M->D <= 0 || M->n_members <= 0) return 0;
    return carve(*M, nullptr, nullptr);
}

extern "C" int egr_i8lm_forward(const egr_i8lm *M, const uint8_t *tokens, int32_t n_seq, int32_t seq_len,
                                const int32_t *member_seq, int8_t *state, int32_t *fitness, void *ws, size_t ws_bytes,
                                void *stream)
{
    if (!M || !tokens || !member_seq || !state || !fitness) return EGR_ERR_BADARG;
    if (M->D < 16 || (M->D & 15) || log4_exact(M->D) < 0 || M->n_layers < 0 || M->n_members <= 0) return EGR_ERR_BADARG;
    if (n_seq <= 0 || seq_len < 2) return EGR_ERR_BADARG;
    if ((M->flags & EGR_ANTITHETIC) && (M->n_members & 1)) return EGR_ERR_BADARG;
    if (M->flags & ~EGR_ANTITHETIC) return EGR_ERR_BADARG;
    if (M->sigma_shift < 0 || M->sigma_shift > 31 || M->table_log2 < 2 || M->table_log2 > 31) return EGR_ERR_BADARG;
    if (!M->emb_t || !M->head || !M->ln_out || !M->lut_sigma || !M->lut_phi || !M->noise_table) return EGR_ERR_BADARG;
    if (M->n_layers > 0 && (!M->ln1 || !M->ln2 || !M->Wf || !M->Uf || !M->Wh || !M->Uh || !M->bf || !M->bh || !M->mlp1 || !M->mlp2))
        return EGR_ERR_BADARG;
    const void *ptrs[] = {M->emb_t, M->head, M->ln_out, M->ln1, M->ln2, M->Wf, M->Uf, M->Wh, M->Uh, M->bf, M->bh,
                          M->mlp1, M->mlp2, state};
    for (const void *p : ptrs) if (reinterpret_cast<uintptr_t>(p) & 15) return EGR_ERR_ALIGN;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) || ws_bytes < egr_i8lm_workspace_bytes(M)) return EGR_ERR_WORKSPACE;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev <= 0) return EGR_ERR_CUDA;
    int rc = tables_ready();
    if (rc != EGR_OK) return rc;

    cudaStream_t st = (cudaStream_t)stream;
    const int N = M->n_members, D = M->D, Lyr = M->n_layers;
    const int64_t ND = (int64_t)N * D;
    Buffers B;
    carve(*M, (unsigned char *)ws, &B);
    const uint32_t mask = (1u << M->table_log2) - 1u;
    const int d = log4_exact(D);
    const size_t pm_ws_bytes = kWsHeader + align_up((size_t)N * 8, 256);

    auto pm = [&](const int8_t *X, const int8_t *W, int n, int m, uint32_t layer_id, int8_t *Y) -> int {
        egr_layer L = {};
        L.d_in = n; L.d_out = m; L.n_members = N; L.rows_per_member = 1; L.rank = 1; L.layer_id = layer_id;
        L.seed = M->seed; L.flags = M->flags; L.x_dtype = L.w_dtype = L.y_dtype = EGR_I8;
        L.ldx = n; L.ldw = n; L.ldy = m;
        return egr_perturbed_linear_i8(&L, X, W, M->sigma_shift, 4 + log4_exact(n), M->noise_table, M->table_log2, Y,
                                       B.pm_ws, pm_ws_bytes, stream);
    };
    const unsigned g16 = (unsigned)((ND / 16 + 255) / 256);
    const unsigned gwarp = (unsigned)(((int64_t)N * 32 + 255) / 256);

    if (D == 256) {
        // ---- fused path: every layer is exactly one tensor-core tile wide, element-wise steps live in the epilogues
        int dev = 0;
        cudaGetDevice(&dev);
        int *status = reinterpret_cast<int *>(B.pm_ws);
        if (cudaMemsetAsync(status, 0, 8, st) != cudaSuccess) return EGR_ERR_CUDA;
        I8LmStep q = {};
        q.rows = N; q.seed = M->seed; q.flags = M->flags; q.sigma_shift = M->sigma_shift;
        q.table = M->noise_table; q.table_log2 = M->table_log2; q.tokens = tokens; q.member_seq = member_seq;
        q.seq_len = seq_len; q.fitness = fitness; q.exp2_tab = g_exp2_ptr[dev]; q.frac_tab = g_frac_ptr[dev];
        q.ln_shift = 2 * d; q.status = status;
        const int64_t DD = (int64_t)D * D;
        lm_transpose_emb_kernel<<<(256 * D + 255) / 256, 256, 0, st>>>(M->emb_t, D, B.emb_rows);
        {
            // all positions in one launch: every CTA pair walks the sequence for its own 256 members
            I8LmSeq sq = {};
            sq.rows = N; sq.n_layers = Lyr; sq.seed = M->seed; sq.flags = M->flags; sq.sigma_shift = M->sigma_shift;
            sq.table = M->noise_table; sq.table_log2 = M->table_log2;
            sq.x = B.x; sq.y = B.y; sq.f = B.f; sq.fh = B.fh; sq.h1 = B.h1; sq.state = state;
            sq.Wf = M->Wf; sq.Uf = M->Uf; sq.Wh = M->Wh; sq.Uh = M->Uh; sq.mlp1 = M->mlp1; sq.mlp2 = M->mlp2; sq.head = M->head;
            sq.bf = M->bf; sq.bh = M->bh; sq.ln1 = M->ln1; sq.ln2 = M->ln2; sq.ln_out = M->ln_out;
            sq.lut_sigma = M->lut_sigma; sq.lut_phi = M->lut_phi; sq.emb_rows = B.emb_rows;
            sq.tokens = tokens; sq.member_seq = member_seq; sq.seq_len = seq_len; sq.fitness = fitness;
            sq.exp2_tab = q.exp2_tab; sq.frac_tab = q.frac_tab; sq.ln_shift = 2 * d; sq.status = status;
            rc = launch_lm_seq(sq, st);
            if (rc != EGR_ERR_UNSUPPORTED) return rc;          // more layers than the kernel's parameter block holds: phase by phase
        }
        // every fused step of a position, prepared once: 4 per layer (gate f, gate h, MLP up, MLP down) and the head
        const size_t pb = lm_plan_bytes();
        std::vector<unsigned char> plans((size_t)(4 * Lyr + 1) * pb + 64);
        unsigned char *plan0 = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(plans.data()) + 63) & ~(uintptr_t)63);
        for (int i = 0; i < Lyr; ++i) {
            int8_t *s_i = state + (int64_t)i * ND;
            const uint32_t id = 16u * (uint32_t)i;
            I8LmStep g = q;                                   // f, fh from x and s
            g.cols = D; g.X0 = B.x; g.W0 = M->Wf + i * DD; g.K0 = D; g.layer_id0 = id + 0;
            g.X1 = s_i; g.W1 = M->Uf + i * DD; g.K1 = D; g.layer_id1 = id + 1;
            g.bias = M->bf + (int64_t)i * D; g.lut = M->lut_sigma; g.s = s_i; g.f = B.f; g.fh = B.fh;
            if ((rc = lm_plan_build(1, g, plan0 + (4 * i + 0) * pb)) != EGR_OK) return rc;
            g = q;                                            // h, state, residual, second layer norm
            g.cols = D; g.X0 = B.x; g.W0 = M->Wh + i * DD; g.K0 = D; g.layer_id0 = id + 2;
            g.X1 = B.fh; g.W1 = M->Uh + i * DD; g.K1 = D; g.layer_id1 = id + 3;
            g.bias = M->bh + (int64_t)i * D; g.lut = M->lut_phi; g.s = s_i; g.f = B.f; g.y = B.y; g.x = B.x;
            g.ln_w = M->ln2 + (int64_t)i * D;
            if ((rc = lm_plan_build(2, g, plan0 + (4 * i + 1) * pb)) != EGR_OK) return rc;
            g = q;                                            // MLP up
            g.cols = 4 * D; g.X0 = B.x; g.W0 = M->mlp1 + i * 4 * DD; g.K0 = D; g.layer_id0 = id + 4; g.Y = B.h1;
            if ((rc = lm_plan_build(0, g, plan0 + (4 * i + 2) * pb)) != EGR_OK) return rc;
            g = q;                                            // MLP down, residual, next layer norm
            g.cols = D; g.X0 = B.h1; g.W0 = M->mlp2 + i * 4 * DD; g.K0 = 4 * D; g.layer_id0 = id + 5;
            g.y = B.y; g.x = B.x; g.ln_w = (i + 1 < Lyr) ? M->ln1 + (int64_t)(i + 1) * D : M->ln_out;
            if ((rc = lm_plan_build(3, g, plan0 + (4 * i + 3) * pb)) != EGR_OK) return rc;
        }
        {
            I8LmStep g = q;                                   // head and integer log-likelihood
            g.cols = 256; g.X0 = B.x; g.W0 = M->head; g.K0 = D; g.layer_id0 = 1001u;
            if ((rc = lm_plan_build(4, g, plan0 + (size_t)(4 * Lyr) * pb)) != EGR_OK) return rc;
        }
        const NoiseKey emb_key = make_noise_key(M->seed, 1000u);
        for (int pos = 0; pos + 1 < seq_len; ++pos) {
            lm_embed_ln256_kernel<<<gwarp, 256, 0, st>>>(B.emb_rows, tokens, seq_len, pos, member_seq, N, M->flags, emb_key,
                                                         M->sigma_shift, M->noise_table, mask, Lyr > 0 ? M->ln1 : M->ln_out,
                                                         2 * d, B.y, B.x);
            for (int k = 0; k < 4 * Lyr + 1; ++k)
                if ((rc = lm_plan_launch(plan0 + (size_t)k * pb, pos, st)) != EGR_OK) return rc;
        }
        return cuda_ok(cudaGetLastError());
    }

    for (int pos = 0; pos + 1 < seq_len; ++pos) {
        lm_embed_kernel<<<g16, 256, 0, st>>>(M->emb_t, tokens, seq_len, pos, member_seq, N, D, M->flags,
                                             make_noise_key(M->seed, 1000u), M->sigma_shift, M->noise_table, mask, B.y);
        for (int i = 0; i < Lyr; ++i) {
            int8_t *s_i = state + (int64_t)i * ND;
            const int64_t DD = (int64_t)D * D;
            const uint32_t id = 16u * (uint32_t)i;
            lm_ln_kernel<<<gwarp, 256, 0, st>>>(M->ln1 + (int64_t)i * D, B.y, N, D, 2 * d, B.x);
            if ((rc = pm(B.x, M->Wf + i * DD, D, D, id + 0, B.a)) != EGR_OK) return rc;
            if ((rc = pm(s_i, M->Uf + i * DD, D, D, id + 1, B.b)) != EGR_OK) return rc;
            lm_gate_f_kernel<<<g16, 256, 0, st>>>(B.a, B.b, M->bf + (int64_t)i * D, s_i, M->lut_sigma, ND, D, B.f, B.fh);
            if ((rc = pm(B.x, M->Wh + i * DD, D, D, id + 2, B.a)) != EGR_OK) return rc;
            if ((rc = pm(B.fh, M->Uh + i * DD, D, D, id + 3, B.b)) != EGR_OK) return rc;
            lm_gate_h_kernel<<<g16, 256, 0, st>>>(B.a, B.b, M->bh + (int64_t)i * D, B.f, M->lut_phi, ND, D, s_i, B.y);
            lm_ln_kernel<<<gwarp, 256, 0, st>>>(M->ln2 + (int64_t)i * D, B.y, N, D, 2 * d, B.x);
            if ((rc = pm(B.x, M->mlp1 + i * 4 * DD, D, 4 * D, id + 4, B.h1)) != EGR_OK) return rc;
            if ((rc = pm(B.h1, M->mlp2 + i * 4 * DD, 4 * D, D, id + 5, B.y2)) != EGR_OK) return rc;
            lm_residual_kernel<<<g16, 256, 0, st>>>(B.y2, ND, B.y);
        }
        lm_ln_kernel<<<gwarp, 256, 0, st>>>(M->ln_out, B.y, N, D, 2 * d, B.x);
        if ((rc = pm(B.x, M->head, D, 256, 1001u, B.logits)) != EGR_OK) return rc;
        lm_loglik_kernel<<<gwarp, 256, 0, st>>>(B.logits, tokens, seq_len, pos, member_seq, N, fitness);
    }
    return cuda_ok(cudaGetLastError());
}

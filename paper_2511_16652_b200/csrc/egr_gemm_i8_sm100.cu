// int8 tensor-core path for sm_100a ("EGG Pretraining with Integer EGGROLL"): the integer perturbed matmul
//   y_j = sat127( (sum_l x_l W[j][l] + ((t * A_p[j]) >> sigma_shift)) >> out_shift ),  t = sign * sum_l x_l B_p[l]
// on tcgen05.mma.kind::i8 (int8 x int8 -> int32 in tensor memory), CTA pairs as in the bf16 kernel, with the
// element-wise steps of the recurrent LM fused into the epilogue when the layer is exactly one tile wide (D = 256):
//   PM      y = pm(x, W)                                              any shape
//   GATE_F  f = lut[sat(pm(x,Wf) + pm(s,Uf) + bf)], fh = sat(((f+127) s) >> 8)                two accumulators
//   GATE_H  hh = lut[sat(pm(x,Wh) + pm(fh,Uh) + bh)], h = sat(s + sat(((f+127)(hh-s)) >> 8)),
//           s <- h, y <- sat(h + y), x <- LN(ln_w, y)                                         two accumulators
//   MLP2    y <- sat(pm(h1, W) + y), x <- LN(ln_w, y)
//   HEAD    logits = pm(x, W); fitness += z[t'] - LOG2(sum_v EXP2[z_v]), z = logits + 128
//   UPDATE  E = At Bt^T (the staged, fitness-signed factors); where |E| >= threshold W moves one bin ("Parameter Update")
// The skinny dot products t are computed by the epilogue warps themselves, for their own rows, while the tensor
// cores run the main loop; the threads that share a row (one per column part, four by default) exchange partial results through
// shared memory.  All arithmetic is integer and bit-exact.  Every wait is bounded.
// lm_seq_sm100_kernel chains these modes for a whole sequence in one launch (see the comment above it).
#include <cuda.h>

#include <mutex>

#include <new>

#include "egr_device.cuh"
#include "egr_internal.h"
#include "egr_tc.cuh"

namespace egr {

namespace {

constexpr int BM = 128, PAIR_M = 256, BN = 256, BNH = 128;
constexpr int BK = 128;          // int8 elements per stage row = 128 bytes = one swizzle span
constexpr int UMMA_K = 32;       // K per tcgen05.mma for 8-bit operands
constexpr int MAX_STAGES = 6;
// TMA stages per mode: the dual-GEMM and row-wise LM modes trade two stages for the staged A slices of two GEMMs
__host__ __device__ constexpr int stages_for(int mode) { return (mode == 0 || mode == 5) ? 5 : 4; }
__host__ __device__ constexpr int gemms_for(int mode) { return (mode == 1 || mode == 2) ? 2 : 1; }
constexpr int A_STAGE_BYTES = BM * BK, B_STAGE_BYTES = BNH * BK, STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int TMEM_COLS = 512;
#ifndef EGR_I8_EPI_WARPS
#define EGR_I8_EPI_WARPS 16
#endif
// Epilogue warps: PARTS per TMEM lane quarter, each owning CP 32-column chunks of the 256-column tile.  The LM
// launches are one tile deep per SM, i.e. a single latency chain per thread, so more (and shorter) threads per row
// hide more of it.
constexpr int EPI_WARPS = EGR_I8_EPI_WARPS, EPI_THREADS = EPI_WARPS * 32;
constexpr int PARTS = EPI_WARPS / 4, CP = 8 / PARTS;
static_assert(PARTS == 2 || PARTS == 4, "8 or 16 epilogue warps");
constexpr int NUM_THREADS = 32 * (2 + EPI_WARPS);
// skinny products t [tile parity][gemm][row], row sums [part][row], target z [part][row]
constexpr int XCHG_INTS = 2 * (2 * BM) + PARTS * BM + PARTS * BM;
constexpr int RPW = 32 / PARTS;      // rows of its lane quarter each epilogue warp takes in the skinny pass
// copies of the small tables the LM modes index per element: lut, bias, ln_w (256 bytes each), EXP2 (256 ints)
constexpr int TAB_BYTES = 3 * 256 + 256 * 4;
// A slices of the 128 rows of a tile: 256 bytes from a 16-byte-aligned start, one bulk copy per row and GEMM
constexpr int ASLICE_ROW_BYTES = 272;
__host__ __device__ constexpr int aslice_bytes(int mode) { return gemms_for(mode) * BM * ASLICE_ROW_BYTES; }
__host__ __device__ constexpr int smem_bytes_for(int mode)
{
    return stages_for(mode) * STAGE_BYTES + 1024 + 256 + XCHG_INTS * 4 + TAB_BYTES + aslice_bytes(mode);
}
static_assert(smem_bytes_for(0) <= 227 * 1024 && smem_bytes_for(1) <= 227 * 1024, "shared memory budget");

__device__ __forceinline__ int sat127(int v) { return max(-127, min(127, v)); }

// named barrier over the epilogue warps only, with an OR-reduction of a per-thread flag
__device__ __forceinline__ bool epi_any(bool flag)
{
    uint32_t out;
    asm volatile(
        "{\n.reg .pred p, q;\n"
        "setp.ne.u32 q, %1, 0;\n"
        "barrier.cta.red.or.pred p, 1, %2, q;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(out) : "r"((uint32_t)flag), "r"(EPI_THREADS) : "memory");
    return out != 0;
}
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, %0;" ::"r"(EPI_THREADS) : "memory"); }

// Skinny products t = sum_l x[l] * table[(off + l) mod size] for NR rows with the whole warp on each row: lane w takes words w, w + 32, ... of a row and of its
// table slice, so every load instruction touches consecutive addresses (one row per lane would cost 32 cache lines
// per instruction and is bound by the L1 tag rate).  All loads of a 128-byte step of all NR rows are issued before
// any is used: the pass costs a few memory round trips instead of one per row.  off[j] = table offset of row j,
// rows at or beyond n_valid give 0.  Results are returned to all lanes.
template <int NR>
__device__ __forceinline__ void skinny_dot_rows_warp(const int8_t *__restrict__ x0, int64_t ldx, int n_valid, int K,
                                                     const uint32_t (&off)[NR], const uint32_t *__restrict__ t32,
                                                     uint32_t wmask, int lane, int (&out)[NR])
{
#pragma unroll
    for (int j = 0; j < NR; ++j) out[j] = 0;
    const int words = K >> 2;
    if ((K & 7) == 0 && (ldx & 7) == 0 && (reinterpret_cast<uintptr_t>(x0) & 7) == 0) {
        // two words per lane and trip (one 64-bit load of x, three table words): half as many memory round trips
        const int pairs = K >> 3;
        for (int p0 = 0; p0 < pairs; p0 += 32) {
            const int pw = p0 + lane;
            int2 xv[NR];
            uint32_t t0[NR], t1[NR], t2[NR];
#pragma unroll
            for (int j = 0; j < NR; ++j) {
                const bool in = (pw < pairs) && (j < n_valid);
                const uint32_t base = (off[j] >> 2) + 2u * (uint32_t)pw;
                xv[j] = in ? __ldcg(reinterpret_cast<const int2 *>(x0 + j * ldx + 8 * pw)) : make_int2(0, 0);   // L2: another warp may have written it
                t0[j] = in ? __ldg(t32 + (base & wmask)) : 0u;
                t1[j] = in ? __ldg(t32 + ((base + 1u) & wmask)) : 0u;
                t2[j] = in ? __ldg(t32 + ((base + 2u) & wmask)) : 0u;
            }
#pragma unroll
            for (int j = 0; j < NR; ++j) {
                const uint32_t sh = (off[j] & 3u) * 8u;
                out[j] = __dp4a(xv[j].x, (int)__funnelshift_r(t0[j], t1[j], sh), out[j]);
                out[j] = __dp4a(xv[j].y, (int)__funnelshift_r(t1[j], t2[j], sh), out[j]);
            }
        }
#pragma unroll
        for (int j = 0; j < NR; ++j)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) out[j] += __shfl_xor_sync(0xffffffffu, out[j], o);
        return;
    }
    for (int w0 = 0; w0 < words; w0 += 32) {
        const int w = w0 + lane;
        int xv[NR];
        uint32_t t0[NR], t1[NR];
#pragma unroll
        for (int j = 0; j < NR; ++j) {
            const bool in = (w < words) && (j < n_valid);
            const uint32_t base = (off[j] >> 2) + (uint32_t)w;
            xv[j] = in ? __ldcg(reinterpret_cast<const int *>(x0 + j * ldx + 4 * w)) : 0;
            t0[j] = in ? __ldg(t32 + (base & wmask)) : 0u;
            t1[j] = in ? __ldg(t32 + ((base + 1u) & wmask)) : 0u;
        }
#pragma unroll
        for (int j = 0; j < NR; ++j) out[j] = __dp4a(xv[j], (int)__funnelshift_r(t0[j], t1[j], (off[j] & 3u) * 8u), out[j]);
    }
#pragma unroll
    for (int j = 0; j < NR; ++j)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) out[j] += __shfl_xor_sync(0xffffffffu, out[j], o);
}

struct I8Args {
    // problem
    int64_t rows; int cols; int K0, K1;            // K1 = 0 for single-GEMM modes
    const int8_t *X0, *X1; int64_t ldx0, ldx1;     // row operands as plain pointers (for the skinny dots)
    uint32_t flags; int T; int mbase; NoiseKey key0, key1;
    const int8_t *table; uint32_t mask; int sigma_shift, out_shift0, out_shift1;
    // PM
    int8_t *Y; int64_t ldy;
    // LM modes (D = 256)
    const int8_t *bias, *lut, *ln_w;
    int8_t *s, *y, *x, *f, *fh;                    // [rows][256]
    const uint8_t *tokens; const int32_t *member_seq; int seq_len, pos; int32_t *fitness;
    const int *exp2_tab, *frac_tab;
    int ln_shift;                                  // 2d
    const int2 *aux;                               // optional: per row (t, off_A) from a prepass; else computed here
    int32_t threshold; int32_t *E_out;             // UPDATE: Y / ldy are W and its pitch, E_out (nullable) is dense [rows][cols]
    int stage_a;                                   // A slices go through shared memory (table 16-byte aligned, >= 512 bytes)
    int *status;
};

struct Pert { int t; uint32_t off_a; };

// 1-D bulk copy global -> this CTA's shared memory, completion bytes on an mbarrier of this CTA
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ void load32(const int8_t *p, int (&v)[32])
{
    const int4 a = reinterpret_cast<const int4 *>(p)[0], b = reinterpret_cast<const int4 *>(p)[1];
    const int w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = (int)(int8_t)((w[i >> 2] >> (8 * (i & 3))) & 0xff);
}
__device__ __forceinline__ void store32(int8_t *p, const int (&v)[32])
{
    int w[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
        w[i] = (v[4 * i] & 0xff) | ((v[4 * i + 1] & 0xff) << 8) | ((v[4 * i + 2] & 0xff) << 16) | ((v[4 * i + 3] & 0xff) << 24);
    reinterpret_cast<int4 *>(p)[0] = make_int4(w[0], w[1], w[2], w[3]);
    reinterpret_cast<int4 *>(p)[1] = make_int4(w[4], w[5], w[6], w[7]);
}

// ---- the same helpers for W = 16 or 32 consecutive columns (the LM modes walk their columns in steps of 16: a
// quarter of the straight-line code of a 2 x 32 unrolled epilogue, which these one-tile-deep launches fetch afresh)
template <int W>
__device__ __forceinline__ void tc_ld_cols(uint32_t taddr, uint32_t (&v)[W])
{
    static_assert(W == 16 || W == 32, "16 or 32 columns");
    if constexpr (W == 32) {
        tc_ld_32x32(taddr, v);
    } else {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
            "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
              "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
            : "r"(taddr) : "memory");
    }
}

template <int W>
__device__ __forceinline__ void pm_cols(const uint32_t (&acc)[W], const Pert &pt, int col0, const uint32_t *t32, uint32_t wmask,
                                        int sigma_shift, int out_shift, bool perturb, int (&out)[W])
{
    uint32_t tw[W / 4 + 1];
    const uint32_t o = pt.off_a + (uint32_t)col0;
    const uint32_t sh = (o & 3u) * 8u;
    if (perturb) {
#pragma unroll
        for (int i = 0; i < W / 4 + 1; ++i) tw[i] = __ldg(t32 + (((o >> 2) + (uint32_t)i) & wmask));
    }
#pragma unroll
    for (int w = 0; w < W / 4; ++w) {
        const uint32_t aw = perturb ? __funnelshift_r(tw[w], tw[w + 1], sh) : 0u;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int a = (int)(int8_t)((aw >> (8 * b)) & 0xffu);
            const int pert = perturb ? ((pt.t * a) >> sigma_shift) : 0;
            out[4 * w + b] = sat127(((int)acc[4 * w + b] + pert) >> out_shift);
        }
    }
}

template <int W>
__device__ __forceinline__ void pm_cols_staged(const uint32_t (&acc)[W], int t, const uint32_t *sl, uint32_t o, int sigma_shift,
                                               int out_shift, int (&out)[W])
{
    uint32_t tw[W / 4 + 1];
    const uint32_t sh = (o & 3u) * 8u;
#pragma unroll
    for (int i = 0; i < W / 4 + 1; ++i) tw[i] = sl[(o >> 2) + (uint32_t)i];
#pragma unroll
    for (int w = 0; w < W / 4; ++w) {
        const uint32_t aw = __funnelshift_r(tw[w], tw[w + 1], sh);
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int a = (int)(int8_t)((aw >> (8 * b)) & 0xffu);
            out[4 * w + b] = sat127(((int)acc[4 * w + b] + ((t * a) >> sigma_shift)) >> out_shift);
        }
    }
}

template <int W>
__device__ __forceinline__ void load_cols(const int8_t *p, int (&v)[W])
{
    int w[W / 4];
#pragma unroll
    for (int q = 0; q < W / 16; ++q) {
        const int4 a = reinterpret_cast<const int4 *>(p)[q];
        w[4 * q] = a.x; w[4 * q + 1] = a.y; w[4 * q + 2] = a.z; w[4 * q + 3] = a.w;
    }
#pragma unroll
    for (int i = 0; i < W; ++i) v[i] = (int)(int8_t)((w[i >> 2] >> (8 * (i & 3))) & 0xff);
}
// the same from global memory that other threads of the running kernel may have written: read at L2, never through
// the non-coherent path
template <int W>
__device__ __forceinline__ void load_cols_g(const int8_t *p, int (&v)[W])
{
    int w[W / 4];
#pragma unroll
    for (int q = 0; q < W / 16; ++q) {
        const int4 a = __ldcg(reinterpret_cast<const int4 *>(p) + q);
        w[4 * q] = a.x; w[4 * q + 1] = a.y; w[4 * q + 2] = a.z; w[4 * q + 3] = a.w;
    }
#pragma unroll
    for (int i = 0; i < W; ++i) v[i] = (int)(int8_t)((w[i >> 2] >> (8 * (i & 3))) & 0xff);
}
template <int W>
__device__ __forceinline__ void store_cols(int8_t *p, const int (&v)[W])
{
    int w[W / 4];
#pragma unroll
    for (int i = 0; i < W / 4; ++i)
        w[i] = (v[4 * i] & 0xff) | ((v[4 * i + 1] & 0xff) << 8) | ((v[4 * i + 2] & 0xff) << 16) | ((v[4 * i + 3] & 0xff) << 24);
#pragma unroll
    for (int q = 0; q < W / 16; ++q) reinterpret_cast<int4 *>(p)[q] = make_int4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
}

struct I8Args;
__device__ __forceinline__ void update_chunk(const I8Args &ar, int64_t row, int col0, const uint32_t (&acc)[32]);

enum { MODE_PM = 0, MODE_GATE_F = 1, MODE_GATE_H = 2, MODE_MLP2 = 3, MODE_HEAD = 4, MODE_UPDATE = 5 };

// Tile walked at step `it` by a CTA pair.  Tiles are dealt round-robin, except for layers wider than one tile whose
// skinny products are computed in this kernel (no prepass): those are walked row tile by row tile, so that a pair keeps
// its rows for all column tiles and computes their products once.
__device__ __forceinline__ bool tile_at(int64_t it, int64_t cluster_id, int64_t num_clusters, int64_t tiles_m, int tiles_n,
                                        bool by_rows, int64_t &tm, int &tn)
{
    // (64-bit divisions are subroutines of several hundred cycles: one 32-bit division whenever the numbers fit)
    const int64_t t = by_rows ? it : cluster_id + it * num_clusters;
    int64_t q;
    if (((uint64_t)t >> 32) == 0) {
        const uint32_t q32 = (uint32_t)t / (uint32_t)tiles_n;
        q = q32; tn = (int)((uint32_t)t - q32 * (uint32_t)tiles_n);
    } else {
        q = t / tiles_n; tn = (int)(t % tiles_n);
    }
    if (by_rows) {
        tm = cluster_id + q * num_clusters;
        return tm < tiles_m;
    }
    tm = q;
    return t < tiles_m * tiles_n;
}

// one-bin move for 32 consecutive columns of row `row`: W += sign(E) where |E| >= threshold, saturating at +-127
__device__ __forceinline__ void update_chunk(const I8Args &ar, int64_t row, int col0, const uint32_t (&acc)[32])
{
    int8_t *w = ar.Y + row * ar.ldy + col0;
    const bool full = col0 + 32 <= ar.cols;
    if (ar.E_out) {
        int32_t *e = ar.E_out + row * (int64_t)ar.cols + col0;
        if (full && (ar.cols & 3) == 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                reinterpret_cast<int4 *>(e)[i] = make_int4((int)acc[4 * i], (int)acc[4 * i + 1], (int)acc[4 * i + 2], (int)acc[4 * i + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) if (col0 + i < ar.cols) e[i] = (int)acc[i];
        }
    }
    const long long thr = (long long)ar.threshold;
    if (full && ((reinterpret_cast<uintptr_t>(w) & 15) == 0)) {
        int wv[32];
        load32(w, wv);
        bool moved = false;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int e = (int)acc[i];
            const long long mag = e < 0 ? -(long long)e : (long long)e;
            if (mag >= thr) { wv[i] = sat127(wv[i] + ((e > 0) - (e < 0))); moved = true; }
        }
        if (moved) store32(w, wv);
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if (col0 + i >= ar.cols) continue;
            const int e = (int)acc[i];
            const long long mag = e < 0 ? -(long long)e : (long long)e;
            if (mag >= thr) w[i] = (int8_t)sat127((int)w[i] + ((e > 0) - (e < 0)));
        }
    }
}

// Shared-memory areas and per-thread state of an epilogue warp
struct EpiCtx {
    int *t_row_all, *row_x, *zt_x;
    int8_t *lut_s, *bias_s, *lnw_s;
    int *exp2_s;
    uint8_t *aslice;
    uint64_t *tfull_bar, *tempty_bar, *aslice_bar;
    volatile int *abort_flag;
    uint32_t tmem_base, cta_rank;
    int lane, quarter, part, lrow;
    Pert pt[2];          // carried from the first column tile of a row tile to the following ones
    int sgn;
    uint32_t n_tiles;    // tiles processed so far (alternates the buffer of the skinny products)
    uint32_t n_aslice;   // completed phases of the slice barrier
};

// per-column and per-value tables of the LM modes (exactly 256 columns wide) into shared memory
template <int MODE>
__device__ __forceinline__ void epi_stage_tables(const I8Args &ar, const EpiCtx &cx)
{
    if (MODE == MODE_PM || MODE == MODE_UPDATE) return;
    const int e = threadIdx.x - 64;
    if (e < 256) {
        if (MODE == MODE_GATE_F || MODE == MODE_GATE_H) { cx.lut_s[e] = ar.lut[e]; cx.bias_s[e] = ar.bias[e]; }
        if (MODE == MODE_GATE_H || MODE == MODE_MLP2) cx.lnw_s[e] = ar.ln_w[e];
        if (MODE == MODE_HEAD) cx.exp2_s[e] = ar.exp2_tab[e];
    }
    epi_sync();
}

// One tile of the epilogue warps: skinny products and A slices while the main loop runs, then the accumulator(s) of
// TMEM slot `slot` (both halves in the dual modes) through the mode's element-wise steps.  `fresh` = the skinny
// products of these rows are not known yet (false for the later column tiles of a row tile).  Returns false when a
// bounded wait ran out.
template <int MODE>
__device__ __forceinline__ bool epi_tile(const I8Args &ar, EpiCtx &cx, int64_t tm, int tile_n, bool fresh, int slot,
                                         uint32_t slot_phase, int pos)
{
    constexpr bool kDual = (MODE == MODE_GATE_F || MODE == MODE_GATE_H);
    const int lane = cx.lane, quarter = cx.quarter, part = cx.part, lrow = cx.lrow;
    const uint32_t cta_rank = cx.cta_rank, tmem_base = cx.tmem_base;
    int *const t_row_all = cx.t_row_all, *const row_x = cx.row_x, *const zt_x = cx.zt_x;
    const int8_t *const lut_s = cx.lut_s, *const bias_s = cx.bias_s, *const lnw_s = cx.lnw_s;
    const int *const exp2_s = cx.exp2_s;
    uint8_t *const aslice = cx.aslice;
    uint64_t *const tfull_bar = cx.tfull_bar, *const tempty_bar = cx.tempty_bar, *const aslice_bar = cx.aslice_bar;
    volatile int *const abort_flag = cx.abort_flag;
    const uint32_t *t32 = reinterpret_cast<const uint32_t *>(ar.table);
    const uint32_t wmask = ar.mask >> 2;
    const bool perturb = !(ar.flags & EGR_NO_PERTURB);
    const int64_t band = tm * 2 + cta_rank;
    const int64_t row = band * BM + lrow;
    const bool live = row < ar.rows;
    const int tile_col0 = tile_n * BN;

    // ---- table offsets of this thread's row: one generator call per product
    int *t_row = t_row_all + (int)(cx.n_tiles & 1u) * (2 * BM);               // alternate buffers between consecutive tiles
    uint32_t off_b[2] = {0u, 0u};
    const bool own_dots = fresh && perturb && !ar.aux;               // the skinny products are computed here
    if (!fresh) {
        // nothing to do: pt and cx.sgn still hold this row's values
    } else if (perturb && ar.aux) {
        // a prepass already produced t (sign included) and the A-slice offset of every row
        if (live) { const int2 a = ar.aux[row]; cx.pt[0].t = a.x; cx.pt[0].off_a = (uint32_t)a.y; }
    } else if (perturb && live) {
        uint32_t p; float sign;
        member_noise(member_of(nullptr, ar.mbase, row, ar.T), ar.flags, p, sign);
        cx.sgn = sign < 0.f ? -1 : 1;
#pragma unroll
        for (int g = 0; g < (kDual ? 2 : 1); ++g) {
            const NoiseKey &key = g ? ar.key1 : ar.key0;
            const uint4 xw = philox4x32_10(0u, p, key.layer_id, kTagI8, key.k0, key.k1);
            cx.pt[g].off_a = xw.x & ar.mask;
            off_b[g] = xw.y & ar.mask;
        }
    }
    // ---- A slices of this tile's columns: one bulk copy per row and GEMM into shared memory, issued by the
    // part-0 thread that owns the row as soon as the offsets are known; they land while the main loop and the
    // skinny products run
    const bool staged = perturb && ar.stage_a != 0;
    uint32_t a_base[2] = {0u, 0u};                           // byte offset of the tile's first column in the row buffer
    if (staged) {
#pragma unroll
        for (int g = 0; g < (kDual ? 2 : 1); ++g) a_base[g] = ((cx.pt[g].off_a + (uint32_t)tile_col0) & ar.mask) & 15u;
        if (part == 0) {
            const uint32_t bar = smem_u32(aslice_bar);
            uint32_t src_off[2] = {0u, 0u};
            bool async_copy[2] = {false, false};
            uint32_t tx = 0;
#pragma unroll
            for (int g = 0; g < (kDual ? 2 : 1); ++g) {
                if (!live) continue;
                src_off[g] = ((cx.pt[g].off_a + (uint32_t)tile_col0) & ar.mask) & ~15u;
                if (src_off[g] + ASLICE_ROW_BYTES <= ar.mask + 1u) { async_copy[g] = true; tx += ASLICE_ROW_BYTES; }
                else {
                    // the slice wraps round the end of the table: copy it byte by byte (rare)
                    uint8_t *dst = aslice + (g * BM + lrow) * ASLICE_ROW_BYTES;
                    for (int i = 0; i < ASLICE_ROW_BYTES; ++i) dst[i] = (uint8_t)ar.table[(src_off[g] + (uint32_t)i) & ar.mask];
                }
            }
            // one arrival per warp with the warp's byte count (four arrivals per phase instead of 128)
            const uint32_t tx_warp = __reduce_add_sync(0xffffffffu, tx);
            if (lane == 0) { if (tx_warp) mbar_expect_tx(bar, tx_warp); else mbar_arrive(bar); }
            __syncwarp();
#pragma unroll
            for (int g = 0; g < (kDual ? 2 : 1); ++g)
                if (async_copy[g])
                    bulk_load_1d(smem_u32(aslice + (g * BM + lrow) * ASLICE_ROW_BYTES), ar.table + src_off[g], ASLICE_ROW_BYTES, bar);
        }
    }
    // ---- skinny dots while the main loop runs: the PARTS warps of a lane quarter split its 32 rows and
    // put the whole warp on one row at a time
    if (own_dots) {
#pragma unroll
        for (int g = 0; g < (kDual ? 2 : 1); ++g) {
            const int K = g ? ar.K1 : ar.K0;
            const int8_t *xbase = g ? ar.X1 : ar.X0;
            const int64_t ldx = g ? ar.ldx1 : ar.ldx0;
            // this warp's RPW rows of the quarter; the lane that owns a row holds its offset
            const int r_first = quarter * 32 + part * RPW;
            const int64_t row_first = band * BM + r_first;
            uint32_t ob[RPW];
#pragma unroll
            for (int j = 0; j < RPW; ++j) ob[j] = __shfl_sync(0xffffffffu, off_b[g], part * RPW + j);
            const int n_valid = (int)max((int64_t)0, min((int64_t)RPW, ar.rows - row_first));
            int tj[RPW];
            skinny_dot_rows_warp<RPW>(xbase + row_first * ldx, ldx, n_valid, K, ob, t32, wmask, lane, tj);
            if (lane < RPW) {
                int mine = 0;
#pragma unroll
                for (int j = 0; j < RPW; ++j) if (lane == j) mine = tj[j];
                t_row[g * BM + r_first + lane] = mine;
            }
        }
    }
    // uniform decision over all epilogue warps: did anybody fail to see the accumulator (or the slices)?
    bool ok = mbar_wait(smem_u32(&tfull_bar[slot]), slot_phase, abort_flag, ar.status, 4);
    if (ok && staged) ok = mbar_wait(smem_u32(aslice_bar), cx.n_aslice & 1u, abort_flag, ar.status, 6);
    if (epi_any(!ok)) return false;                                 // also publishes t_row
    const uint32_t *sl0 = reinterpret_cast<const uint32_t *>(aslice + lrow * ASLICE_ROW_BYTES);
    const uint32_t *sl1 = reinterpret_cast<const uint32_t *>(aslice + (BM + lrow) * ASLICE_ROW_BYTES);
    tc_fence_after();
    if (perturb && !ar.aux && fresh) {
#pragma unroll
        for (int g = 0; g < (kDual ? 2 : 1); ++g) cx.pt[g].t = cx.sgn * t_row[g * BM + lrow];
    }

    int row_acc = 0;               // sum|y| (LN modes) or sum EXP2 (HEAD)
    int zt = 0;                    // HEAD: z of the target byte if it falls in this part
    int tn = 0;
    if (MODE == MODE_HEAD && live)
        tn = ar.tokens[(int64_t)ar.member_seq[row] * ar.seq_len + pos + 1];

    // One copy of the body, walked in a loop: these epilogues are long straight-line code that every launch executes
    // once, and fetching it is a visible part of their time (the capture shows as many stall cycles for "no
    // instruction" as for memory in the gate modes).  The LM modes step through their columns 16 at a time, the
    // generic product and the update 32 at a time.
    constexpr int W = (MODE == MODE_PM || MODE == MODE_UPDATE) ? 32 : 16;
    constexpr int NSTEP = CP * (32 / W);
#pragma unroll 1
    for (int c = 0; c < NSTEP; ++c) {
        const int tcol = (part * NSTEP + c) * W;                 // first column of the step inside the tile
        const int col0 = tile_col0 + tcol;
        if (col0 < ar.cols) {
            uint32_t v0[W];
            const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
            tc_ld_cols<W>(tmem_base + lane_addr + (uint32_t)((kDual ? 0 : slot) * BN + tcol), v0);
            tc_wait_ld();
            if constexpr (MODE == MODE_UPDATE) {
                if (live) update_chunk(ar, row, col0, v0);
                continue;
            } else {
            int r0[W];
            if (staged) pm_cols_staged<W>(v0, cx.pt[0].t, sl0, a_base[0] + (uint32_t)tcol, ar.sigma_shift, ar.out_shift0, r0);
            else pm_cols<W>(v0, cx.pt[0], col0, t32, wmask, ar.sigma_shift, ar.out_shift0, perturb, r0);
            if constexpr (MODE == MODE_PM) {
                if (live) {
                    int8_t *out = ar.Y + row * ar.ldy + col0;
                    if (col0 + W <= ar.cols && (ar.ldy & 15) == 0) store_cols<W>(out, r0);
                    else
#pragma unroll
                        for (int i = 0; i < W; ++i) if (col0 + i < ar.cols) out[i] = (int8_t)r0[i];
                }
            } else if constexpr (MODE == MODE_HEAD) {
                if (live) {
#pragma unroll
                    for (int i = 0; i < W; ++i) {
                        row_acc += exp2_s[r0[i] + 128];
                        if (col0 + i == tn) zt = r0[i] + 128;
                    }
                }
            } else if constexpr (MODE == MODE_MLP2) {
                if (live) {
                    int yv[W];
                    load_cols_g<W>(ar.y + row * 256 + col0, yv);
#pragma unroll
                    for (int i = 0; i < W; ++i) { yv[i] = sat127(r0[i] + yv[i]); row_acc += abs(yv[i]); }
                    store_cols<W>(ar.y + row * 256 + col0, yv);
                }
            } else {
                uint32_t v1[W];
                tc_ld_cols<W>(tmem_base + lane_addr + (uint32_t)(BN + tcol), v1);
                tc_wait_ld();
                int r1[W];
                if (staged) pm_cols_staged<W>(v1, cx.pt[1].t, sl1, a_base[1] + (uint32_t)tcol, ar.sigma_shift, ar.out_shift1, r1);
                else pm_cols<W>(v1, cx.pt[1], col0, t32, wmask, ar.sigma_shift, ar.out_shift1, perturb, r1);
                if (live) {
                    int bv[W], sv[W];
                    load_cols<W>(bias_s + col0, bv);
                    load_cols_g<W>(ar.s + row * 256 + col0, sv);
                    if constexpr (MODE == MODE_GATE_F) {
                        int fv[W], fhv[W];
#pragma unroll
                        for (int i = 0; i < W; ++i) {
                            fv[i] = (int)lut_s[sat127(r0[i] + r1[i] + bv[i]) + 128];
                            fhv[i] = sat127(((fv[i] + 127) * sv[i]) >> 8);
                        }
                        store_cols<W>(ar.f + row * 256 + col0, fv);
                        store_cols<W>(ar.fh + row * 256 + col0, fhv);
                    } else {
                        int fv[W], yv[W];
                        load_cols_g<W>(ar.f + row * 256 + col0, fv);
                        load_cols_g<W>(ar.y + row * 256 + col0, yv);
#pragma unroll
                        for (int i = 0; i < W; ++i) {
                            const int hh = (int)lut_s[sat127(r0[i] + r1[i] + bv[i]) + 128];
                            const int h = sat127(sv[i] + sat127(((fv[i] + 127) * (hh - sv[i])) >> 8));
                            sv[i] = h;
                            yv[i] = sat127(h + yv[i]);
                            row_acc += abs(yv[i]);
                        }
                        store_cols<W>(ar.s + row * 256 + col0, sv);
                        store_cols<W>(ar.y + row * 256 + col0, yv);
                    }
                }
            }
            }
        }
    }
    // the accumulators have been read: hand them back before the row-wise tail
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&tempty_bar[slot]), 0));

    if (MODE == MODE_GATE_H || MODE == MODE_MLP2 || MODE == MODE_HEAD) {
        // row-wise tail: combine the column parts of every row through shared memory
        row_x[part * BM + lrow] = row_acc;
        if (MODE == MODE_HEAD) zt_x[part * BM + lrow] = zt;
        epi_sync();
        int total = 0;
#pragma unroll
        for (int q = 0; q < PARTS; ++q) total += row_x[q * BM + lrow];
        if (MODE == MODE_HEAD) {
            if (live && part == 0) {
                int z_target = 0;                                     // exactly one part holds it, the others add 0
#pragma unroll
                for (int q = 0; q < PARTS; ++q) z_target += zt_x[q * BM + lrow];
                const int e = 31 - __clz(total);
                const int mant = (int)((((long long)total << 8) >> e) & 0xff);
                ar.fitness[row] += z_target - (16 * (e - 4) + ar.frac_tab[mant]);
            }
        } else if (live) {
            const int mav = max(1, sat127(total >> ar.ln_shift));
            // (y w) / mav truncated toward zero, exactly, as one high multiply: |y w| <= 127^2 and
            // M = floor(2^32 / mav) + 1 (floor for powers of two) give floor(|n| / mav) = umulhi(|n|, M)
            const uint32_t rcp = (mav > 1) ? 0xffffffffu / (uint32_t)mav + 1u : 0u;
#pragma unroll 1
            for (int c = 0; c < NSTEP; ++c) {
                const int col0 = (part * NSTEP + c) * W;
                int wv[W], xv[W], yk[W];
                load_cols<W>(lnw_s + col0, wv);
                load_cols<W>(ar.y + row * 256 + col0, yk);    // this thread's own stores of a moment ago
#pragma unroll
                for (int i = 0; i < W; ++i) {
                    const int yv = yk[i];
                    const int n = yv * wv[i];
                    const int q = (mav > 1) ? (int)__umulhi((uint32_t)abs(n), rcp) : abs(n);
                    xv[i] = sat127(n < 0 ? -q : q);
                }
                store_cols<W>(ar.x + row * 256 + col0, xv);
            }
        }
        epi_sync();          // exchange buffers may be overwritten by the next tile
    }
    if (staged) { fence_async_smem(); epi_sync(); }      // the slice buffers are free for the next tile's copies
    if (staged) ++cx.n_aslice;
    ++cx.n_tiles;
    return true;
}

// Context of an epilogue thread from the addresses every kernel of this file lays out the same way: `xchg` = start of the
// exchange area (behind the stage ring and the barriers), `bars` = the barrier block
__device__ __forceinline__ EpiCtx make_epi_ctx(int *xchg, uint64_t *bars, uint32_t tmem_base, uint32_t cta_rank)
{
    EpiCtx cx;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int8_t *lut_s = reinterpret_cast<int8_t *>(xchg + XCHG_INTS);
    cx.t_row_all = xchg; cx.row_x = xchg + 2 * (2 * BM); cx.zt_x = cx.row_x + PARTS * BM;
    cx.lut_s = lut_s; cx.bias_s = lut_s + 256; cx.lnw_s = lut_s + 512; cx.exp2_s = reinterpret_cast<int *>(lut_s + 768);
    cx.aslice = reinterpret_cast<uint8_t *>(lut_s) + TAB_BYTES;
    cx.tfull_bar = bars + 2 * MAX_STAGES; cx.tempty_bar = bars + 2 * MAX_STAGES + 2; cx.aslice_bar = bars + 2 * MAX_STAGES + 4;
    cx.abort_flag = reinterpret_cast<volatile int *>(reinterpret_cast<uint32_t *>(bars + 2 * MAX_STAGES + 5) + 1);
    cx.tmem_base = tmem_base; cx.cta_rank = cta_rank;
    cx.lane = lane; cx.quarter = warp & 3; cx.part = (warp - 2) >> 2; cx.lrow = cx.quarter * 32 + lane;
    cx.pt[0] = Pert{0, 0u}; cx.pt[1] = Pert{0, 0u}; cx.sgn = 1; cx.n_tiles = 0; cx.n_aslice = 0;
    return cx;
}

// One phase of the kernel that chains all modes, out of line and with scalar arguments only: each mode keeps the
// register allocation it has in a kernel of its own, and nothing of the context lives in local memory.  n_col_tiles
// column tiles of row tile tm (four for the MLP up-projection, whose later tiles reuse the skinny products of the
// first); cnt0 / cnt1 = uses of the two accumulator slots so far, n_tiles / n_aslice = the running counts of EpiCtx.
template <int MODE>
__device__ __noinline__ bool epi_phase(const I8Args *__restrict__ ar, int *xchg, uint64_t *bars, uint32_t tmem_base, uint32_t cta_rank,
                                       int64_t tm, int n_col_tiles, uint32_t cnt0, uint32_t cnt1, uint32_t n_tiles,
                                       uint32_t n_aslice, int pos)
{
    EpiCtx cx = make_epi_ctx(xchg, bars, tmem_base, cta_rank);
    cx.n_tiles = n_tiles; cx.n_aslice = n_aslice;
    epi_stage_tables<MODE>(*ar, cx);
    for (int tn = 0; tn < n_col_tiles; ++tn) {
        const int slot = (MODE == MODE_PM) ? (tn & 1) : 0;
        const uint32_t ph = (slot ? cnt1 : cnt0) & 1u;
        if (slot) ++cnt1; else ++cnt0;
        if (!epi_tile<MODE>(*ar, cx, tm, tn, tn == 0, slot, ph, pos)) return false;
    }
    return true;
}

template <int MODE>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_i8_sm100_kernel(const __grid_constant__ CUtensorMap tmap_a0, const __grid_constant__ CUtensorMap tmap_b0,
                     const __grid_constant__ CUtensorMap tmap_a1, const __grid_constant__ CUtensorMap tmap_b1,
                     const I8Args ar)
{
    constexpr bool kDual = (MODE == MODE_GATE_F || MODE == MODE_GATE_H);
    constexpr int STAGES = stages_for(MODE);
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + STAGES * STAGE_BYTES);
    uint64_t *full_bar = bars, *empty_bar = bars + MAX_STAGES, *tfull_bar = bars + 2 * MAX_STAGES, *tempty_bar = bars + 2 * MAX_STAGES + 2;
    uint64_t *aslice_bar = bars + 2 * MAX_STAGES + 4;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * MAX_STAGES + 5);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    int *xchg = reinterpret_cast<int *>(smem + STAGES * STAGE_BYTES + 256);
    int *t_row_all = xchg;                       // [2 tile parities][2 gemms][BM]
    int *row_x = xchg + 2 * (2 * BM);            // [PARTS][BM]
    int *zt_x = row_x + PARTS * BM;              // [PARTS][BM]
    int8_t *lut_s = reinterpret_cast<int8_t *>(xchg + XCHG_INTS);      // 16-byte aligned: XCHG_INTS is a multiple of 4
    int8_t *bias_s = lut_s + 256, *lnw_s = lut_s + 512;
    int *exp2_s = reinterpret_cast<int *>(lut_s + 768);
    uint8_t *aslice = reinterpret_cast<uint8_t *>(lut_s) + TAB_BYTES;       // [gemm][BM][272], 16-byte aligned

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = cluster_ctarank();
    const int64_t cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
    const int tiles_n = (ar.cols + BN - 1) / BN;
    const int64_t tiles_m = (ar.rows + PAIR_M - 1) / PAIR_M;
    const int kb0 = (ar.K0 + BK - 1) / BK, kb1 = kDual ? (ar.K1 + BK - 1) / BK : 0;
    const bool by_rows = (MODE == MODE_PM) && tiles_n > 1 && !ar.aux && !(ar.flags & EGR_NO_PERTURB);

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(smem_u32(&full_bar[i]), 1); mbar_init(smem_u32(&empty_bar[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&tfull_bar[i]), 1); mbar_init(smem_u32(&tempty_bar[i]), 2 * EPI_WARPS); }
        mbar_init(smem_u32(aslice_bar), BM / 32);   // one arrival per part-0 warp (the warps whose lanes own the rows)
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // accumulator slot of local tile `it`: single-GEMM modes alternate between the two halves of TMEM, dual modes
    // use both halves for one tile
    if (warp == 0) {
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool alive = true;
            int64_t tm; int tn;
            for (int64_t it = 0; alive && tile_at(it, cluster_id, num_clusters, tiles_m, tiles_n, by_rows, tm, tn); ++it) {
                const int row0 = (int)tm * PAIR_M + (int)cta_rank * BM;
                const int col0 = tn * BN + (int)cta_rank * BNH;
                for (int g = 0; g < (kDual ? 2 : 1) && alive; ++g) {
                    const CUtensorMap *ma = g ? &tmap_a1 : &tmap_a0, *mb = g ? &tmap_b1 : &tmap_b0;
                    const int nkb = g ? kb1 : kb0;
                    for (int kb = 0; kb < nkb; ++kb) {
                        if (!mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abort_flag, ar.status, 1)) { alive = false; break; }
                        const uint32_t leader_full = map_to_cta(smem_u32(&full_bar[stage]), 0);
                        if (cta_rank == 0) mbar_expect_tx(smem_u32(&full_bar[stage]), 2 * STAGE_BYTES);
                        const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES);
                        tma_load_2d_pair(sa, ma, kb * BK, row0, leader_full);
                        tma_load_2d_pair(sa + A_STAGE_BYTES, mb, kb * BK, col0, leader_full);
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && cta_rank == 0) {
            constexpr uint32_t idesc = make_idesc_i8(PAIR_M, BN);
            int stage = 0; uint32_t phase = 0;
            bool alive = true;
            int64_t tm; int tn;
            for (int64_t it = 0; alive && tile_at(it, cluster_id, num_clusters, tiles_m, tiles_n, by_rows, tm, tn); ++it) {
                // barrier slot: dual modes always use slot 0 (one tile in flight), single modes alternate
                const int slot = kDual ? 0 : (int)(it & 1);
                const uint32_t slot_phase = kDual ? (uint32_t)(it & 1) : (uint32_t)((it >> 1) & 1);
                if (!mbar_wait(smem_u32(&tempty_bar[slot]), slot_phase ^ 1u, abort_flag, ar.status, 2)) { alive = false; break; }
                tc_fence_after();
                for (int g = 0; g < (kDual ? 2 : 1) && alive; ++g) {
                    const uint32_t d_tmem = tmem_base + (uint32_t)((kDual ? g : slot) * BN);
                    const int nkb = g ? kb1 : kb0;
                    for (int kb = 0; kb < nkb; ++kb) {
                        if (!mbar_wait(smem_u32(&full_bar[stage]), phase, abort_flag, ar.status, 3)) { alive = false; break; }
                        tc_fence_after();
                        const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES);
                        const uint64_t da = make_kmajor_sw128_desc(sa), db = make_kmajor_sw128_desc(sa + A_STAGE_BYTES);
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k)
                            tc_mma_i8_pair(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) ? 1u : 0u);
                        tc_commit_pair(smem_u32(&empty_bar[stage]));
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
                if (alive) tc_commit_pair(smem_u32(&tfull_bar[slot]));
            }
        }
    } else {
        // ---------------- epilogue warps: TMEM lane quarter = warp % 4, column part = (warp - 2) / 4
        EpiCtx cx;
        cx.t_row_all = t_row_all; cx.row_x = row_x; cx.zt_x = zt_x;
        cx.lut_s = lut_s; cx.bias_s = bias_s; cx.lnw_s = lnw_s; cx.exp2_s = exp2_s; cx.aslice = aslice;
        cx.tfull_bar = tfull_bar; cx.tempty_bar = tempty_bar; cx.aslice_bar = aslice_bar; cx.abort_flag = abort_flag;
        cx.tmem_base = tmem_base; cx.cta_rank = cta_rank;
        cx.lane = lane; cx.quarter = warp & 3; cx.part = (warp - 2) >> 2; cx.lrow = cx.quarter * 32 + lane;
        cx.pt[0] = Pert{0, 0u}; cx.pt[1] = Pert{0, 0u}; cx.sgn = 1; cx.n_tiles = 0; cx.n_aslice = 0;
        epi_stage_tables<MODE>(ar, cx);
        int64_t tm; int tn;
        for (int64_t it = 0; tile_at(it, cluster_id, num_clusters, tiles_m, tiles_n, by_rows, tm, tn); ++it) {
            const int slot = kDual ? 0 : (int)(it & 1);
            const uint32_t slot_phase = kDual ? (uint32_t)(it & 1) : (uint32_t)((it >> 1) & 1);
            if (!epi_tile<MODE>(ar, cx, tm, tn, !(by_rows && tn > 0), slot, slot_phase, ar.pos)) break;
        }
    }

    tc_fence_before();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------- the recurrent LM, all positions in one launch
// At width 256 every step of the model is local to a row: a CTA pair that owns 256 rows (members) can walk all
// positions and layers for them without ever meeting another pair.  One launch then replaces 18 per position: per
// position the pair runs  E (embedding + layer norm, no product), and per layer  F, H (gate modes, two products
// each), P (MLP up, four column tiles), M (MLP down), and finally HEAD -- the same epilogues as the per-mode kernel
// above.  Activations go through global memory (L2) between phases: the epilogue warps write them with ordinary
// stores, order them before the asynchronous proxy with a proxy fence, and signal the CTA's `act` barrier; the TMA
// producer of the same CTA waits for it before loading them as the A operand of the next phase.  Every phase that
// feeds a product arrives exactly once and every product phase consumes exactly one arrival, so the barrier's
// parity never runs ahead.  Accumulator slots: 0 for F, H, M, HEAD and the even column tiles of P, 1 for the odd
// ones; the gate modes use both halves of tensor memory under slot 0's barriers.
constexpr int LM_MAXL = 8;
struct LmSeqParams {
    CUtensorMap a_x, a_fh, a_h1, a_s[LM_MAXL];
    CUtensorMap b_wf[LM_MAXL], b_uf[LM_MAXL], b_wh[LM_MAXL], b_uh[LM_MAXL], b_m1[LM_MAXL], b_m2[LM_MAXL], b_head;
    int64_t rows; int n_layers; uint32_t flags; uint64_t seed; int sigma_shift;
    const int8_t *table; uint32_t mask; int stage_a;
    int8_t *x, *y, *f, *fh, *h1, *state;                       // state: [n_layers][rows][256]
    const int8_t *bf, *bh, *ln1, *ln2, *ln_out, *lut_sigma, *lut_phi, *emb_rows;
    const uint8_t *tokens; const int32_t *member_seq; int seq_len; int32_t *fitness;
    const int *exp2_tab, *frac_tab; int ln_shift; int *status;
    // arguments of every product phase, in parameter (constant) space like those of the per-mode kernel: four per layer
    // (F, H, P, M), then HEAD
    I8Args phase[4 * LM_MAXL + 1];
};

constexpr int LM_PHASE_OFFSET = (smem_bytes_for(MODE_GATE_F) - 1024 + 15) / 16 * 16;      // behind the A slices (the 1024 is alignment slack)
constexpr int LM_SMEM_BYTES = LM_PHASE_OFFSET + 1024 + (int)sizeof(I8Args) * (4 * LM_MAXL + 1);
static_assert(LM_SMEM_BYTES <= 227 * 1024, "shared memory budget");

__global__ void __launch_bounds__(NUM_THREADS, 1)
lm_seq_sm100_kernel(const __grid_constant__ LmSeqParams P)
{
    constexpr int STAGES = 4;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + STAGES * STAGE_BYTES);
    uint64_t *full_bar = bars, *empty_bar = bars + MAX_STAGES, *tfull_bar = bars + 2 * MAX_STAGES, *tempty_bar = bars + 2 * MAX_STAGES + 2;
    uint64_t *aslice_bar = bars + 2 * MAX_STAGES + 4;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * MAX_STAGES + 5);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    uint64_t *act_bar = bars + 2 * MAX_STAGES + 6;
    int *xchg = reinterpret_cast<int *>(smem + STAGES * STAGE_BYTES + 256);
    // the phases' arguments in shared memory: the out-of-line phase functions read them through a pointer, and a pointer
    // into parameter space costs a trip to memory per field
    I8Args *phase_s = reinterpret_cast<I8Args *>(smem + LM_PHASE_OFFSET);
    static_assert(sizeof(I8Args) % 4 == 0, "copied as words");
    for (int w = threadIdx.x; w < (int)(sizeof(I8Args) / 4) * (4 * P.n_layers + 1); w += NUM_THREADS)
        reinterpret_cast<uint32_t *>(phase_s)[w] = reinterpret_cast<const uint32_t *>(P.phase)[w];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = cluster_ctarank();
    const int64_t cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
    const int64_t tiles_m = (P.rows + PAIR_M - 1) / PAIR_M;
    const int n_pos = P.seq_len - 1, NL = P.n_layers;

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(smem_u32(&full_bar[i]), 1); mbar_init(smem_u32(&empty_bar[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&tfull_bar[i]), 1); mbar_init(smem_u32(&tempty_bar[i]), 2 * EPI_WARPS); }
        mbar_init(smem_u32(aslice_bar), BM / 32);
        mbar_init(smem_u32(act_bar), 1);            // one arrival per phase, after the epilogue warps' barrier
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer: waits for the activations of each phase, then streams its k-blocks
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0, act_n = 0;
            bool alive = true;
            auto load_gemm = [&](const CUtensorMap *ma, const CUtensorMap *mb, int nkb, int row0, int col0) {
                for (int kb = 0; kb < nkb && alive; ++kb) {
                    if (!mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abort_flag, P.status, 1)) { alive = false; break; }
                    const uint32_t leader_full = map_to_cta(smem_u32(&full_bar[stage]), 0);
                    if (cta_rank == 0) mbar_expect_tx(smem_u32(&full_bar[stage]), 2 * STAGE_BYTES);
                    const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES);
                    tma_load_2d_pair(sa, ma, kb * BK, row0, leader_full);
                    tma_load_2d_pair(sa + A_STAGE_BYTES, mb, kb * BK, col0, leader_full);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            };
            auto wait_act = [&]() {
                if (alive && !mbar_wait_long(smem_u32(act_bar), act_n & 1u, abort_flag, P.status, 7)) alive = false;
                ++act_n;
            };
            for (int64_t tm = cluster_id; tm < tiles_m && alive; tm += num_clusters) {
                const int row0 = (int)tm * PAIR_M + (int)cta_rank * BM, colh = (int)cta_rank * BNH;
                for (int pos = 0; pos < n_pos && alive; ++pos) {
                    for (int i = 0; i < NL && alive; ++i) {
                        wait_act();                                              // F
                        load_gemm(&P.a_x, &P.b_wf[i], 2, row0, colh); load_gemm(&P.a_s[i], &P.b_uf[i], 2, row0, colh);
                        wait_act();                                              // H
                        load_gemm(&P.a_x, &P.b_wh[i], 2, row0, colh); load_gemm(&P.a_fh, &P.b_uh[i], 2, row0, colh);
                        wait_act();                                              // P
                        for (int tn = 0; tn < 4; ++tn) load_gemm(&P.a_x, &P.b_m1[i], 2, row0, tn * BN + colh);
                        wait_act();                                              // M
                        load_gemm(&P.a_h1, &P.b_m2[i], 8, row0, colh);
                    }
                    wait_act();                                                  // HEAD
                    load_gemm(&P.a_x, &P.b_head, 2, row0, colh);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA)
        if (lane == 0 && cta_rank == 0) {
            constexpr uint32_t idesc = make_idesc_i8(PAIR_M, BN);
            int stage = 0; uint32_t phase = 0, cnt0 = 0, cnt1 = 0;
            bool alive = true;
            auto mma_gemm = [&](uint32_t d_tmem, int nkb) {
                for (int kb = 0; kb < nkb && alive; ++kb) {
                    if (!mbar_wait(smem_u32(&full_bar[stage]), phase, abort_flag, P.status, 3)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES);
                    const uint64_t da = make_kmajor_sw128_desc(sa), db = make_kmajor_sw128_desc(sa + A_STAGE_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        tc_mma_i8_pair(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) ? 1u : 0u);
                    tc_commit_pair(smem_u32(&empty_bar[stage]));
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            };
            auto tile = [&](int slot, bool dual, int nkb0, int nkb1) {
                if (!alive) return;
                const uint32_t uses = slot ? cnt1 : cnt0;
                if (!mbar_wait_long(smem_u32(&tempty_bar[slot]), (uses & 1u) ^ 1u, abort_flag, P.status, 2)) { alive = false; return; }
                tc_fence_after();
                mma_gemm(tmem_base + (uint32_t)((dual ? 0 : slot) * BN), nkb0);
                if (dual) mma_gemm(tmem_base + (uint32_t)BN, nkb1);
                if (alive) tc_commit_pair(smem_u32(&tfull_bar[slot]));
                if (slot) ++cnt1; else ++cnt0;
            };
            for (int64_t tm = cluster_id; tm < tiles_m && alive; tm += num_clusters)
                for (int pos = 0; pos < n_pos && alive; ++pos) {
                    for (int i = 0; i < NL && alive; ++i) {
                        tile(0, true, 2, 2);                                     // F
                        tile(0, true, 2, 2);                                     // H
                        for (int tn = 0; tn < 4; ++tn) tile(tn & 1, false, 2, 0);// P
                        tile(0, false, 8, 0);                                    // M
                    }
                    tile(0, false, 2, 0);                                        // HEAD
                }
        }
    } else {
        // ---------------- epilogue warps
        uint32_t cnt0 = 0, cnt1 = 0, n_tiles = 0, n_aslice = 0;
        const uint32_t staged = (P.stage_a && !(P.flags & EGR_NO_PERTURB)) ? 1u : 0u;
        bool alive = true;
        // the phase's stores are ordered before the asynchronous proxy, all epilogue warps meet, one thread signals
        auto arrive_act = [&]() {
            asm volatile("fence.proxy.async;" ::: "memory");
            epi_sync();
            if (threadIdx.x == 64) mbar_arrive(smem_u32(act_bar));
        };
        for (int64_t tm = cluster_id; tm < tiles_m && alive; tm += num_clusters) {
            const int64_t band0 = (tm * 2 + cta_rank) * BM;
            for (int pos = 0; pos < n_pos && alive; ++pos) {
                // E: embedding and first layer norm of this CTA's rows, one warp per row (a row per lane would touch 32
                // cache lines with every load; tried, slower)
                {
                    const NoiseKey ekey = make_noise_key(P.seed, 1000u);
                    const int8_t *lnw = NL > 0 ? P.ln1 : P.ln_out;
                    for (int r = warp - 2; r < BM; r += EPI_WARPS) {
                        const int64_t row = band0 + r;
                        if (row < P.rows)
                            lm_embed_ln256_row(P.emb_rows, P.tokens, P.seq_len, pos, P.member_seq, row, P.flags, ekey, P.sigma_shift,
                                               P.table, P.mask, lnw, P.ln_shift, P.y, P.x, lane);
                    }
                    arrive_act();
                }
                for (int i = 0; i < NL && alive; ++i) {
                    // F: f, fh from x and s
                    alive = epi_phase<MODE_GATE_F>(phase_s + 4 * i + 0, xchg, bars, tmem_base, cta_rank, tm, 1, cnt0, cnt1, n_tiles, n_aslice, pos);
                    if (!alive) break;
                    ++cnt0; ++n_tiles; n_aslice += staged;
                    arrive_act();
                    // H: h, state, residual, second layer norm
                    alive = epi_phase<MODE_GATE_H>(phase_s + 4 * i + 1, xchg, bars, tmem_base, cta_rank, tm, 1, cnt0, cnt1, n_tiles, n_aslice, pos);
                    if (!alive) break;
                    ++cnt0; ++n_tiles; n_aslice += staged;
                    arrive_act();
                    // P: MLP up, four column tiles of the same rows
                    alive = epi_phase<MODE_PM>(phase_s + 4 * i + 2, xchg, bars, tmem_base, cta_rank, tm, 4, cnt0, cnt1, n_tiles, n_aslice, pos);
                    if (!alive) break;
                    cnt0 += 2; cnt1 += 2; n_tiles += 4; n_aslice += 4 * staged;
                    arrive_act();
                    // M: MLP down, residual, next layer norm
                    alive = epi_phase<MODE_MLP2>(phase_s + 4 * i + 3, xchg, bars, tmem_base, cta_rank, tm, 1, cnt0, cnt1, n_tiles, n_aslice, pos);
                    if (!alive) break;
                    ++cnt0; ++n_tiles; n_aslice += staged;
                    arrive_act();
                }
                if (!alive) break;
                // HEAD: logits and integer log-likelihood of the next byte
                alive = epi_phase<MODE_HEAD>(phase_s + 4 * NL, xchg, bars, tmem_base, cta_rank, tm, 1, cnt0, cnt1, n_tiles, n_aslice, pos);
                ++cnt0; ++n_tiles; n_aslice += staged;
            }
        }
    }

    tc_fence_before();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

template <int MODE>
int launch_mode(const CUtensorMap (&tm)[4], const I8Args &ar_in, cudaStream_t st)
{
    I8Args ar = ar_in;
    ar.stage_a = ((reinterpret_cast<uintptr_t>(ar.table) & 15) == 0 && ar.mask + 1u >= 512u) ? 1 : 0;
    static bool configured[64] = {};          // per device
    auto kern = gemm_i8_sm100_kernel<MODE>;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return EGR_ERR_CUDA;
    {
        std::lock_guard<std::mutex> cfg_lock(config_mutex());
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes_for(MODE)) != cudaSuccess) return EGR_ERR_CUDA;
            configured[dev] = true;
        }
    }
    const int sms = sm_count();
    if (sms < 2) return EGR_ERR_CUDA;
    const int64_t tiles = ((ar.rows + PAIR_M - 1) / PAIR_M) * ((ar.cols + BN - 1) / BN);
    const int64_t max_clusters = sms / 2;
    const unsigned clusters = (unsigned)(tiles < max_clusters ? tiles : max_clusters);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * clusters, 1, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes_for(MODE);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cuda_ok(cudaLaunchKernelEx(&cfg, kern, tm[0], tm[1], tm[2], tm[3], ar));
}

int log4_of(int n) { int d = 0; while ((1 << (2 * d)) < n) ++d; return d; }

}  // namespace

bool i8_tc_eligible(const void *X, int64_t ldx, const void *W, int64_t ldw)
{
    return ((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W)) & 15) == 0 && (ldx & 15) == 0 && (ldw & 15) == 0;
}

// generic perturbed matmul on the tensor cores (operands 16-byte aligned, pitches multiples of 16)
int launch_forward_i8_tc(const egr_layer &L, const int8_t *X, const int8_t *W, int sigma_shift, int out_shift,
                         const int8_t *table, uint32_t table_log2, int8_t *Y, const int2 *aux, int *status, cudaStream_t st)
{
    const int64_t R = (int64_t)L.n_members * L.rows_per_member;
    CUtensorMap tm[4];
    int rc = make_tmap_2d(&tm[0], CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, X, R, L.d_in, L.ldx, BK, BM);
    if (rc != EGR_OK) return rc;
    rc = make_tmap_2d(&tm[1], CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, W, L.d_out, L.d_in, L.ldw, BK, BNH);
    if (rc != EGR_OK) return rc;
    tm[2] = tm[0]; tm[3] = tm[1];
    I8Args ar = {};
    ar.rows = R; ar.cols = L.d_out; ar.K0 = L.d_in; ar.K1 = 0;
    ar.X0 = X; ar.ldx0 = L.ldx; ar.flags = L.flags; ar.T = L.rows_per_member; ar.mbase = L.member_base;
    ar.key0 = make_noise_key(L.seed, L.layer_id); ar.key1 = ar.key0;
    ar.table = table; ar.mask = (1u << table_log2) - 1u; ar.sigma_shift = sigma_shift; ar.out_shift0 = out_shift;
    ar.Y = Y; ar.ldy = L.ldy; ar.aux = aux; ar.status = status;
    return launch_mode<MODE_PM>(tm, ar, st);
}

// integer update: contraction of the staged factors with the one-bin epilogue
int launch_update_i8_tc(const egr_layer &L, const int8_t *At, const int8_t *Bt, int64_t p_pad, int8_t *W, int32_t threshold,
                        int32_t *E_out, int *status, cudaStream_t st)
{
    CUtensorMap tm[4];
    int rc = make_tmap_2d(&tm[0], CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, At, L.d_out, p_pad, p_pad, BK, BM);
    if (rc != EGR_OK) return rc;
    rc = make_tmap_2d(&tm[1], CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Bt, L.d_in, p_pad, p_pad, BK, BNH);
    if (rc != EGR_OK) return rc;
    tm[2] = tm[0]; tm[3] = tm[1];
    I8Args ar = {};
    ar.rows = L.d_out; ar.cols = L.d_in; ar.K0 = (int)p_pad; ar.K1 = 0;
    ar.flags = EGR_NO_PERTURB; ar.T = 1;
    ar.Y = W; ar.ldy = L.ldw; ar.threshold = threshold; ar.E_out = E_out; ar.status = status;
    return launch_mode<MODE_UPDATE>(tm, ar, st);
}

// One fused step of the recurrent LM at width 256 (see the mode list at the top of this file), prepared once and
// launched for every position: the tensor maps and arguments do not depend on the position, and looking the maps up
// anew for each of the 18 x 127 launches of a pass was a visible part of the host's time per launch.
namespace {
struct LmPlan { CUtensorMap tm[4]; I8Args ar; int mode; };
}  // namespace

size_t lm_plan_bytes() { return (sizeof(LmPlan) + 63) / 64 * 64; }

int lm_plan_build(int mode, const I8LmStep &q, void *plan_mem)
{
    LmPlan &pl = *new (plan_mem) LmPlan();
    int rc = cached_tmap_2d(&pl.tm[0], CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, q.X0, q.rows, q.K0, q.K0, BK, BM);
    if (rc != EGR_OK) return rc;
    rc = cached_tmap_2d(&pl.tm[1], CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, q.W0, q.cols, q.K0, q.K0, BK, BNH);
    if (rc != EGR_OK) return rc;
    pl.tm[2] = pl.tm[0]; pl.tm[3] = pl.tm[1];
    if (q.X1) {
        rc = cached_tmap_2d(&pl.tm[2], CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, q.X1, q.rows, q.K1, q.K1, BK, BM);
        if (rc != EGR_OK) return rc;
        rc = cached_tmap_2d(&pl.tm[3], CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, q.W1, q.cols, q.K1, q.K1, BK, BNH);
        if (rc != EGR_OK) return rc;
    }
    I8Args &ar = pl.ar;
    ar = I8Args{};
    ar.rows = q.rows; ar.cols = q.cols; ar.K0 = q.K0; ar.K1 = q.X1 ? q.K1 : 0;
    ar.X0 = q.X0; ar.X1 = q.X1; ar.ldx0 = q.K0; ar.ldx1 = q.K1;
    ar.flags = q.flags; ar.T = 1;
    ar.key0 = make_noise_key(q.seed, q.layer_id0); ar.key1 = make_noise_key(q.seed, q.layer_id1);
    ar.table = q.table; ar.mask = (1u << q.table_log2) - 1u; ar.sigma_shift = q.sigma_shift;
    ar.out_shift0 = 4 + log4_of(q.K0); ar.out_shift1 = q.X1 ? 4 + log4_of(q.K1) : 0;
    ar.Y = q.Y; ar.ldy = q.cols;
    ar.bias = q.bias; ar.lut = q.lut; ar.ln_w = q.ln_w; ar.s = q.s; ar.y = q.y; ar.x = q.x; ar.f = q.f; ar.fh = q.fh;
    ar.tokens = q.tokens; ar.member_seq = q.member_seq; ar.seq_len = q.seq_len; ar.pos = q.pos; ar.fitness = q.fitness;
    ar.exp2_tab = q.exp2_tab; ar.frac_tab = q.frac_tab; ar.ln_shift = q.ln_shift; ar.status = q.status;
    if (mode < MODE_PM || mode > MODE_HEAD) return EGR_ERR_BADARG;
    pl.mode = mode;
    return EGR_OK;
}

int lm_plan_launch(const void *plan_mem, int pos, cudaStream_t st)
{
    const LmPlan &pl = *static_cast<const LmPlan *>(plan_mem);
    I8Args ar = pl.ar;
    ar.pos = pos;
    switch (pl.mode) {
        case MODE_PM:     return launch_mode<MODE_PM>(pl.tm, ar, st);
        case MODE_GATE_F: return launch_mode<MODE_GATE_F>(pl.tm, ar, st);
        case MODE_GATE_H: return launch_mode<MODE_GATE_H>(pl.tm, ar, st);
        case MODE_MLP2:   return launch_mode<MODE_MLP2>(pl.tm, ar, st);
        case MODE_HEAD:   return launch_mode<MODE_HEAD>(pl.tm, ar, st);
    }
    return EGR_ERR_BADARG;
}

// the whole sequence of the width-256 LM in one launch; returns EGR_ERR_UNSUPPORTED when the model does not fit the
// kernel's parameter block (more than LM_MAXL layers), in which case the caller launches phase by phase
int launch_lm_seq(const I8LmSeq &q, cudaStream_t st)
{
    if (q.n_layers > LM_MAXL) return EGR_ERR_UNSUPPORTED;
    static LmSeqParams P;                                   // large: keep it off the stack (calls are serialised per process by the caller's stream use)
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    P = LmSeqParams{};
    auto amap = [&](CUtensorMap *m, const int8_t *X, int K) { return cached_tmap_2d(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, X, q.rows, K, K, BK, BM); };
    auto bmap = [&](CUtensorMap *m, const int8_t *W, int cols, int K) { return cached_tmap_2d(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, W, cols, K, K, BK, BNH); };
    int rc;
    if ((rc = amap(&P.a_x, q.x, 256)) != EGR_OK || (rc = amap(&P.a_fh, q.fh, 256)) != EGR_OK || (rc = amap(&P.a_h1, q.h1, 1024)) != EGR_OK) return rc;
    const int64_t ND = q.rows * 256, DD = 256 * 256;
    for (int i = 0; i < q.n_layers; ++i) {
        if ((rc = amap(&P.a_s[i], q.state + i * ND, 256)) != EGR_OK) return rc;
        if ((rc = bmap(&P.b_wf[i], q.Wf + i * DD, 256, 256)) != EGR_OK || (rc = bmap(&P.b_uf[i], q.Uf + i * DD, 256, 256)) != EGR_OK ||
            (rc = bmap(&P.b_wh[i], q.Wh + i * DD, 256, 256)) != EGR_OK || (rc = bmap(&P.b_uh[i], q.Uh + i * DD, 256, 256)) != EGR_OK ||
            (rc = bmap(&P.b_m1[i], q.mlp1 + i * 4 * DD, 1024, 256)) != EGR_OK || (rc = bmap(&P.b_m2[i], q.mlp2 + i * 4 * DD, 256, 1024)) != EGR_OK)
            return rc;
    }
    if ((rc = bmap(&P.b_head, q.head, 256, 256)) != EGR_OK) return rc;
    P.rows = q.rows; P.n_layers = q.n_layers; P.flags = q.flags; P.seed = q.seed; P.sigma_shift = q.sigma_shift;
    P.table = q.table; P.mask = (1u << q.table_log2) - 1u;
    P.stage_a = ((reinterpret_cast<uintptr_t>(q.table) & 15) == 0 && P.mask + 1u >= 512u) ? 1 : 0;
    P.x = q.x; P.y = q.y; P.f = q.f; P.fh = q.fh; P.h1 = q.h1; P.state = q.state;
    P.bf = q.bf; P.bh = q.bh; P.ln1 = q.ln1; P.ln2 = q.ln2; P.ln_out = q.ln_out; P.lut_sigma = q.lut_sigma; P.lut_phi = q.lut_phi;
    P.emb_rows = q.emb_rows; P.tokens = q.tokens; P.member_seq = q.member_seq; P.seq_len = q.seq_len; P.fitness = q.fitness;
    P.exp2_tab = q.exp2_tab; P.frac_tab = q.frac_tab; P.ln_shift = q.ln_shift; P.status = q.status;
    I8Args base = {};
    base.rows = q.rows; base.flags = q.flags; base.T = 1; base.mbase = 0;
    base.table = q.table; base.mask = P.mask; base.sigma_shift = q.sigma_shift; base.stage_a = P.stage_a;
    base.tokens = q.tokens; base.member_seq = q.member_seq; base.seq_len = q.seq_len; base.fitness = q.fitness;
    base.exp2_tab = q.exp2_tab; base.frac_tab = q.frac_tab; base.ln_shift = q.ln_shift; base.status = q.status;
    base.y = q.y; base.x = q.x; base.f = q.f; base.fh = q.fh;
    for (int i = 0; i < q.n_layers; ++i) {
        int8_t *s_i = q.state + i * ND;
        const uint32_t id = 16u * (uint32_t)i;
        I8Args &F = P.phase[4 * i + 0], &H = P.phase[4 * i + 1], &U = P.phase[4 * i + 2], &M = P.phase[4 * i + 3];
        F = base;                                                   // f, fh from x and s
        F.cols = 256; F.K0 = F.K1 = 256; F.X0 = q.x; F.X1 = s_i; F.ldx0 = F.ldx1 = 256;
        F.key0 = make_noise_key(q.seed, id + 0); F.key1 = make_noise_key(q.seed, id + 1); F.out_shift0 = F.out_shift1 = 8;
        F.bias = q.bf + i * 256; F.lut = q.lut_sigma; F.s = s_i;
        H = base;                                                   // h, state, residual, second layer norm
        H.cols = 256; H.K0 = H.K1 = 256; H.X0 = q.x; H.X1 = q.fh; H.ldx0 = H.ldx1 = 256;
        H.key0 = make_noise_key(q.seed, id + 2); H.key1 = make_noise_key(q.seed, id + 3); H.out_shift0 = H.out_shift1 = 8;
        H.bias = q.bh + i * 256; H.lut = q.lut_phi; H.s = s_i; H.ln_w = q.ln2 + i * 256;
        U = base;                                                   // MLP up
        U.cols = 1024; U.K0 = 256; U.X0 = q.x; U.ldx0 = 256;
        U.key0 = U.key1 = make_noise_key(q.seed, id + 4); U.out_shift0 = 8; U.Y = q.h1; U.ldy = 1024;
        M = base;                                                   // MLP down, residual, next layer norm
        M.cols = 256; M.K0 = 1024; M.X0 = q.h1; M.ldx0 = 1024;
        M.key0 = M.key1 = make_noise_key(q.seed, id + 5); M.out_shift0 = 9;
        M.ln_w = (i + 1 < q.n_layers) ? q.ln1 + (i + 1) * 256 : q.ln_out;
    }
    {
        I8Args &Hd = P.phase[4 * q.n_layers];                        // logits and integer log-likelihood
        Hd = base;
        Hd.cols = 256; Hd.K0 = 256; Hd.X0 = q.x; Hd.ldx0 = 256;
        Hd.key0 = Hd.key1 = make_noise_key(q.seed, 1001u); Hd.out_shift0 = 8;
    }

    static bool configured[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return EGR_ERR_CUDA;
    constexpr int kSmem = LM_SMEM_BYTES;
    {
        std::lock_guard<std::mutex> cfg_lock(config_mutex());
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(lm_seq_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) != cudaSuccess) return EGR_ERR_CUDA;
            configured[dev] = true;
        }
    }
    const int sms = sm_count();
    if (sms < 2) return EGR_ERR_CUDA;
    const int64_t tiles = (q.rows + PAIR_M - 1) / PAIR_M, max_clusters = sms / 2;
    const unsigned clusters = (unsigned)(tiles < max_clusters ? tiles : max_clusters);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * clusters, 1, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cuda_ok(cudaLaunchKernelEx(&cfg, lm_seq_sm100_kernel, P));
}

}  // namespace egr

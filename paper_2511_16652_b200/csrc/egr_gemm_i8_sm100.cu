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
#include <cuda.h>

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
                xv[j] = in ? *reinterpret_cast<const int2 *>(x0 + j * ldx + 8 * pw) : make_int2(0, 0);
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
            xv[j] = in ? *reinterpret_cast<const int *>(x0 + j * ldx + 4 * w) : 0;
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
    if (by_rows) {
        tm = cluster_id + (it / tiles_n) * num_clusters; tn = (int)(it % tiles_n);
        return tm < tiles_m;
    }
    const int64_t t = cluster_id + it * num_clusters;
    tm = t / tiles_n; tn = (int)(t % tiles_n);
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
        mbar_init(smem_u32(aslice_bar), BM);        // one arrival per row (the part-0 thread that owns it)
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
        const int quarter = warp & 3, part = (warp - 2) >> 2;
        const int lrow = quarter * 32 + lane;                       // row inside this CTA's band
        const uint32_t *t32 = reinterpret_cast<const uint32_t *>(ar.table);
        const uint32_t wmask = ar.mask >> 2;
        const bool perturb = !(ar.flags & EGR_NO_PERTURB);
        if (MODE != MODE_PM) {
            // the LM modes are exactly 256 columns wide: stage the per-column and per-value tables once
            const int e = threadIdx.x - 64;
            if (e < 256) {
                if (MODE == MODE_GATE_F || MODE == MODE_GATE_H) { lut_s[e] = ar.lut[e]; bias_s[e] = ar.bias[e]; }
                if (MODE == MODE_GATE_H || MODE == MODE_MLP2) lnw_s[e] = ar.ln_w[e];
                if (MODE == MODE_HEAD) exp2_s[e] = ar.exp2_tab[e];
            }
            epi_sync();
        }
        int64_t tm; int tn;
        Pert pt[2] = {{0, 0u}, {0, 0u}};
        int sgn = 1;
        for (int64_t it = 0; tile_at(it, cluster_id, num_clusters, tiles_m, tiles_n, by_rows, tm, tn); ++it) {
            const int slot = kDual ? 0 : (int)(it & 1);
            const uint32_t slot_phase = kDual ? (uint32_t)(it & 1) : (uint32_t)((it >> 1) & 1);
            const int64_t band = tm * 2 + cta_rank;
            const int64_t row = band * BM + lrow;
            const bool live = row < ar.rows;
            const int tile_col0 = tn * BN;
            const bool fresh = !(by_rows && tn > 0);      // a later column tile of the same rows reuses their products

            // ---- table offsets of this thread's row: one generator call per product
            int *t_row = t_row_all + (int)(it & 1) * (2 * BM);               // alternate buffers between consecutive tiles
            uint32_t off_b[2] = {0u, 0u};
            const bool own_dots = fresh && perturb && !ar.aux;               // the skinny products are computed here
            if (!fresh) {
                // nothing to do: pt and sgn still hold this row's values
            } else if (perturb && ar.aux) {
                // a prepass already produced t (sign included) and the A-slice offset of every row
                if (live) { const int2 a = ar.aux[row]; pt[0].t = a.x; pt[0].off_a = (uint32_t)a.y; }
            } else if (perturb && live) {
                uint32_t p; float sign;
                member_noise(ar.mbase + (int)(row / ar.T), ar.flags, p, sign);
                sgn = sign < 0.f ? -1 : 1;
#pragma unroll
                for (int g = 0; g < (kDual ? 2 : 1); ++g) {
                    const NoiseKey &key = g ? ar.key1 : ar.key0;
                    const uint4 xw = philox4x32_10(0u, p, key.layer_id, kTagI8, key.k0, key.k1);
                    pt[g].off_a = xw.x & ar.mask;
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
                for (int g = 0; g < (kDual ? 2 : 1); ++g) a_base[g] = ((pt[g].off_a + (uint32_t)tile_col0) & ar.mask) & 15u;
                if (part == 0) {
                    const uint32_t bar = smem_u32(aslice_bar);
                    uint32_t src_off[2] = {0u, 0u};
                    bool async_copy[2] = {false, false};
                    uint32_t tx = 0;
#pragma unroll
                    for (int g = 0; g < (kDual ? 2 : 1); ++g) {
                        if (!live) continue;
                        src_off[g] = ((pt[g].off_a + (uint32_t)tile_col0) & ar.mask) & ~15u;
                        if (src_off[g] + ASLICE_ROW_BYTES <= ar.mask + 1u) { async_copy[g] = true; tx += ASLICE_ROW_BYTES; }
                        else {
                            // the slice wraps round the end of the table: copy it byte by byte (rare)
                            uint8_t *dst = aslice + (g * BM + lrow) * ASLICE_ROW_BYTES;
                            for (int i = 0; i < ASLICE_ROW_BYTES; ++i) dst[i] = (uint8_t)ar.table[(src_off[g] + (uint32_t)i) & ar.mask];
                        }
                    }
                    if (tx) mbar_expect_tx(bar, tx); else mbar_arrive(bar);
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
            if (ok && staged) ok = mbar_wait(smem_u32(aslice_bar), (uint32_t)(it & 1), abort_flag, ar.status, 6);
            if (epi_any(!ok)) break;                                 // also publishes t_row
            const uint32_t *sl0 = reinterpret_cast<const uint32_t *>(aslice + lrow * ASLICE_ROW_BYTES);
            const uint32_t *sl1 = reinterpret_cast<const uint32_t *>(aslice + (BM + lrow) * ASLICE_ROW_BYTES);
            tc_fence_after();
            if (perturb && !ar.aux && fresh) {
#pragma unroll
                for (int g = 0; g < (kDual ? 2 : 1); ++g) pt[g].t = sgn * t_row[g * BM + lrow];
            }

            int row_acc = 0;               // sum|y| (LN modes) or sum EXP2 (HEAD)
            int zt = 0;                    // HEAD: z of the target byte if it falls in this part
            int tn = 0;
            if (MODE == MODE_HEAD && live)
                tn = ar.tokens[(int64_t)ar.member_seq[row] * ar.seq_len + ar.pos + 1];

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
                    if (staged) pm_cols_staged<W>(v0, pt[0].t, sl0, a_base[0] + (uint32_t)tcol, ar.sigma_shift, ar.out_shift0, r0);
                    else pm_cols<W>(v0, pt[0], col0, t32, wmask, ar.sigma_shift, ar.out_shift0, perturb, r0);
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
                            load_cols<W>(ar.y + row * 256 + col0, yv);
#pragma unroll
                            for (int i = 0; i < W; ++i) { yv[i] = sat127(r0[i] + yv[i]); row_acc += abs(yv[i]); }
                            store_cols<W>(ar.y + row * 256 + col0, yv);
                        }
                    } else {
                        uint32_t v1[W];
                        tc_ld_cols<W>(tmem_base + lane_addr + (uint32_t)(BN + tcol), v1);
                        tc_wait_ld();
                        int r1[W];
                        if (staged) pm_cols_staged<W>(v1, pt[1].t, sl1, a_base[1] + (uint32_t)tcol, ar.sigma_shift, ar.out_shift1, r1);
                        else pm_cols<W>(v1, pt[1], col0, t32, wmask, ar.sigma_shift, ar.out_shift1, perturb, r1);
                        if (live) {
                            int bv[W], sv[W];
                            load_cols<W>(bias_s + col0, bv);
                            load_cols<W>(ar.s + row * 256 + col0, sv);
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
                                load_cols<W>(ar.f + row * 256 + col0, fv);
                                load_cols<W>(ar.y + row * 256 + col0, yv);
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
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes_for(MODE)) != cudaSuccess) return EGR_ERR_CUDA;
        configured[dev] = true;
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

}  // namespace egr

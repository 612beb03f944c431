// bf16 tensor-core path for sm_100a: one persistent, warp-specialised TN GEMM (both operands K-major)
//   D[rows x cols] = A[rows x K] * B[cols x K]^T,  fp32 accumulation in tensor memory
// fed by TMA (128-byte swizzled tiles) and issued with tcgen05.mma, with three epilogues:
//   FORWARD  Y = acc + sign (sigma/sqrt r) sum_k s[rho][k] A_p[j][k]     (Section 4.2, right-hand side)
//   PLAIN    Y = acc                                                     (unperturbed inference)
//   UPDATE   W_master += scale * acc, optional bf16 shadow and dW copy   (boxed EGGROLL update)
//
// Two CTAs on neighbouring SMs form a cluster and work on one 256x256 output tile with
// tcgen05.mma.cta_group::2: each CTA stages its own 128 rows of A and its own 128 of the 256 rows of B (so every
// byte of an operand tile crosses L2 -> shared memory once per pair, not once per CTA), the leader CTA issues the
// MMAs for both, and each CTA ends up with its 128 x 256 fp32 slice of the accumulator in its own tensor memory.
// No cluster multicast loads are used: each CTA fetches what it stages.
//
// Roles inside a CTA: warp 0 = TMA producer, warp 1 = MMA issuer (leader CTA only) and TMEM owner,
// warps 2..9 = epilogue (each reads its own quarter of the 128 TMEM lanes and half of the tile's columns).
// Two accumulators live in TMEM so that the epilogue of one tile overlaps the main loop of the next.
// The FORWARD variant adds ten warps.  Most of them are "side" warps that compute the skinny products s = X B_p (warp
// shuffles, B_p regenerated in registers) while the tensor cores run: they claim groups of rows from a global counter,
// publish s through L2 and bump a per-band ready counter that the epilogue warps acquire before they touch a
// band.  Side warps wait for nothing, so a band can never depend on a CTA that is not running.
// Which warp does what in the forward follows from one measurement (time stamps per tile and role): the single thread
// that issues the MMAs needs its scheduler (warp index mod 4) to itself.  Next to noise-generating warps a tile's main
// loop took 43 K cycles instead of 34 K; see the comment at FWD_EXTRA_WARPS for the resulting layout.
//
// Every mbarrier wait is bounded: when a limit is hit the CTA records EGR_ERR_TIMEOUT in the workspace
// status word, raises a CTA-wide abort flag, drains and frees its TMEM.
#include <cuda.h>

#include "egr_device.cuh"
#include "egr_internal.h"
#include "egr_skinny.cuh"
#include "egr_tc.cuh"

namespace egr {

namespace {

constexpr int BM = 128;          // output rows per CTA (TMEM lanes); a CTA pair covers 256
constexpr int PAIR_M = 2 * BM;
constexpr int BN = 256;          // output columns per tile (TMEM columns per accumulator)
constexpr int BNH = BN / 2;      // rows of B staged by each CTA of the pair
constexpr int BK = 64;           // K elements per stage = 128 bytes of bf16 = one swizzle span
constexpr int UMMA_K = 16;       // K per tcgen05.mma for 16-bit operands
constexpr int MAX_STAGES = 6;
// TMA stages: the forward and the reduce-add update trade one stage for shared-memory buffers of their epilogues
__host__ __device__ constexpr int stages_for(int epi) { return (epi == 0 || epi == 3 || epi == 5) ? 5 : 6; }
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int B_STAGE_BYTES = BNH * BK * 2;
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int TMEM_COLS = 512;   // two accumulators of 256 columns
constexpr int EPI_WARPS = 8;                 // two per TMEM lane quarter, each taking half of the tile's columns
constexpr int EPI_PARTS = EPI_WARPS / 4;
constexpr int BASE_WARPS = 2 + EPI_WARPS;    // producer, MMA, epilogue warps
// The forward launches ten more warps (10 .. 19).  A warp's scheduler is fixed by its index (index mod 4), and the one
// thread that issues the MMAs (warp 1) loses tensor-pipe time whenever it queues behind arithmetic-heavy warps on its
// scheduler: with side warps and the noise-generating epilogue warps of lane quarter 1 next to it, a tile's main loop
// took 43 K cycles against 34 K unperturbed (4096 x 4096, rank 1, one token per member).  So for ranks below 4, where
// the tensor pipe is the bound, scheduler 1 only hosts threads that issue a few instructions per stage or chunk:
//   * warps 5 and 9 (quarter 1) only relay their accumulator chunks from tensor memory to shared memory; warps 10 and
//     11 (schedulers 2, 3) pick them up and do the quarter's epilogue arithmetic;
//   * warp 13 is the TMA producer (it, too, is one thread that must not wait for a scheduler slot), warp 17 idles at
//     the final barrier;
//   * warps 0, 12, 14, 15, 16, 18, 19 compute skinny products.
// With that the main loop is back at 33.6 K cycles per tile and the whole launch at 1.04 x the cycles of the
// unperturbed kernel (1.30 x before).  For ranks 4 and more the generator is the bound, every scheduler is needed, the
// roles are the plain ones and all ten extra warps are side warps.
constexpr int FWD_EXTRA_WARPS = 10;
__host__ __device__ constexpr bool relay_for(int epi, int rank) { return epi == 0 && rank < 4; }
constexpr int RELAY_BUF_BYTES = 32 * 32 * 4;                 // one 32 x 32 fp32 chunk
constexpr int RELAY_BYTES = 2 * 2 * RELAY_BUF_BYTES;         // two channels (column halves), double-buffered
// The last tile of a CTA pair has no main loop to hide behind, and by then the side warps, the producer warp and the
// idle warp have nothing left to do: warps 12 .. 19 (two per lane quarter of tensor memory) take the second half of
// every epilogue warp's chunks of that tile (quarter 1: of what warps 5 and 9 would have relayed).  Each has one
// staging slot behind the relay buffers.  They wait at a named hardware barrier at which warp 2 arrives once it has
// seen the last accumulator complete: a warp that has not followed the accumulator barriers' phases cannot tell their
// parities apart, and with eight warps polling an mbarrier of their own for most of a long launch every main loop was
// 4 % slower.  Warp 2 arrives exactly once on every path out of its loop, so the helpers cannot be left waiting.
constexpr int TAIL_WARP0 = 12, TAIL_WARPS = 8;
constexpr int SPIN_LIMIT = 1 << 22;   // polls of a band's ready counter before giving up
// Output staging for the TMA-store epilogue: every epilogue warp owns two slots of 32 rows x 32 bf16 columns
// (64 bytes per row, 64-byte swizzle), so that a slot is being written while the other one is being stored.
// (the update stages 32 x 32 fp32 blocks, 128 bytes per row with the 128-byte swizzle, for TMA reduce-add stores)
__host__ __device__ constexpr int store_slot_bytes(int epi) { return (epi == 3 || epi == 5) ? 32 * 128 : 32 * 64; }
__host__ __device__ constexpr int store_bytes(int epi) { return EPI_WARPS * 2 * store_slot_bytes(epi); }
constexpr int STORE_SLOT_BYTES = 32 * 64;
constexpr int BAR_BYTES = 1024;      // barriers, TMEM slot, flags (padded so that the staging stays 1024-byte aligned)
__host__ __device__ constexpr int smem_bytes_for(int epi)
{
    return stages_for(epi) * STAGE_BYTES + 1024 /*alignment slack*/ + BAR_BYTES + store_bytes(epi) +
           (epi == 0 ? RELAY_BYTES + TAIL_WARPS * STORE_SLOT_BYTES : 0);
}
static_assert(smem_bytes_for(0) <= 227 * 1024 && smem_bytes_for(3) <= 227 * 1024 && smem_bytes_for(5) <= 227 * 1024, "shared memory budget");

enum { EPI_FORWARD = 0, EPI_PLAIN = 1, EPI_UPDATE = 2, EPI_UPDATE_REDUCE = 3, EPI_UPDATE_FUSED = 4, EPI_UPDATE_FUSED_REDUCE = 5 };
// 3: update through TMA reduce-add stores; 4, 5: a contraction of several K-chunks in one launch, the factors staged by
// this kernel's own side warps into a ring of chunk buffers, with the register epilogue (4: dW_out or gradient only) or
// with reduce-add stores (5: what a caller's update runs)

struct EpiParams {
    // forward / plain
    void *Y; int64_t ldy; int y_f32; int y_tma;     // y_tma: bf16 output goes through shared memory and TMA stores
    const float *s; float coef; int T; int mbase; const int32_t *rowmap; uint32_t flags; NoiseKey key;
    // update
    float *Wm; int64_t ldw; __nv_bfloat16 *Wsh; float *dW; int64_t lddw; float scale; int dw_accumulate;
    // forward: skinny pass done by the side warps
    const __nv_bfloat16 *X; int64_t ldx; float *s_out; int *side_counter; int *ready;
    int split_rows;                                 // the first rows (a multiple of BM) are reduced in two K-halves each
    // forward through a quantised matrix: per-column scales (null = none), input scale, deviation of the scale noise
    const __nv_bfloat16 *col_scale; float x_scale; float sigma_s;
    // update in one launch: chunk c of the stacked factors lives in ring slot c % n_slots of At [rows][n_slots * kc] and
    // Bt [cols][n_slots * kc]; ready_u [chunk][factor][256-row band] counts staged items, loaded [chunk] counts the CTAs
    // whose loads of that chunk have landed (the slot may then be overwritten), done [tile] the epilogue warps that have
    // added their part of a chunk to the tile
    int n_chunks; int kc; int n_slots; int64_t K_total; const float *fitness; __nv_bfloat16 *At, *Bt; int64_t ldk;
    int *ready_u; int *loaded; int *done; int max_bands; int ipr;
    // forward that ends in a token log-likelihood instead of an output matrix: per-row targets, and per (column part,
    // row) the running maximum and the sum of exponentials of the part's logits; the target's logit per row
    const int32_t *targets; float2 *ll_part; float *ll_tgt;
    // common
    int64_t rows; int cols; int K;
    int *status;
};

// running maximum / sum of exponentials / target logit of one row over the chunks a warp has seen of it
struct LogLikState { float m, s, t; };

__host__ __device__ constexpr int threads_for(int epi) { return 32 * (BASE_WARPS + ((epi == 0 || epi == 4 || epi == 5) ? FWD_EXTRA_WARPS : 0)); }

// ---------------------------------------------------------------- epilogues (one thread = one output row, 32 columns)
// Rank-r term for 32 consecutive columns when aligned groups of G lanes (G rows) see the same noise index: the
// group generates each Philox block once (block b on group lane b % G) and hands the normals round with shuffles.
// G = 32 is a whole warp of rows of one member; G = 2 is an antithetic pair with one token per member.
template <int RANK, int G>
__device__ __forceinline__ void add_noise_shared(const EpiParams &ep, uint32_t p, uint32_t q0, float c,
                                                 const float (&sv)[RANK], float (&y)[32], int lane)
{
    constexpr int kBlocks = 32 * RANK / 4;
    constexpr int kBatch = (8 * G < kBlocks) ? 8 * G : kBlocks;        // blocks per batch: at most 8 per lane
    constexpr int kSlots = (kBatch + G - 1) / G;
    const int g = lane & (G - 1), base = lane & ~(G - 1);
#pragma unroll
    for (int b0 = 0; b0 < kBlocks; b0 += kBatch) {
        float z[kSlots][4];
#pragma unroll
        for (int sl = 0; sl < kSlots; ++sl) {
            const int b = b0 + sl * G + g;
            float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (sl * G + g < kBatch) z4 = noise_block_call<false>(ep.key, p, kTagA, q0 + (uint32_t)b);
            z[sl][0] = z4.x; z[sl][1] = z4.y; z[sl][2] = z4.z; z[sl][3] = z4.w;
        }
#pragma unroll
        for (int t = 0; t < 4 * kBatch; ++t) {
            const int bl = t >> 2;                                   // block inside the batch, compile-time
            const int el = 4 * b0 + t;
            const float v = __shfl_sync(0xffffffffu, z[bl / G][t & 3], base + (bl % G));
            y[el / RANK] = fmaf(c * sv[el % RANK], v, y[el / RANK]);
        }
    }
}

// The same for groups of eight or more rows, through shared memory instead of shuffles (one shuffle per normal and
// row made the shuffle unit the bound of short-K layers): lane g of a group generates blocks g, g + G, ... of a
// batch into the warp's staging slot, then every lane reads its group's normals back as broadcast 128-bit loads.
// `xbuf` holds 512 floats; group regions are padded by one block so that the groups' loads fall into different banks.
template <int RANK, int G>
__device__ __forceinline__ void add_noise_smem(const EpiParams &ep, uint32_t p, uint32_t q0, float c,
                                               const float (&sv)[RANK], float (&y)[32], int lane, float *xbuf)
{
    constexpr int kBlocks = 32 * RANK / 4;
    constexpr int kGroups = 32 / G;
    constexpr int kFit = (G == 32) ? 64 : (G == 16) ? 32 : 16;         // kGroups * (kFit + 1) blocks <= 128 blocks = 2 KiB
    constexpr int kBatch = (kBlocks < kFit) ? kBlocks : kFit;
    static_assert(kGroups * (kBatch + 1) * 16 <= STORE_SLOT_BYTES, "exchange buffer");
    const int g = lane & (G - 1);
    float4 *mine = reinterpret_cast<float4 *>(xbuf) + (lane / G) * (kBatch + 1);
#pragma unroll
    for (int b0 = 0; b0 < kBlocks; b0 += kBatch) {
        // lane g generates blocks g, g + G, ... of the batch, their generator chains in lock step
        if constexpr (kBatch >= G) noise_blocks_store<kBatch / G>(ep.key, p, kTagA, q0 + (uint32_t)(b0 + g), G, mine + g, G);
        else if (g < kBatch) noise_blocks_store<1>(ep.key, p, kTagA, q0 + (uint32_t)(b0 + g), G, mine + g, G);
        __syncwarp();
#pragma unroll
        for (int bl = 0; bl < kBatch; ++bl) {
            const float4 z4 = mine[bl];
            const float z[4] = {z4.x, z4.y, z4.z, z4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int el = 4 * (b0 + bl) + u;                   // compile-time after unrolling
                y[el / RANK] = fmaf(c * sv[el % RANK], z[u], y[el / RANK]);
            }
        }
        __syncwarp();
    }
}

// Multipliers of a quantised matrix for the four columns from col (a multiple of 4):
//   (s_x + a e_p[cols]) (s_j + a e_p[j]),  a = sign * sigma_s (0: no scale noise),
// e_p = the factor with the scale tag, one element per column and one more for the input scale.  Kept out of line so
// that the kernels that do not use it keep their register allocation.
__device__ __noinline__ float4 col_scale4(const __nv_bfloat16 *__restrict__ col_scale, int cols, int col, float x_scale,
                                          float a, NoiseKey key, uint32_t p)
{
    float sc[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) sc[i] = (col + i < cols) ? __bfloat162float(col_scale[col + i]) : 0.f;
    float xs = x_scale;
    if (a != 0.f) {
        const float4 z = noise_block<false>(key, p, kTagScale, (uint32_t)col >> 2);
        sc[0] = fmaf(a, z.x, sc[0]); sc[1] = fmaf(a, z.y, sc[1]); sc[2] = fmaf(a, z.z, sc[2]); sc[3] = fmaf(a, z.w, sc[3]);
        const float4 zx = noise_block<false>(key, p, kTagScale, (uint32_t)cols >> 2);
        const int l = cols & 3;
        xs = fmaf(a, l == 0 ? zx.x : l == 1 ? zx.y : l == 2 ? zx.z : zx.w, xs);
    }
    return make_float4(xs * sc[0], xs * sc[1], xs * sc[2], xs * sc[3]);
}

template <int RANK, bool PERTURB, int SHARE, bool SCALED, bool LOGLIK = false, bool ONE_SLOT = false>
__device__ __forceinline__ void epilogue_forward(const EpiParams &ep, int64_t row, int col0, const uint32_t (&acc)[32],
                                                 const float (&sv)[RANK > 0 ? RANK : 1], float c, uint32_t p, int lane,
                                                 float scale_noise, const CUtensorMap *tmap_y, uint8_t *stage,
                                                 int64_t warp_row0, uint32_t &n_stores, LogLikState *ll = nullptr, int target = -1)
{
    float y[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) y[i] = __uint_as_float(acc[i]);
    if constexpr (PERTURB) {
        // elements e = j*RANK + k of factor A for the 32 columns j = col0 .. col0+31
        constexpr int kBlocks = 32 * RANK / 4;
        const uint32_t q0 = (uint32_t)((col0 * RANK) >> 2);
        if constexpr (SHARE >= 8) {
            // the exchange goes through the staging slot that this chunk's output will use afterwards
            if (ep.y_tma) {
                if (lane == 0) bulk_wait_read<ONE_SLOT ? 0 : 1>();
                __syncwarp();
            }
            add_noise_smem<RANK, SHARE>(ep, p, q0, c, sv, y, lane,
                                        reinterpret_cast<float *>(stage + (ONE_SLOT ? 0u : (n_stores & 1u) * STORE_SLOT_BYTES)));
        } else if constexpr (SHARE > 1) {
            add_noise_shared<RANK, SHARE>(ep, p, q0, c, sv, y, lane);
        } else {
            // one row, one member: every lane generates all of its blocks
            if constexpr (RANK >= 8) {
                // a column's RANK normals come from RANK / 4 consecutive blocks: one out-of-line call per column that
                // walks those blocks in lock step (inlining 32 RANK / 4 generator bodies would overflow the
                // instruction cache, single-block calls leave the dependent Philox chains without overlap)
                float csv[RANK];
#pragma unroll
                for (int k = 0; k < RANK; ++k) csv[k] = c * sv[k];
#pragma unroll
                for (int jl = 0; jl < 32; ++jl)
                    y[jl] += noise_dot_call<RANK / 4>(ep.key, p, kTagA, q0 + (uint32_t)(jl * (RANK / 4)), csv);
            } else {
#pragma unroll
                for (int b = 0; b < kBlocks; ++b) {
                    const float4 z4 = noise_block<false>(ep.key, p, kTagA, q0 + (uint32_t)b);
                    const float z[4] = {z4.x, z4.y, z4.z, z4.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int el = 4 * b + u;              // compile-time after unrolling
                        const int jl = el / RANK, k = el % RANK;
                        y[jl] = fmaf(c * sv[k], z[u], y[jl]);
                    }
                }
            }
        }
    }
    if constexpr (SCALED) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 f = col_scale4(ep.col_scale, ep.cols, col0 + 4 * i, ep.x_scale, scale_noise, ep.key, p);
            y[4 * i] *= f.x; y[4 * i + 1] *= f.y; y[4 * i + 2] *= f.z; y[4 * i + 3] *= f.w;
        }
    }
    if (const uint32_t act = ep.flags & EGR_ACT_MASK) {                   // uniform over the grid
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 in = make_float4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
            const float4 o = ep.y_f32 ? apply_act4<true>(in, act) : apply_act4<false>(in, act);
            y[4 * i] = o.x; y[4 * i + 1] = o.y; y[4 * i + 2] = o.z; y[4 * i + 3] = o.w;
        }
    }
    if constexpr (LOGLIK) {
        // nothing is stored: the chunk's 32 logits (fp32, perturbed) update the row's running maximum and sum of
        // exponentials, and the target's logit is picked up when it lies in this chunk
        constexpr float kLog2e = 1.4426950408889634f;
        float cm = -INFINITY;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if (col0 + i >= ep.cols) y[i] = -INFINITY;               // past the vocabulary's edge
            cm = fmaxf(cm, y[i]);
        }
        const float mn = fmaxf(ll->m, cm);
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) sum += exp2f((y[i] - mn) * kLog2e);
        ll->s = ll->s * exp2f((ll->m - mn) * kLog2e) + sum;
        ll->m = mn;
        const int tl = target - col0;
#pragma unroll
        for (int i = 0; i < 32; ++i) if (tl == i) ll->t = y[i];
        return;
    }
    if (ep.y_tma) {
        // the slot used two stores ago (ONE_SLOT: by the last store) must have been read out before it is overwritten
        uint8_t *slot = stage + (ONE_SLOT ? 0u : (n_stores & 1u) * STORE_SLOT_BYTES);
        if (lane == 0) bulk_wait_read<ONE_SLOT ? 0 : 1>();
        __syncwarp();
        const int sw = (lane >> 1) & 3;                      // 64-byte swizzle: 16-byte chunk ^= address bits 7..8
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint4 v;
            v.x = pack_bf16x2(y[8 * i], y[8 * i + 1]); v.y = pack_bf16x2(y[8 * i + 2], y[8 * i + 3]);
            v.z = pack_bf16x2(y[8 * i + 4], y[8 * i + 5]); v.w = pack_bf16x2(y[8 * i + 6], y[8 * i + 7]);
            *reinterpret_cast<uint4 *>(slot + lane * 64 + ((i ^ sw) << 4)) = v;
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0 && warp_row0 < ep.rows) {               // rows and columns past the edge are clipped by the map
            tma_store_2d_hint(tmap_y, smem_u32(slot), col0, (int)warp_row0, l2_policy_evict_first());   // written once
            bulk_commit();
        }
        ++n_stores;
        return;
    }
    if (row >= ep.rows) return;
    if (ep.y_f32) {
        float *out = reinterpret_cast<float *>(ep.Y) + row * ep.ldy + col0;
        if (col0 + 32 <= ep.cols) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                reinterpret_cast<float4 *>(out)[i] = make_float4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) if (col0 + i < ep.cols) out[i] = y[i];
        }
    } else {
        __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(ep.Y) + row * ep.ldy + col0;
        if (col0 + 32 <= ep.cols) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 v;
                v.x = pack_bf16x2(y[8 * i], y[8 * i + 1]); v.y = pack_bf16x2(y[8 * i + 2], y[8 * i + 3]);
                v.z = pack_bf16x2(y[8 * i + 4], y[8 * i + 5]); v.w = pack_bf16x2(y[8 * i + 6], y[8 * i + 7]);
                reinterpret_cast<uint4 *>(out)[i] = v;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) if (col0 + i < ep.cols) out[i] = __float2bfloat16_rn(y[i]);
        }
    }
}

// W_master[32 rows][32 columns] += scale * acc as one TMA reduce-add: the warp stages its block in shared memory
// (128 bytes per row, 128-byte swizzle) and the addition happens at L2, so the epilogue neither loads W nor issues
// per-lane 16-byte stores.  Rows and columns past the edge are clipped by the tensor map.
__device__ __forceinline__ void epilogue_update_reduce(const EpiParams &ep, int col0, const uint32_t (&acc)[32], int lane,
                                                       const CUtensorMap *tmap_w, uint8_t *stage, int64_t warp_row0,
                                                       uint32_t &n_stores)
{
    uint8_t *slot = stage + (n_stores & 1u) * (32 * 128);
    if (lane == 0) bulk_wait_read<1>();                    // the slot used two stores ago has been read out
    __syncwarp();
    const int sw = lane & 7;                               // 128-byte swizzle: 16-byte chunk ^= row mod 8
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float4 v = make_float4(ep.scale * __uint_as_float(acc[4 * i]), ep.scale * __uint_as_float(acc[4 * i + 1]),
                                     ep.scale * __uint_as_float(acc[4 * i + 2]), ep.scale * __uint_as_float(acc[4 * i + 3]));
        *reinterpret_cast<float4 *>(slot + lane * 128 + ((i ^ sw) << 4)) = v;
    }
    fence_async_smem();
    __syncwarp();
    if (lane == 0 && warp_row0 < ep.rows) {
        tma_reduce_add_2d(tmap_w, smem_u32(slot), col0, (int)warp_row0);
        bulk_commit();
    }
    ++n_stores;
}

// G (+)= scale * acc, nothing else touched
__device__ __forceinline__ void epilogue_gradient(const EpiParams &ep, int64_t row, int col0, const uint32_t (&acc)[32], bool full,
                                                  bool accumulate)
{
    float *o = ep.dW + row * ep.lddw + col0;
    if (full && (ep.lddw & 3) == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float4 v = make_float4(ep.scale * __uint_as_float(acc[4 * i]), ep.scale * __uint_as_float(acc[4 * i + 1]),
                                   ep.scale * __uint_as_float(acc[4 * i + 2]), ep.scale * __uint_as_float(acc[4 * i + 3]));
            if (accumulate) {
                const float4 o4 = reinterpret_cast<const float4 *>(o)[i];
                v.x += o4.x; v.y += o4.y; v.z += o4.z; v.w += o4.w;
            }
            reinterpret_cast<float4 *>(o)[i] = v;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (col0 + i < ep.cols) o[i] = ep.scale * __uint_as_float(acc[i]) + (accumulate ? o[i] : 0.f);
    }
}

// accumulate: dW_out (+)= ; shadow: also write the bf16 copy of the master (last chunk of K only)
__device__ __forceinline__ void epilogue_update(const EpiParams &ep, int64_t row, int col0, const uint32_t (&acc)[32],
                                                bool accumulate, bool shadow)
{
    const bool full = (col0 + 32 <= ep.cols);
    if (!ep.Wm) { epilogue_gradient(ep, row, col0, acc, full, accumulate); return; }     // gradient estimate only
    float *w = ep.Wm + row * ep.ldw + col0;
    float d[32], wn[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) d[i] = ep.scale * __uint_as_float(acc[i]);
    if (full) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 v = reinterpret_cast<const float4 *>(w)[i];
            wn[4 * i] = v.x + d[4 * i]; wn[4 * i + 1] = v.y + d[4 * i + 1];
            wn[4 * i + 2] = v.z + d[4 * i + 2]; wn[4 * i + 3] = v.w + d[4 * i + 3];
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)
            reinterpret_cast<float4 *>(w)[i] = make_float4(wn[4 * i], wn[4 * i + 1], wn[4 * i + 2], wn[4 * i + 3]);
        if (shadow) {
            __nv_bfloat16 *sh = ep.Wsh + row * ep.ldw + col0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 v;
                v.x = pack_bf16x2(wn[8 * i], wn[8 * i + 1]); v.y = pack_bf16x2(wn[8 * i + 2], wn[8 * i + 3]);
                v.z = pack_bf16x2(wn[8 * i + 4], wn[8 * i + 5]); v.w = pack_bf16x2(wn[8 * i + 6], wn[8 * i + 7]);
                reinterpret_cast<uint4 *>(sh)[i] = v;
            }
        }
        if (ep.dW) {
            float *o = ep.dW + row * ep.lddw + col0;
            if ((ep.lddw & 3) == 0) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float4 v = make_float4(d[4 * i], d[4 * i + 1], d[4 * i + 2], d[4 * i + 3]);
                    if (accumulate) {
                        const float4 o4 = reinterpret_cast<const float4 *>(o)[i];
                        v.x += o4.x; v.y += o4.y; v.z += o4.z; v.w += o4.w;
                    }
                    reinterpret_cast<float4 *>(o)[i] = v;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = accumulate ? o[i] + d[i] : d[i];
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if (col0 + i < ep.cols) {
                const float nv = w[i] + d[i];
                w[i] = nv;
                if (shadow) ep.Wsh[row * ep.ldw + col0 + i] = __float2bfloat16_rn(nv);
                if (ep.dW) {
                    float *o = ep.dW + row * ep.lddw + col0 + i;
                    *o = accumulate ? *o + d[i] : d[i];
                }
            }
        }
    }
}

// Tile order: groups of GROUP_M row tiles are swept column by column, so the CTA pairs that run at the same time
// share a handful of B (weight) tiles and GROUP_M A tiles in L2 even when the whole B matrix does not fit in L2
// (e.g. a 32000 x 2048 vocabulary head against 126 MB of L2).
constexpr int GROUP_M = 8;
// q = a / b, r = a % b for non-negative a and positive b.  A 64-bit division is a subroutine of several hundred cycles,
// and the roles of these kernels divide once or more per tile (a tile's main loop is 8 K cycles at K = 1024; the TMA
// producer is only a few stages ahead of the tensor cores): one 32-bit division whenever the numbers fit.
__device__ __forceinline__ void div_mod(int64_t a, int64_t b, int64_t &q, int64_t &r)
{
    if ((((uint64_t)a | (uint64_t)b) >> 32) == 0) {
        const uint32_t q32 = (uint32_t)a / (uint32_t)b;
        q = q32; r = (uint32_t)a - q32 * (uint32_t)b;
    } else {
        q = a / b; r = a % b;
    }
}
__device__ __forceinline__ void tile_coords(int64_t t, int64_t tiles_m, int tiles_n, int64_t &tm, int &tn)
{
    const int64_t per_group = (int64_t)GROUP_M * tiles_n;
    int64_t g, r;
    div_mod(t, per_group, g, r);
    const int64_t first = g * GROUP_M;
    const int64_t gsz = min((int64_t)GROUP_M, tiles_m - first);
    if (gsz == GROUP_M) {                                      // full groups: shifts
        tm = first + (r & (GROUP_M - 1));
        tn = (int)(r >> 3);
    } else {
        const uint32_t q = (uint32_t)r / (uint32_t)gsz;        // ragged last group; r < 8 tiles_n fits in 32 bits
        tm = first + ((uint32_t)r - q * (uint32_t)gsz);
        tn = (int)q;
    }
}
static_assert(GROUP_M == 8, "tile_coords shifts by 3");

// ---------------------------------------------------------------- update: staging of the regenerated factors
// One staging unit: RPU consecutive factor rows (the four elements of a generated block are four rows at r = 1) by eight
// consecutive kappa = p * r + k positions starting at kappa0, as bf16, K-major:
//   At[j][kappa] = bf16(g_p * A_p[j][k]),  Bt[l][kappa] = bf16(B_p[l][k])
// (g_p = the member's or the pair's shaped fitness when scale_by_fitness).  `out` points at the unit's first column of
// row 0; positions at or beyond K_total are written as zeros.
template <int R>
__device__ __forceinline__ void stage_unit(__nv_bfloat16 *__restrict__ out, int64_t ld, int rows, int64_t kappa0, int j0,
                                           int64_t K_total, const float *__restrict__ fitness, uint32_t flags,
                                           const NoiseKey &key, uint32_t tag, int scale_by_fitness)
{
    constexpr int RPU = (R <= 4) ? 4 / R : 1;          // rows per unit
    float v[RPU][8];
#pragma unroll
    for (int a = 0; a < RPU; ++a)
#pragma unroll
        for (int i = 0; i < 8; ++i) v[a][i] = 0.f;

    auto gval = [&](int64_t p) -> float {
        if (!scale_by_fitness) return 1.f;
        return (flags & EGR_ANTITHETIC) ? (fitness[2 * p] - fitness[2 * p + 1]) : fitness[p];
    };

    if (R <= 4) {
        constexpr int PPG = 8 / (R <= 4 ? R : 4);      // noise indices per 8-kappa group: consecutive, from kappa0 / R
        const int64_t p0 = kappa0 / R;
        // the group's fitness values first, all loads in flight together (one after the other, each in front of its
        // generator call, they cost a trip to L2 per noise index)
        float g[PPG];
#pragma unroll
        for (int pi = 0; pi < PPG; ++pi) g[pi] = (kappa0 + (int64_t)pi * R < K_total) ? gval(p0 + pi) : 0.f;
#pragma unroll
        for (int pi = 0; pi < PPG; ++pi) {
            if (kappa0 + (int64_t)pi * R >= K_total) break;
            const float4 z4 = noise_block<false>(key, (uint32_t)(p0 + pi), tag, (uint32_t)(((int64_t)j0 * R) >> 2));
            const float z[4] = {z4.x, z4.y, z4.z, z4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u / R][pi * R + (u % R)] = g[pi] * z[u];
        }
    } else {
        // one row, 8 consecutive rank columns k0..k0+7 of a single noise index
        if (kappa0 < K_total) {
            const int64_t p = kappa0 / R;
            const int k0 = (int)(kappa0 % R);
            const float g = gval(p);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float4 z4 = noise_block<false>(key, (uint32_t)p, tag, (uint32_t)((((int64_t)j0 * R + k0) >> 2) + h));
                v[0][4 * h] = g * z4.x; v[0][4 * h + 1] = g * z4.y; v[0][4 * h + 2] = g * z4.z; v[0][4 * h + 3] = g * z4.w;
            }
        }
    }
#pragma unroll
    for (int a = 0; a < RPU; ++a) {
        if (j0 + a < rows) {
            uint4 w;
            w.x = pack_bf16x2(v[a][0], v[a][1]); w.y = pack_bf16x2(v[a][2], v[a][3]);
            w.z = pack_bf16x2(v[a][4], v[a][5]); w.w = pack_bf16x2(v[a][6], v[a][7]);
            *reinterpret_cast<uint4 *>(out + (int64_t)(j0 + a) * ld) = w;
        }
    }
}

// One-launch update: an item of the side warps is one row unit by FUSED_ITEM_GROUPS groups of eight kappa positions
constexpr int FUSED_ITEM_GROUPS = 256;
__host__ __device__ inline int fused_band_units(int rows, int band, int rank)
{
    const int rpu = (rank <= 4) ? 4 / rank : 1;
    int in_band = rows - band * PAIR_M;
    if (in_band > PAIR_M) in_band = PAIR_M;
    if (in_band < 0) in_band = 0;
    return (in_band + rpu - 1) / rpu;
}

// ---------------------------------------------------------------- the kernel
// BN_T = output columns per tile: 256, or 64 for problems of a handful of tiles (more, narrower tiles put more SMs to
// work; the stage layout stays the same, the B part of a stage is just shorter)
// TAIL: with the tail helpers (see TAIL_WARP0).  A variant of its own, launched for problems of few tiles per CTA pair:
// compiled in, they cost long launches 2 % (a tile's main loop 34.5 K against 33.8 K cycles at 65536 rows) for an
// epilogue that is one of hundreds there.
template <int EPI, int RANK, int SHARE, bool SCALED, int BN_T, bool LOGLIK = false, bool TAIL = false>
__global__ void __launch_bounds__(threads_for(EPI), 1)
gemm_sm100_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const __grid_constant__ CUtensorMap tmap_y, const EpiParams ep)
{
    constexpr int STAGES = stages_for(EPI);
    extern __shared__ uint8_t smem_raw[];
    // 128-byte-swizzled tiles need 1024-byte alignment
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + STAGES * STAGE_BYTES);
    uint64_t *full_bar = bars;                           // [STAGES]  used in the leader CTA only
    uint64_t *empty_bar = bars + MAX_STAGES;             // [STAGES]  one per CTA
    uint64_t *tfull_bar = bars + 2 * MAX_STAGES;         // [2]       one per CTA
    uint64_t *tempty_bar = bars + 2 * MAX_STAGES + 2;    // [2]       used in the leader CTA only
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * MAX_STAGES + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    uint64_t *rfull_bar = bars + 2 * MAX_STAGES + 6;     // [2 channels][2 buffers]  relay -> worker
    uint64_t *rfree_bar = bars + 2 * MAX_STAGES + 10;    // [2 channels][2 buffers]  worker -> relay
    constexpr bool kRelay = relay_for(EPI, RANK);
    // with the relay the TMA producer is warp 13 (scheduler 1, next to the MMA warp and the relay warps: all of them one
    // thread or a few instructions per chunk), and warp 0 joins the side warps
    // the one-launch updates use the same placement: producer beside the MMA warp, side warps on the other schedulers
    constexpr bool kFused = (EPI == EPI_UPDATE_FUSED || EPI == EPI_UPDATE_FUSED_REDUCE);
    constexpr int kProducerWarp = (kRelay || kFused) ? 13 : 0;
    constexpr int kSideActive = kRelay ? 7 : FWD_EXTRA_WARPS;
    constexpr bool kTail = TAIL && kRelay && !LOGLIK && BN_T == BN;  // tail helpers (see TAIL_WARP0)
    // how the side warps claim rows (see their loop): single rows for very small problems; the first rows (the first
    // row-tile group, or all rows of a small problem) in two K-halves, and their bands are counted twice by whoever
    // waits for them
    const int64_t side_single = (EPI == EPI_FORWARD && SHARE < 8 && ep.rows < (int64_t)2 * gridDim.x * kSideActive) ? ep.rows : 0;
    const int64_t side_split = (EPI == EPI_FORWARD && SHARE < 8) ? (int64_t)ep.split_rows : 0;
    constexpr int kTailBarThreads = 32 * (TAIL_WARPS + 1);           // the helpers wait, warp 2 arrives

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = cluster_ctarank();                // 0 = leader
    const int64_t cluster_id = blockIdx.x >> 1;
    const int64_t num_clusters = gridDim.x >> 1;
    constexpr int BNH_T = BN_T / 2;                  // rows of B staged by each CTA of the pair
    constexpr uint32_t kStageTxBytes = 2u * (uint32_t)(A_STAGE_BYTES + BNH_T * BK * 2);
    const int tiles_n = (ep.cols + BN_T - 1) / BN_T;
    const int64_t tiles_m = (ep.rows + PAIR_M - 1) / PAIR_M;
    const int64_t num_tiles = tiles_m * tiles_n;
    const int num_kb = (ep.K + BK - 1) / BK;
    // the one-launch update walks (K-chunk, tile) items, chunk-major; every other variant has one chunk
    const int64_t num_items = kFused ? num_tiles * ep.n_chunks : num_tiles;
    auto chunk_kb = [&](int c) -> int {                  // k-blocks of chunk c (ep.K = padded total length, ep.kc = chunk length)
        const int64_t left = (int64_t)ep.K - (int64_t)c * ep.kc;
        return (int)(((left < ep.kc ? left : (int64_t)ep.kc) + BK - 1) / BK);
    };
    // bounded acquire-spin on a global counter; false when the CTA is aborting
    auto spin_until = [&](const int *ctr, int expected, int where) -> bool {
        int spins = 0;
        while (true) {
            int v;
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
            if (v >= expected) return true;
            if (*abort_flag) return false;
            if (++spins > SPIN_LIMIT) {
                *abort_flag = 1;
                atomicExch(ep.status, EGR_ERR_TIMEOUT); atomicExch(ep.status + 1, where);
                return false;
            }
            __nanosleep(128);
        }
    };

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(smem_u32(&full_bar[i]), 1); mbar_init(smem_u32(&empty_bar[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&tfull_bar[i]), 1); mbar_init(smem_u32(&tempty_bar[i]), 2 * EPI_WARPS); }
        if (kRelay) for (int i = 0; i < 4; ++i) { mbar_init(smem_u32(&rfull_bar[i]), 1); mbar_init(smem_u32(&rfree_bar[i]), 1); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
    }
    if (warp == 1) {
        // both CTAs of the pair take part in the paired allocation and receive the same column base
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync();                     // barriers of both CTAs are initialised before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == kProducerWarp) {
        // ---------------- TMA producer (both CTAs): own 128 rows of A, own 128 of the tile's 256 rows of B
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool alive = true;
            // one-launch update: counters that say an item's two factor bands are staged, and what they must reach
            auto item_ready = [&](int64_t item, const int *(&ctr)[2], int (&expected)[2]) {
                int64_t c64, tile_;
                div_mod(item, num_tiles, c64, tile_);
                const int c = (int)c64;
                int64_t tm; int tn;
                tile_coords(tile_, tiles_m, tiles_n, tm, tn);
                const int ipr_c = (chunk_kb(c) * (BK / 8) + FUSED_ITEM_GROUPS - 1) / FUSED_ITEM_GROUPS;
                for (int f = 0; f < 2; ++f) {
                    const int band = f ? tn : (int)tm;
                    expected[f] = fused_band_units(f ? ep.cols : (int)ep.rows, band, RANK) * ipr_c;
                    ctr[f] = ep.ready_u + ((int64_t)c * 2 + f) * ep.max_bands + band;
                }
            };
            bool known_ready = false;            // the next item's bands were seen staged while this item's loads were issued
            for (int64_t item = cluster_id; alive && item < num_items; item += num_clusters) {
                int64_t c64 = 0, tile = item;
                if constexpr (kFused) div_mod(item, num_tiles, c64, tile);
                const int c = (int)c64;
                int64_t tm; int tn;
                tile_coords(tile, tiles_m, tiles_n, tm, tn);
                const int row0 = (int)tm * PAIR_M + (int)cta_rank * BM;
                const int col0 = tn * BN_T + (int)cta_rank * BNH_T;
                const int nkb = kFused ? chunk_kb(c) : num_kb;
                const int kx0 = kFused ? (c % ep.n_slots) * ep.kc : 0;            // the chunk's ring slot
                if constexpr (kFused) {
                    // the side warps (of every CTA) have staged this chunk's rows of both factors: acquire the two bands'
                    // counters, then order what they wrote before this thread's asynchronous loads
                    if (!known_ready) {
                        const int *ctr[2]; int expected[2];
                        item_ready(item, ctr, expected);
                        for (int f = 0; f < 2 && alive; ++f) alive = spin_until(ctr[f], expected[f], 8);
                        if (!alive) break;
                    }
                    asm volatile("fence.proxy.async;" ::: "memory");
                    known_ready = false;
                }
                for (int kb = 0; kb < nkb; ++kb) {
                    if constexpr (kFused) {
                        // A look at the next item's counters a few stages before this item's loads end: the two loads
                        // take a trip to L2, which the stages already queued cover here and would not at the item's start.
                        if (kb == nkb - 3 && item + num_clusters < num_items) {
                            const int *ctr[2]; int expected[2];
                            item_ready(item + num_clusters, ctr, expected);
                            int v0, v1;
                            asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v0) : "l"(ctr[0]) : "memory");
                            asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v1) : "l"(ctr[1]) : "memory");
                            if (v0 >= expected[0] && v1 >= expected[1]) {
                                asm volatile("fence.acq_rel.gpu;" ::: "memory");
                                known_ready = true;
                            }
                        }
                    }
                    if (!mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abort_flag, ep.status, 1)) { alive = false; break; }
                    const uint32_t leader_full = map_to_cta(smem_u32(&full_bar[stage]), 0);
                    if (cta_rank == 0) mbar_expect_tx(smem_u32(&full_bar[stage]), kStageTxBytes);   // both CTAs' bytes
                    const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES);
                    tma_load_2d_pair(sa, &tmap_a, kx0 + kb * BK, row0, leader_full);
                    tma_load_2d_pair(sa + A_STAGE_BYTES, &tmap_b, kx0 + kb * BK, col0, leader_full);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer: one thread of the leader CTA drives the tensor cores of both SMs
        if (lane == 0 && cta_rank == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(PAIR_M, BN_T);
            int stage = 0; uint32_t phase = 0;
            int64_t it = 0;
            bool alive = true;
            // everything the loop needs per stage is an offset from these
            const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
            const uint32_t desc_lo0 = (smem_u32(smem) & 0x3FFFFu) >> 4;
            constexpr uint32_t kDescHi = (uint32_t)(make_kmajor_sw128_desc(0) >> 32);
            for (int64_t item = cluster_id; alive && item < num_items; item += num_clusters, ++it) {
                const int acc = (int)(it & 1);
                const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
                if (!mbar_wait(smem_u32(&tempty_bar[acc]), acc_phase ^ 1u, abort_flag, ep.status, 2)) { alive = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                int nkb = num_kb;
                if constexpr (kFused) { int64_t c64, t64; div_mod(item, num_tiles, c64, t64); nkb = chunk_kb((int)c64); }
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(full0 + 8u * (uint32_t)stage, phase, abort_flag, ep.status, 3)) { alive = false; break; }
                    tc_fence_after();
                    // the four MMAs of a stage as one instruction sequence: descriptors differ in their low word only
                    const uint32_t a_lo = desc_lo0 + (uint32_t)stage * (uint32_t)(STAGE_BYTES >> 4);
                    tc_mma_bf16_pair_x4(d_tmem, a_lo, a_lo + (uint32_t)(A_STAGE_BYTES >> 4), kDescHi, idesc, kb ? 1u : 0u);
                    tc_commit_pair(empty0 + 8u * (uint32_t)stage);     // frees the stage in both CTAs
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (alive) tc_commit_pair(smem_u32(&tfull_bar[acc]));  // accumulator complete, both CTAs
            }
        }
    } else if (warp >= BASE_WARPS + (kRelay ? 2 : 0) || ((kRelay || kFused) && warp == 0)) {
        if constexpr (kFused) if ((warp & 3) != 1) {
            // ---------------- side warps of the one-launch update: stage the factors, chunk by chunk, into the ring.  An
            // item is one row unit (RPU rows) by FUSED_ITEM_GROUPS groups of eight kappa positions; items are claimed in
            // an order that finishes chunk 0 first and, inside a chunk, interleaves the 256-row bands of the two factors.
            // Before the first item of a chunk that reuses a slot, the warp waits until every CTA has taken the slot's
            // previous chunk out of it (that chunk was staged by warps that waited for nothing later, so this ends).
            constexpr int R = RANK;
            constexpr int RPU = (R <= 4) ? 4 / R : 1;
            constexpr int UPB = PAIR_M / RPU;                       // row units per 256-row band
            const int bands_a = (int)((ep.rows + PAIR_M - 1) / PAIR_M), bands_b = (ep.cols + PAIR_M - 1) / PAIR_M;
            const int nb = min(bands_a, bands_b);
            const int cap = UPB * ep.ipr;                           // items of a full band (ipr = items per row unit and chunk)
            const int64_t per_chunk = (int64_t)(bands_a + bands_b) * cap;
            const int64_t total = per_chunk * ep.n_chunks;
            int released = ep.n_slots - 1;                          // chunks up to this one may be written
            bool alive = true;
            while (alive) {
                long long item = 0;
                if (lane == 0) item = (long long)atomicAdd(reinterpret_cast<unsigned long long *>(ep.side_counter), 1ull);
                item = __shfl_sync(0xffffffffu, item, 0);
                if (item >= total) break;
                int64_t c64, idx;
                div_mod(item, per_chunk, c64, idx);
                const int c = (int)c64;
                if (c > released) {
                    // slot c % n_slots held chunk c - n_slots: both CTAs of every pair report each of their items of it
                    if (lane == 0) alive = spin_until(ep.loaded + (c - ep.n_slots), (int)(2 * num_tiles), 10);
                    alive = __shfl_sync(0xffffffffu, (int)alive, 0) != 0;
                    if (!alive) break;
                    released = c;
                }
                int band, f;
                int64_t rem;
                int64_t q64;
                if (idx < (int64_t)2 * nb * cap) { div_mod(idx, cap, q64, rem); band = (int)q64 >> 1; f = (int)q64 & 1; }
                else { div_mod(idx - (int64_t)2 * nb * cap, cap, q64, rem); band = nb + (int)q64; f = (bands_a > bands_b) ? 0 : 1; }
                const int unit_in_band = (int)((uint32_t)rem / (uint32_t)ep.ipr), ksub = (int)rem - unit_in_band * ep.ipr;   // rem < cap
                const int rows_f = f ? ep.cols : (int)ep.rows;
                const int j0 = band * PAIR_M + unit_in_band * RPU;
                const int groups = chunk_kb(c) * (BK / 8);
                const int kg0 = ksub * FUSED_ITEM_GROUPS;
                if (j0 >= rows_f || kg0 >= groups) continue;        // past the edge of the factor or of a short last chunk
                const int kg1 = min(kg0 + FUSED_ITEM_GROUPS, groups);
                __nv_bfloat16 *out = (f ? ep.Bt : ep.At) + (int64_t)(c % ep.n_slots) * ep.kc;
                const int64_t kbase = (int64_t)c * ep.kc;
                for (int kg = kg0 + lane; kg < kg1; kg += 32)
                    stage_unit<R>(out + (int64_t)kg * 8, ep.ldk, rows_f, kbase + (int64_t)kg * 8, j0, ep.K_total, ep.fitness,
                                  ep.flags, ep.key, f ? kTagB : kTagA, f ? 0 : 1);
                // the rows are in memory before the counter says so, also for the asynchronous proxy of the reader
                asm volatile("fence.proxy.async;" ::: "memory");
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(ep.ready_u + ((int64_t)c * 2 + f) * ep.max_bands + band, 1);
            }
        }
        // ---------------- side warps (FORWARD only): skinny products for groups of rows
        if constexpr (EPI == EPI_FORWARD) if (ep.side_counter && (!kRelay || (warp & 3) != 1)) {
            // Claims are four rows, except for problems so small that four-row claims would leave most side warps
            // without work (fewer than two rows per side warp on the chip): those go row by row.  (Single-row claims for
            // the first bands of large problems were tried: a trip of the reduction lasts as long as the round trip of
            // its rows' loads whether it reduces one row or four, so they only multiplied the number of trips - at 4096
            // rows the last bands were ready after 150 K cycles instead of 60 K.)
            const int64_t single = side_single;
            // later claims: four rows, or eight (sixteen) when aligned runs of that many rows are known to share their noise
            constexpr int kItem = (SHARE == 16) ? 16 : (SHARE >= 8) ? 8 : 4;
            // The rows of the first row-tile group (ep.split_rows; none for shared runs) are claimed
            // as two items per four rows, one per half of K: a whole four-row item takes about 60 K cycles at K = 4096,
            // so with one item per side warp the first tiles' bands were ready only long after their main loop (34 K
            // cycles; at 4096 rows the first epilogue of every CTA pair waited 47 K cycles).  In halves all side warps work
            // on the first group's rows first and its bands are complete after about 30 K cycles.
            // (in single-row mode the halves are halves of single rows: with fewer side warps than rows - the grid has
            // no more CTA pairs than tiles - whole rows would leave some warps two of them, 62 K cycles at K = 4096)
            const int64_t split = side_split;
            const int64_t split_items = single ? 2 * split : split / 2;     // rows x 2 halves, or (split / 4) groups x 2
            const int64_t num_items = single ? split_items + (ep.rows - split)
                                             : split_items + ((ep.rows - split + kItem - 1) / kItem);
            while (true) {
                int item = 0;
                if (lane == 0) item = atomicAdd(ep.side_counter, 1);
                item = __shfl_sync(0xffffffffu, item, 0);
                if (item >= num_items) break;
                if (item < split_items) {
                    const int hn = single ? 1 : 4;
                    const int64_t r0 = (int64_t)(item >> 1) * hn;
                    skinny_rows4_half<__nv_bfloat16, RANK>(ep.X, ep.ldx, ep.K, ep.T, ep.mbase, ep.rowmap, ep.flags, ep.key, r0, hn,
                                                           ep.s_out, lane, item & 1);
                    __syncwarp();
                    if (lane == 0) { __threadfence(); atomicAdd(ep.ready + r0 / BM, hn); }
                    continue;
                }
                const int64_t row0 = single ? split + ((int64_t)item - split_items) : split + ((int64_t)item - split_items) * kItem;
                const int nrows = single ? 1 : (int)min((int64_t)kItem, ep.rows - row0);
                if (SHARE >= 8 && nrows == kItem) {
                    uint32_t p8; float sign8;
                    member_noise(member_of(ep.rowmap, ep.mbase, row0, ep.T), ep.flags, p8, sign8);
                    skinny_rows_same<__nv_bfloat16, RANK, false, kItem>(ep.X, ep.ldx, ep.K, p8, ep.key, row0, ep.s_out, lane);
                } else {
                    for (int sub = 0; sub < nrows; sub += 4)
                        skinny_rows4<__nv_bfloat16, RANK, false>(ep.X, ep.ldx, ep.K, ep.T, ep.mbase, ep.rowmap, ep.flags, ep.key,
                                                                 row0 + sub, min(4, nrows - sub), ep.s_out, lane);
                }
                __syncwarp();
                if (lane == 0) { __threadfence(); atomicAdd(ep.ready + row0 / BM, nrows); }
            }
        }
    } else {
        // ---------------- epilogue warps (2..9); TMEM lane quarter = warp % 4, column half = (warp - 2) / 4
        // With the relay (see the top of the file) warps 5 and 9 only move their chunks to shared memory and warps
        // 10 and 11 ("workers") run the epilogue of quarter 1 on them, with the staging slots of the warps they stand in for.
        const bool worker = kRelay && warp >= BASE_WARPS;
        const bool relay = kRelay && !worker && (warp & 3) == 1;
        const int quarter = worker ? 1 : (warp & 3);
        const int part = worker ? (warp - BASE_WARPS) : ((warp - 2) >> 2);
        const int slot_owner = worker ? (3 + 4 * part) : (warp - 2);
        uint8_t *stage = smem + STAGES * STAGE_BYTES + BAR_BYTES + slot_owner * 2 * store_slot_bytes(EPI);
        // relay buffers of this column half: chunk element (row, column c) at float4 index (c / 4) * 32 + row, so that both
        // sides touch consecutive 16-byte pieces with consecutive lanes
        float4 *rbuf = reinterpret_cast<float4 *>(smem + STAGES * STAGE_BYTES + BAR_BYTES + store_bytes(EPI)) + part * 2 * (RELAY_BUF_BYTES / 16);
        const uint32_t rfull0 = smem_u32(&rfull_bar[2 * part]), rfree0 = smem_u32(&rfree_bar[2 * part]);
        uint32_t n_stores = 0, n_relay = 0;
        int64_t it = 0;
        bool alive = true;
        bool tail_signalled = false;
        for (int64_t item = cluster_id; alive && item < num_items; item += num_clusters, ++it) {
            const int acc = (int)(it & 1);
            const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
            int64_t c64 = 0, tile = item;
            if constexpr (kFused) div_mod(item, num_tiles, c64, tile);
            const int c_item = (int)c64;
            int64_t tm; int tn;
            tile_coords(tile, tiles_m, tiles_n, tm, tn);
            const int64_t band = tm * 2 + cta_rank;                        // 128-row band this CTA owns
            const int64_t row = band * BM + quarter * 32 + lane;
            const int tile_col0 = tn * BN_T;
            constexpr int kChunksPerPart = BN_T / 32 / EPI_PARTS;
            // the second half of the last tile's chunks belongs to the tail helpers (loop bounds stay compile-time)
            const bool last_tile = kTail && item + num_clusters >= num_items;
            if (!worker) {
                if (!mbar_wait(smem_u32(&tfull_bar[acc]), acc_phase, abort_flag, ep.status, 4)) { alive = false; break; }
                tc_fence_after();
                if (kTail && last_tile && warp == 2) {
                    asm volatile("barrier.cta.arrive 2, %0;" ::"r"(kTailBarThreads) : "memory");
                    tail_signalled = true;
                }
            }
            if constexpr (kFused) {
                // the item's MMAs are complete, so its loads have left the chunk's ring slot: one report per CTA
                if (warp == 2 && lane == 0) atomicAdd(ep.loaded + c_item, 1);
                // chunk c of a tile is added after chunk c - 1, whoever computed that: all 2 * EPI_WARPS warps of the pair
                // that held the tile then have bumped its counter behind their stores
                if (c_item > 0) {
                    if (lane == 0) spin_until(ep.done + tile, c_item * 2 * EPI_WARPS, 9);
                    __syncwarp();
                    if (*abort_flag) { alive = false; break; }
                }
            }
            if (relay) {
                for (int chunk = part * kChunksPerPart; chunk < (part + 1) * kChunksPerPart; ++chunk, ++n_relay) {
                    if (last_tile && chunk >= part * kChunksPerPart + kChunksPerPart / 2) break;
                    if (tile_col0 + chunk * 32 >= ep.cols) break;                     // the worker stops at the same chunk
                    const uint32_t b = n_relay & 1u;
                    if (!mbar_wait(rfree0 + 8u * b, ((n_relay >> 1) & 1u) ^ 1u, abort_flag, ep.status, 6)) { alive = false; break; }
                    uint32_t v[32];
                    tc_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + chunk * 32), v);
                    tc_wait_ld();
                    float4 *dst = rbuf + b * (RELAY_BUF_BYTES / 16) + lane;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        dst[i * 32] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                                  __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
                    __syncwarp();                                                     // one arrival per warp, not one per lane
                    if (lane == 0) mbar_arrive(rfull0 + 8u * b);                      // releases the warp's stores
                }
                if (!alive) break;
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&tempty_bar[acc]), 0));
                continue;
            }

            // per-row perturbation context
            constexpr bool kPerturb = (EPI == EPI_FORWARD);
            float sv[RANK > 0 ? RANK : 1];
            float c = 0.f, scale_noise = 0.f; uint32_t p = 0;
            if (kPerturb && ep.ready && band * BM < ep.rows) {
                // the band's skinny products come from side warps somewhere on the chip: acquire its counter
                // (rows reduced in two halves are counted twice)
                const int expected = (int)min((int64_t)BM, ep.rows - band * BM) * (band * BM < side_split ? 2 : 1);
                if (lane == 0) {
                    int spins = 0;
                    while (true) {
                        int v;
                        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ep.ready + band) : "memory");
                        if (v >= expected) break;
                        if (*abort_flag) break;
                        if (++spins > SPIN_LIMIT) {
                            *abort_flag = 1;
                            atomicExch(ep.status, EGR_ERR_TIMEOUT); atomicExch(ep.status + 1, 5);
                            break;
                        }
                        __nanosleep(128);
                    }
                }
                __syncwarp();
                if (*abort_flag) { alive = false; break; }
            }
            // SHARE > 1: aligned groups of SHARE rows see the same noise index and share the generation of A_p
            if (kPerturb) {
                float sign;
                member_noise(member_of(ep.rowmap, ep.mbase, (ep.rowmap && row >= ep.rows) ? 0 : row, ep.T), ep.flags, p, sign);
                c = ep.coef * sign;
                scale_noise = ep.sigma_s * sign;
#pragma unroll
                for (int k = 0; k < (RANK > 0 ? RANK : 1); ++k) sv[k] = (row < ep.rows) ? __ldcg(ep.s + row * (RANK > 0 ? RANK : 1) + k) : 0.f;
            } else {
#pragma unroll
                for (int k = 0; k < (RANK > 0 ? RANK : 1); ++k) sv[k] = 0.f;
            }

            LogLikState ll = {-INFINITY, 0.f, 0.f};
            int target = -1;
            if constexpr (LOGLIK) target = (row < ep.rows) ? __ldg(ep.targets + row) : -1;
            for (int chunk = part * kChunksPerPart; chunk < (part + 1) * kChunksPerPart; ++chunk) {
                if (last_tile && chunk >= part * kChunksPerPart + kChunksPerPart / 2) break;
                const int col0 = tile_col0 + chunk * 32;
                if (col0 >= ep.cols) break;                     // uniform across the warp
                uint32_t v[32];
                if (worker) {
                    const uint32_t b = n_relay & 1u;
                    if (!mbar_wait(rfull0 + 8u * b, (n_relay >> 1) & 1u, abort_flag, ep.status, 7)) { alive = false; break; }
                    const float4 *src = rbuf + b * (RELAY_BUF_BYTES / 16) + lane;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 f = src[i * 32];
                        v[4 * i] = __float_as_uint(f.x); v[4 * i + 1] = __float_as_uint(f.y);
                        v[4 * i + 2] = __float_as_uint(f.z); v[4 * i + 3] = __float_as_uint(f.w);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(rfree0 + 8u * b);    // every lane has read its part of the buffer
                    ++n_relay;
                } else {
                    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + chunk * 32);
                    tc_ld_32x32(taddr, v);
                    tc_wait_ld();
                }
                if (EPI == EPI_UPDATE_REDUCE || EPI == EPI_UPDATE_FUSED_REDUCE) {
                    epilogue_update_reduce(ep, col0, v, lane, &tmap_y, stage, band * BM + quarter * 32, n_stores);
                } else if (EPI == EPI_UPDATE_FUSED) {
                    if (row < ep.rows) epilogue_update(ep, row, col0, v, c_item > 0, ep.Wsh != nullptr && c_item + 1 == ep.n_chunks);
                } else if (EPI == EPI_UPDATE) {
                    if (row < ep.rows) epilogue_update(ep, row, col0, v, ep.dw_accumulate != 0, ep.Wsh != nullptr);
                } else {
                    epilogue_forward<RANK, kPerturb, SHARE, SCALED, LOGLIK>(ep, row, col0, v, sv, c, p, lane, scale_noise, &tmap_y, stage,
                                                                            band * BM + quarter * 32, n_stores, &ll, target);
                }
            }
            if constexpr (LOGLIK) {
                // this warp's share of the tile for its row: partial [column part of the whole matrix][row]
                if (alive && row < ep.rows) {
                    ep.ll_part[((int64_t)tn * EPI_PARTS + part) * ep.rows + row] = make_float2(ll.m, ll.s);
                    if (target >= tile_col0 + part * kChunksPerPart * 32 && target < tile_col0 + (part + 1) * kChunksPerPart * 32 &&
                        target < ep.cols)
                        ep.ll_tgt[row] = ll.t;
                }
            }
            if (!alive) break;
            if (!worker) {
                tc_fence_before();
                __syncwarp();
                // the leader's MMA thread may overwrite this accumulator once all 16 TMEM-reading warps of the pair are done
                if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&tempty_bar[acc]), 0));
            }
            if constexpr (kFused) {
                // this warp's part of the tile is in memory (reduce-add stores: complete, not merely read out of shared
                // memory): the next chunk of the same tile may be added
                if (EPI == EPI_UPDATE_FUSED_REDUCE && lane == 0) bulk_wait<0>();
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(ep.done + tile, 1);
            }
        }
        if (lane == 0) bulk_wait<0>();      // the last stores have left shared memory and landed
        // (a launch that gave up before its last tile still releases the tail helpers)
        if (kTail && warp == 2 && !tail_signalled && cluster_id < num_items)
            asm volatile("barrier.cta.arrive 2, %0;" ::"r"(kTailBarThreads) : "memory");
    }

    // ---------------- tail helpers: the second half of the last tile's chunks (see TAIL_WARP0)
    if constexpr (kTail) {
        const int64_t n_my = cluster_id < num_items ? (num_items - cluster_id + num_clusters - 1) / num_clusters : 0;
        __syncwarp();
        if (warp >= TAIL_WARP0 && n_my > 0) {
            const int64_t tile = cluster_id + (n_my - 1) * num_clusters;
            const int acc = (int)((n_my - 1) & 1);
            const int quarter = warp & 3, part = (warp - TAIL_WARP0) >> 2;
            int64_t tm; int tn;
            tile_coords(tile, tiles_m, tiles_n, tm, tn);
            const int64_t band = tm * 2 + cta_rank;
            const int64_t row = band * BM + quarter * 32 + lane;
            uint8_t *stage = smem + STAGES * STAGE_BYTES + BAR_BYTES + store_bytes(EPI) + RELAY_BYTES + (warp - TAIL_WARP0) * STORE_SLOT_BYTES;
            asm volatile("barrier.cta.sync 2, %0;" ::"r"(kTailBarThreads) : "memory");     // no issue slots while waiting
            tc_fence_after();
            bool ok = !*abort_flag;
            if (ok && ep.ready && band * BM < ep.rows) {
                const int expected = (int)min((int64_t)BM, ep.rows - band * BM) * (band * BM < side_split ? 2 : 1);
                if (lane == 0) spin_until(ep.ready + band, expected, 14);
                __syncwarp();
                ok = !*abort_flag;
            }
            if (ok) {
                float sv[RANK > 0 ? RANK : 1];
                uint32_t p; float sign;
                member_noise(member_of(ep.rowmap, ep.mbase, (ep.rowmap && row >= ep.rows) ? 0 : row, ep.T), ep.flags, p, sign);
                const float c = ep.coef * sign, scale_noise = ep.sigma_s * sign;
#pragma unroll
                for (int k = 0; k < (RANK > 0 ? RANK : 1); ++k) sv[k] = (row < ep.rows) ? __ldcg(ep.s + row * (RANK > 0 ? RANK : 1) + k) : 0.f;
                constexpr int kChunksPerPart = BN_T / 32 / EPI_PARTS;
                uint32_t n_stores = 0;
                for (int chunk = part * kChunksPerPart + kChunksPerPart / 2; chunk < (part + 1) * kChunksPerPart; ++chunk) {
                    const int col0 = tn * BN_T + chunk * 32;
                    if (col0 >= ep.cols) break;
                    uint32_t v[32];
                    tc_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + chunk * 32), v);
                    tc_wait_ld();
                    epilogue_forward<RANK, true, SHARE, SCALED, false, true>(ep, row, col0, v, sv, c, p, lane, scale_noise, &tmap_y,
                                                                             stage, band * BM + quarter * 32, n_stores);
                }
                tc_fence_before();
                if (lane == 0) bulk_wait<0>();
            }
        }
    }

    // nobody leaves (or frees tensor memory) while the peer may still read this CTA's shared memory or signal
    // its barriers
    tc_fence_before();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

template <int EPI, int RANK, int SHARE = 1, bool SCALED = false, int BN_T = BN, bool LOGLIK = false>
int launch_gemm(const CUtensorMap &ta, const CUtensorMap &tb, const EpiParams &ep, cudaStream_t st,
                const CUtensorMap *ty = nullptr)
{
    static bool configured[2][64] = {};       // per device: the attribute belongs to the device's copy of the kernel
    const int sms = sm_count();
    if (sms < 2) return EGR_ERR_CUDA;
    const int64_t tiles = ((ep.rows + PAIR_M - 1) / PAIR_M) * ((ep.cols + BN_T - 1) / BN_T);
    const int64_t max_clusters = sms / 2;
    unsigned clusters = (unsigned)(tiles < max_clusters ? tiles : max_clusters);
    // a forward whose skinny products come from its own side warps is launched on every SM pair even when there are
    // fewer tiles: the pairs without a tile still lend their side warps (1024 rows of a 4096 x 4096 layer are 64 tiles;
    // with 64 pairs the rows met 896 side warps and the products took a round and a half of claims)
    if (EPI == EPI_FORWARD && ep.side_counter != nullptr) clusters = (unsigned)max_clusters;
    // the variant with tail helpers where the last tile's epilogue is a visible share of the launch (up to eight tiles
    // per CTA pair); not for the scaled or the log-likelihood forms
    constexpr bool kHasTail = relay_for(EPI, RANK) && !SCALED && !LOGLIK && BN_T == BN;
    const bool tail = kHasTail && tiles <= 8 * (int64_t)clusters;
    auto kern = gemm_sm100_kernel<EPI, RANK, SHARE, SCALED, BN_T, LOGLIK, false>;
    if constexpr (kHasTail) if (tail) kern = gemm_sm100_kernel<EPI, RANK, SHARE, SCALED, BN_T, LOGLIK, true>;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return EGR_ERR_CUDA;
    {
        std::lock_guard<std::mutex> cfg_lock(config_mutex());
        if (!configured[tail][dev]) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes_for(EPI)) != cudaSuccess)
                return EGR_ERR_CUDA;
            configured[tail][dev] = true;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * clusters, 1, 1);
    cfg.blockDim = dim3(threads_for(EPI), 1, 1);
    cfg.dynamicSmemBytes = smem_bytes_for(EPI);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cuda_ok(cudaLaunchKernelEx(&cfg, kern, ta, tb, ty ? *ty : ta, ep));
}

// Tile width for small problems: when even four times as many tiles do not exceed the CTA pairs, 64-wide tiles put more
// SMs to work.  Beyond that the narrow tiles lose: every column tile re-reads its A tile, and with four times the
// column tiles the L2 -> SM traffic becomes the bound (4096 x 4096 with 1024 rows: 38 us wide, 88 us narrow).
constexpr int BN_NARROW = 64;
inline bool narrow_tiles(int64_t rows, int64_t cols)
{
    const int64_t tiles = ((rows + PAIR_M - 1) / PAIR_M) * ((cols + BN - 1) / BN);
    return 4 * tiles <= sm_count() / 2;
}

// ---------------------------------------------------------------- update: factor staging
// Writes one K-chunk of a stacked factor: one thread per unit.
template <int R>
__global__ void __launch_bounds__(256)
stage_factors_kernel(__nv_bfloat16 *__restrict__ out, int64_t ld, int rows, int64_t kc0, int kc_len, int64_t K_total,
                     const float *__restrict__ fitness, uint32_t flags, NoiseKey key, uint32_t tag, int scale_by_fitness)
{
    constexpr int RPU = (R <= 4) ? 4 / R : 1;
    const int groups = (kc_len + 7) / 8;               // 8-kappa groups in this chunk
    const int64_t unit = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t row_units = (rows + RPU - 1) / RPU;
    if (unit >= row_units * groups) return;
    const int kg = (int)(unit % groups);
    const int j0 = (int)(unit / groups) * RPU;
    stage_unit<R>(out + (int64_t)kg * 8, ld, rows, kc0 + (int64_t)kg * 8, j0, K_total, fitness, flags, key, tag, scale_by_fitness);
}

template <int R>
int launch_stage(__nv_bfloat16 *out, int64_t ld, int rows, int64_t kc0, int kc_len, int64_t K_total, const float *fitness,
                 uint32_t flags, NoiseKey key, uint32_t tag, int scale_by_fitness, cudaStream_t st)
{
    constexpr int RPU = (R <= 4) ? 4 / R : 1;
    const int64_t units = (int64_t)((rows + RPU - 1) / RPU) * ((kc_len + 7) / 8);
    stage_factors_kernel<R><<<(unsigned)((units + 255) / 256), 256, 0, st>>>(out, ld, rows, kc0, kc_len, K_total, fitness,
                                                                            flags, key, tag, scale_by_fitness);
    return cuda_ok(cudaGetLastError());
}

int launch_stage_r(int r, __nv_bfloat16 *out, int64_t ld, int rows, int64_t kc0, int kc_len, int64_t K_total,
                   const float *fitness, uint32_t flags, NoiseKey key, uint32_t tag, int sbf, cudaStream_t st)
{
    switch (r) {
        case 1:  return launch_stage<1>(out, ld, rows, kc0, kc_len, K_total, fitness, flags, key, tag, sbf, st);
        case 2:  return launch_stage<2>(out, ld, rows, kc0, kc_len, K_total, fitness, flags, key, tag, sbf, st);
        case 4:  return launch_stage<4>(out, ld, rows, kc0, kc_len, K_total, fitness, flags, key, tag, sbf, st);
        case 8:  return launch_stage<8>(out, ld, rows, kc0, kc_len, K_total, fitness, flags, key, tag, sbf, st);
        case 16: return launch_stage<16>(out, ld, rows, kc0, kc_len, K_total, fitness, flags, key, tag, sbf, st);
    }
    return EGR_ERR_BADARG;
}

// bf16 copy of the fp32 master, eight values per thread (two 128-bit loads, one 128-bit store)
__global__ void __launch_bounds__(256)
shadow_bf16_kernel(const float *__restrict__ Wm, int64_t ldw, __nv_bfloat16 *__restrict__ Wsh, int64_t ldsh, int rows, int n8)
{
    const int64_t vecs = (int64_t)rows * n8;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < vecs; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / n8;
        const int c = (int)(i % n8) * 8;
        const float4 a = reinterpret_cast<const float4 *>(Wm + r * ldw + c)[0], b = reinterpret_cast<const float4 *>(Wm + r * ldw + c)[1];
        uint4 w;
        w.x = pack_bf16x2(a.x, a.y); w.y = pack_bf16x2(a.z, a.w); w.z = pack_bf16x2(b.x, b.y); w.w = pack_bf16x2(b.z, b.w);
        *reinterpret_cast<uint4 *>(Wsh + r * ldsh + c) = w;
    }
}

// K-chunk length used by the update for a layer: bounded so that both staged factors of a chunk stay within ~128 MiB
int64_t update_chunk_len(const egr_layer &L)
{
    const int64_t P = (L.flags & EGR_ANTITHETIC) ? L.n_members / 2 : L.n_members;
    const int64_t K = P * L.rank;
    int64_t kc = (int64_t)(64ll << 20) / ((int64_t)L.d_in + L.d_out);
    kc = kc / 64 * 64;
    if (kc < 64) kc = 64;
    if (kc > 8192) kc = 8192;
    const int64_t kpad = (K + 63) / 64 * 64;
    return kc < kpad ? kc : kpad;
}

// One warp waits, with the kernels' bounded wait, on a barrier that nobody completes: after the limit the wait gives up,
// records EGR_ERR_TIMEOUT and the kernel returns normally.
__global__ void __launch_bounds__(32) bounded_wait_probe_kernel(int *status, uint64_t limit_ns)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) { mbar_init(smem_u32(&bar), 1); abort_flag = 0; }
    __syncwarp();
    if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0u, &abort_flag, status, 99, limit_ns);
}

}  // namespace

int launch_bounded_wait_probe(int *status, uint32_t limit_ms, cudaStream_t st)
{
    if (cudaMemsetAsync(status, 0, 8, st) != cudaSuccess) return EGR_ERR_CUDA;
    bounded_wait_probe_kernel<<<1, 32, 0, st>>>(status, (uint64_t)limit_ms * 1000000ull);
    return cuda_ok(cudaGetLastError());
}

// per-band ready counters of the forward, one int per 128 rows
size_t forward_ready_bytes(size_t rows) { return align_up(((rows + BM - 1) / BM) * sizeof(int), 256); }

// The update in one launch: workspace = header, counters (staged items per chunk, factor and 256-row band; CTAs done
// loading per chunk; epilogue warps done per tile), then a ring of kFusedSlots chunk buffers per factor,
// [rows][slots * kc] bf16.  Measured against the launch-by-launch path (alternating in one process, one token per
// member, microseconds): 4096 x 4096 with 65536 noise vectors 1835 against 1980, 32768 antithetic pairs 970 against
// 1050, 16384 x rank 4 and 4096 x rank 16 equal within the noise; a 2048 x 2048 matrix loses (515 against 420: 64 tiles
// leave the CTA pairs short of work per chunk either way, and the ordered epilogues add to it).  So it is used for
// contractions of at least four chunks over matrices of at least two tiles per CTA pair.
constexpr int kFusedSlots = 3;
struct FusedUpdateLayout { int64_t K, Kpad, kc; int n_chunks, n_slots, max_bands, ipr; size_t ready_off, loaded_off, done_off, a_off, b_off, total; };
bool fused_update_layout(const egr_layer &L, FusedUpdateLayout *out)
{
    const int64_t P = (L.flags & EGR_ANTITHETIC) ? L.n_members / 2 : L.n_members;
    const int64_t K = P * L.rank;
    // Ranks of 4 and more stay launch by launch: alternated on one box it was as fast or faster there (4096 x 4096:
    // N = 8192 r = 4 1.08 against 1.17 - 1.26 ms, N = 4096 r = 16 2.05 - 2.10 against 2.20 - 2.27 ms; 8192 x 2048 with
    // N = 32768 r = 4 5.2 - 5.3 against 5.6 - 6.0 ms; only N = 65536 r = 4 was 2 % slower).
    if (L.rank >= 4) return false;
    int64_t kc = update_chunk_len(L);
    const int64_t Kpad = (K + 63) / 64 * 64;
    // Contractions of two or three full chunks are cut into four shorter ones instead (N = 24576: 0.76 - 0.79 against
    // 0.87 - 0.88 ms launch by launch, N = 32768 as antithetic pairs 0.51 against 0.64 - 0.70 ms, N = 12288 0.39 against 0.43)
    if ((K + kc - 1) / kc < 4 && Kpad >= 4 * 2048) kc = ((Kpad + 3) / 4 + 63) / 64 * 64;
    const int64_t n_chunks = (K + kc - 1) / kc;
    const int64_t n_tiles = (int64_t)((L.d_out + PAIR_M - 1) / PAIR_M) * ((L.d_in + BN - 1) / BN);
    if (n_chunks < 4 || n_chunks > 65536 || n_tiles < 2 * (int64_t)(sm_count() / 2)) return false;
    FusedUpdateLayout f;
    f.K = K; f.Kpad = Kpad; f.kc = kc; f.n_chunks = (int)n_chunks;
    f.n_slots = kFusedSlots;
    const int bands_a = (L.d_out + PAIR_M - 1) / PAIR_M, bands_b = (L.d_in + PAIR_M - 1) / PAIR_M;
    f.max_bands = bands_a > bands_b ? bands_a : bands_b;
    f.ipr = (int)((kc / 8 + FUSED_ITEM_GROUPS - 1) / FUSED_ITEM_GROUPS);
    const size_t tiles = (size_t)bands_a * (size_t)((L.d_in + BN - 1) / BN);
    f.ready_off = kWsHeader;
    f.loaded_off = f.ready_off + align_up((size_t)n_chunks * 2 * f.max_bands * sizeof(int), 256);
    f.done_off = f.loaded_off + align_up((size_t)n_chunks * sizeof(int), 256);
    f.a_off = align_up(f.done_off + tiles * sizeof(int), 1024);
    f.b_off = f.a_off + align_up((size_t)L.d_out * f.n_slots * kc * 2, 1024);
    f.total = f.b_off + align_up((size_t)L.d_in * f.n_slots * kc * 2, 1024);
    *out = f;
    return true;
}

size_t gemm_sm100_workspace(const egr_layer &L, int op)
{
    if (op == EGR_OP_PERTURBED_LINEAR) {
        const size_t R = (size_t)L.n_members * L.rows_per_member;
        return kWsHeader + forward_ready_bytes(R) + align_up(R * L.rank * sizeof(float), 256);
    }
    // update chunk by chunk: two staging buffers per factor, so that chunk c+1 is generated while chunk c is contracted;
    // or the one-launch form's ring, whichever is larger (the launch-by-launch path remains the fall-back)
    const int64_t kc = update_chunk_len(L);
    const size_t by_launch = kWsHeader + 2 * (align_up((size_t)L.d_out * kc * 2, 1024) + align_up((size_t)L.d_in * kc * 2, 1024));
    FusedUpdateLayout fl;
    if (fused_update_layout(L, &fl) && fl.total > by_launch) return fl.total;
    return by_launch;
}

namespace {
// logp[row] = logit[row][target] - log sum_j exp(logit[row][j]) from the per-part maxima and sums the forward left
// behind (parts are walked in order, so the result does not depend on which CTA pair wrote what when)
__global__ void __launch_bounds__(256)
loglik_finish_kernel(const float2 *__restrict__ part, int n_part, const float *__restrict__ tgt, const int32_t *__restrict__ targets,
                     int cols, int64_t rows, float *__restrict__ logp)
{
    const int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows) return;
    const int t = targets[row];
    if (t < 0 || t >= cols) { logp[row] = 0.f; return; }
    float m = -INFINITY;
    for (int k = 0; k < n_part; ++k) m = fmaxf(m, part[(int64_t)k * rows + row].x);
    float sum = 0.f;
    for (int k = 0; k < n_part; ++k) {
        const float2 ms = part[(int64_t)k * rows + row];
        sum += ms.y * expf(ms.x - m);
    }
    logp[row] = tgt[row] - (m + logf(sum));
}
}  // namespace

size_t forward_loglik_extra_bytes(const egr_layer &L)
{
    const size_t R = (size_t)L.n_members * L.rows_per_member;
    const size_t n_part = (size_t)((L.d_out + BN - 1) / BN) * EPI_PARTS;
    return align_up(n_part * R * sizeof(float2), 256) + align_up(R * sizeof(float), 256);
}

int launch_forward_bf16(const egr_layer &L, const void *X, const void *W, float coef, const int32_t *rowmap, void *Y,
                        void *ws, size_t ws_bytes, cudaStream_t st, const ColScales *cs, const int32_t *targets, float *logp)
{
    (void)ws_bytes;
    const int64_t R = (int64_t)L.n_members * L.rows_per_member;
    CUtensorMap ta, tb;
    int rc = cached_tmap_2d(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, R, L.d_in, L.ldx, BK, BM);
    if (rc != EGR_OK) return rc;
    // a handful of 256-wide tiles only: 64-wide tiles instead (not for the scaled variants)
    const bool narrow = !cs && !targets && narrow_tiles(R, L.d_out);
    rc = cached_tmap_2d(&tb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, W, L.d_out, L.d_in, L.ldw, BK, narrow ? BN_NARROW / 2 : BNH);
    if (rc != EGR_OK) return rc;
    // workspace: [status, where, side counter | per-band ready counters | s]
    int *status = reinterpret_cast<int *>(ws);
    const size_t ready_bytes = forward_ready_bytes((size_t)R);
    int *ready = reinterpret_cast<int *>((unsigned char *)ws + kWsHeader);
    float *s = reinterpret_cast<float *>((unsigned char *)ws + kWsHeader + ready_bytes);
    // rows of the first row-tile group whose products the side warps add up from two halves (see the kernel): whole
    // bands; none when runs of rows share their noise or when the products come from a pass of their own
    const bool perturb = !(L.flags & EGR_NO_PERTURB);
    int split_rows = 0;
    if (perturb && L.d_in > 1024) {
        const int64_t run = rowmap ? 1 : (int64_t)L.rows_per_member * ((L.flags & EGR_ANTITHETIC) ? 2 : 1);
        // the first row-tile group; every row when there are fewer than two four-row items per side warp (one round
        // of halves and one of whole items would otherwise leave half of the warps without work in the second)
        const int64_t side_warps = 2 * (int64_t)(sm_count() / 2) * (relay_for(EPI_FORWARD, L.rank) ? 7 : FWD_EXTRA_WARPS);
        const int64_t group = (int64_t)GROUP_M * PAIR_M;
        int64_t first = (R < group || R / 4 < 2 * side_warps) ? R : group;
        if (R < 2 * side_warps) {
            // single-row claims (the kernel's rule): halves only where they shorten the last round of claims - a half
            // item costs about 0.55 of a whole one (4096 x 4096, alternating builds: 512 rows at r = 4 0.089 ms whole,
            // 0.099 ms in halves; 256 rows at r = 16 0.252 against 0.148 ms)
            const int64_t rounds_whole = (R + side_warps - 1) / side_warps, rounds_half = (2 * R + side_warps - 1) / side_warps;
            if (!(55 * rounds_half < 100 * rounds_whole)) first = 0;
        }
        if (run % 8 != 0) split_rows = (int)(first / BM * BM);
    }
    if (cudaMemsetAsync(ws, 0, kWsHeader + ready_bytes + (size_t)split_rows * L.rank * sizeof(float), st) != cudaSuccess) return EGR_ERR_CUDA;
    EpiParams ep = {};
    ep.X = reinterpret_cast<const __nv_bfloat16 *>(X); ep.ldx = L.ldx; ep.s_out = s;
    ep.side_counter = status + 2; ep.ready = ready; ep.split_rows = split_rows;
    // Short contractions: a tile's main loop (at most 16 stages) is over before a side warp has reduced the first rows it
    // claimed (their loads come from DRAM), and the first epilogues of every CTA pair would wait for tens of thousands of
    // cycles.  There the skinny products are a pass of their own in front of the GEMM (one warp per four rows, the chip
    // full of them), and the kernel's side warps stay idle.
    if (perturb && L.d_in <= 1024) {
        rc = launch_skinny_xb(L, X, rowmap, s, false, st);
        if (rc != EGR_OK) return rc;
        ep.side_counter = nullptr; ep.ready = nullptr;
    }
    ep.Y = Y; ep.ldy = L.ldy; ep.y_f32 = (L.y_dtype == EGR_F32);
    ep.s = s; ep.coef = coef; ep.T = L.rows_per_member; ep.mbase = L.member_base; ep.rowmap = rowmap; ep.flags = L.flags;
    ep.key = make_noise_key(L.seed, L.layer_id);
    ep.rows = R; ep.cols = L.d_out; ep.K = L.d_in; ep.status = status;
    if (cs) {
        ep.col_scale = reinterpret_cast<const __nv_bfloat16 *>(cs->scales_bf16); ep.x_scale = cs->s_x;
        ep.sigma_s = perturb ? cs->sigma_s : 0.f;
    }
    // bf16 output: 32 x 32 boxes through shared memory (coalesced bulk stores instead of 16-byte pieces per lane)
    CUtensorMap ty;
    const CUtensorMap *typ = nullptr;
    // (the bulk store moves whole 16-byte pieces: a row that ends inside one would spill into the padding)
    if (!targets && L.y_dtype == EGR_BF16 && R < (int64_t)1 << 31 && (L.d_out & 7) == 0) {
        rc = cached_tmap_2d(&ty, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, R, L.d_out, L.ldy, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B);
        if (rc != EGR_OK) return rc;
        ep.y_tma = 1; typ = &ty;
    }
    if (targets) {
        // log-likelihood instead of an output matrix: the partials live behind the forward's own scratch
        const size_t n_part = (size_t)((L.d_out + BN - 1) / BN) * EPI_PARTS;
        unsigned char *extra = (unsigned char *)ws + kWsHeader + ready_bytes + align_up((size_t)R * L.rank * sizeof(float), 256);
        ep.targets = targets;
        ep.ll_part = reinterpret_cast<float2 *>(extra);
        ep.ll_tgt = reinterpret_cast<float *>(extra + align_up(n_part * (size_t)R * sizeof(float2), 256));
        if (perturb) {
            int run_share = 1;
            if (!rowmap) {
                const int64_t run = (int64_t)L.rows_per_member * ((L.flags & EGR_ANTITHETIC) ? 2 : 1);
                run_share = (run % 32 == 0) ? 32 : 1;
            }
            switch (L.rank * (run_share == 32 ? 32 : 1)) {
                case 1:       rc = launch_gemm<EPI_FORWARD, 1, 1, false, BN, true>(ta, tb, ep, st); break;
                case 2:       rc = launch_gemm<EPI_FORWARD, 2, 1, false, BN, true>(ta, tb, ep, st); break;
                case 4:       rc = launch_gemm<EPI_FORWARD, 4, 1, false, BN, true>(ta, tb, ep, st); break;
                case 8:       rc = launch_gemm<EPI_FORWARD, 8, 1, false, BN, true>(ta, tb, ep, st); break;
                case 16:      rc = launch_gemm<EPI_FORWARD, 16, 1, false, BN, true>(ta, tb, ep, st); break;
                case 1 * 32:  rc = launch_gemm<EPI_FORWARD, 1, 32, false, BN, true>(ta, tb, ep, st); break;
                case 2 * 32:  rc = launch_gemm<EPI_FORWARD, 2, 32, false, BN, true>(ta, tb, ep, st); break;
                case 4 * 32:  rc = launch_gemm<EPI_FORWARD, 4, 32, false, BN, true>(ta, tb, ep, st); break;
                case 8 * 32:  rc = launch_gemm<EPI_FORWARD, 8, 32, false, BN, true>(ta, tb, ep, st); break;
                case 16 * 32: rc = launch_gemm<EPI_FORWARD, 16, 32, false, BN, true>(ta, tb, ep, st); break;
                default:      rc = EGR_ERR_BADARG;
            }
        } else {
            rc = launch_gemm<EPI_PLAIN, 0, 1, false, BN, true>(ta, tb, ep, st);
        }
        if (rc != EGR_OK) return rc;
        loglik_finish_kernel<<<(unsigned)((R + 255) / 256), 256, 0, st>>>(ep.ll_part, (int)n_part, ep.ll_tgt, targets, L.d_out, R, logp);
        return cuda_ok(cudaGetLastError());
    }
    if (!perturb) {
        if (cs) return launch_gemm<EPI_PLAIN, 0, 1, true>(ta, tb, ep, st, typ);
        return narrow ? launch_gemm<EPI_PLAIN, 0, 1, false, BN_NARROW>(ta, tb, ep, st, typ) : launch_gemm<EPI_PLAIN, 0>(ta, tb, ep, st, typ);
    }
    // Rows that see the same noise index come in aligned runs of T (2T with antithetic pairs); lanes of such a run
    // share the generation of A_p in the epilogue.  share = the largest of 32, 16, 8, 2 that divides the run length.
    int share = 1;
    if (!rowmap) {
        const int64_t run = (int64_t)L.rows_per_member * ((L.flags & EGR_ANTITHETIC) ? 2 : 1);
        share = (run % 32 == 0) ? 32 : (run % 16 == 0) ? 16 : (run % 8 == 0) ? 8 : (run % 2 == 0) ? 2 : 1;
    }
#define EGR_FWD_CASE(R_)                                                                                              \
    case R_:                                                                                                          \
        if (narrow) switch (share) {                                                                                  \
            case 32: return launch_gemm<EPI_FORWARD, R_, 32, false, BN_NARROW>(ta, tb, ep, st, typ);                  \
            case 16: return launch_gemm<EPI_FORWARD, R_, 16, false, BN_NARROW>(ta, tb, ep, st, typ);                  \
            case 8:  return launch_gemm<EPI_FORWARD, R_, 8, false, BN_NARROW>(ta, tb, ep, st, typ);                   \
            case 2:  return launch_gemm<EPI_FORWARD, R_, 2, false, BN_NARROW>(ta, tb, ep, st, typ);                   \
            default: return launch_gemm<EPI_FORWARD, R_, 1, false, BN_NARROW>(ta, tb, ep, st, typ);                   \
        }                                                                                                             \
        switch (share) {                                                                                              \
            case 32: return launch_gemm<EPI_FORWARD, R_, 32>(ta, tb, ep, st, typ);                                    \
            case 16: return launch_gemm<EPI_FORWARD, R_, 16>(ta, tb, ep, st, typ);                                    \
            case 8:  return launch_gemm<EPI_FORWARD, R_, 8>(ta, tb, ep, st, typ);                                     \
            case 2:  return launch_gemm<EPI_FORWARD, R_, 2>(ta, tb, ep, st, typ);                                     \
            default: return launch_gemm<EPI_FORWARD, R_, 1>(ta, tb, ep, st, typ);                                     \
        }
    // scaled (quantised-matrix) variants: whole warps of one member share, everything else takes the general path
    if (cs) {
        switch (L.rank * ((share == 32) ? 32 : 1)) {
            case 1:       return launch_gemm<EPI_FORWARD, 1, 1, true>(ta, tb, ep, st, typ);
            case 2:       return launch_gemm<EPI_FORWARD, 2, 1, true>(ta, tb, ep, st, typ);
            case 4:       return launch_gemm<EPI_FORWARD, 4, 1, true>(ta, tb, ep, st, typ);
            case 8:       return launch_gemm<EPI_FORWARD, 8, 1, true>(ta, tb, ep, st, typ);
            case 16:      return launch_gemm<EPI_FORWARD, 16, 1, true>(ta, tb, ep, st, typ);
            case 1 * 32:  return launch_gemm<EPI_FORWARD, 1, 32, true>(ta, tb, ep, st, typ);
            case 2 * 32:  return launch_gemm<EPI_FORWARD, 2, 32, true>(ta, tb, ep, st, typ);
            case 4 * 32:  return launch_gemm<EPI_FORWARD, 4, 32, true>(ta, tb, ep, st, typ);
            case 8 * 32:  return launch_gemm<EPI_FORWARD, 8, 32, true>(ta, tb, ep, st, typ);
            case 16 * 32: return launch_gemm<EPI_FORWARD, 16, 32, true>(ta, tb, ep, st, typ);
        }
        return EGR_ERR_BADARG;
    }
    switch (L.rank) {
        EGR_FWD_CASE(1)
        EGR_FWD_CASE(2)
        EGR_FWD_CASE(4)
        EGR_FWD_CASE(8)
        EGR_FWD_CASE(16)
    }
#undef EGR_FWD_CASE
    return EGR_ERR_BADARG;
}

namespace {
// A second stream (and the events that fork from / join back into the caller's stream) on which the factor
// staging of chunk c+1 runs while the tensor cores contract chunk c.  Created once per device, never destroyed.
struct SideStream { cudaStream_t stream = nullptr; cudaEvent_t fork = nullptr, staged[2] = {nullptr, nullptr}, gemm_done[2] = {nullptr, nullptr}; bool ok = false; };

SideStream *side_stream()
{
    static SideStream per_dev[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    SideStream &s = per_dev[dev];
    std::lock_guard<std::mutex> lock(config_mutex());
    if (!s.ok) {
        if (cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        cudaEvent_t *evs[] = {&s.fork, &s.staged[0], &s.staged[1], &s.gemm_done[0], &s.gemm_done[1]};
        for (cudaEvent_t *e : evs)
            if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        s.ok = true;
    }
    return &s;
}
}  // namespace

namespace {
// the reduce-add epilogues never see the sums: the bf16 copy of the master is one more streaming pass
int launch_shadow_bf16(const float *W_master, const egr_layer &L, void *W_shadow, cudaStream_t st)
{
    const int64_t vecs = (int64_t)L.d_out * (L.d_in / 8);
    const int blocks = (int)((vecs + 255) / 256 < 148 * 16 ? (vecs + 255) / 256 : 148 * 16);
    shadow_bf16_kernel<<<blocks, 256, 0, st>>>(W_master, L.ldw, reinterpret_cast<__nv_bfloat16 *>(W_shadow), L.ldw, L.d_out, L.d_in / 8);
    return cuda_ok(cudaGetLastError());
}
}  // namespace

int launch_update_bf16(const egr_layer &L, float *W_master, const float *fitness, float scale, void *W_shadow,
                       float *dW_out, void *ws, size_t ws_bytes, cudaStream_t st)
{
    (void)ws_bytes;
    const int64_t P = (L.flags & EGR_ANTITHETIC) ? L.n_members / 2 : L.n_members;
    const int64_t K = P * L.rank;
    const int64_t kc = update_chunk_len(L);
    int *status = reinterpret_cast<int *>(ws);
    const size_t a_bytes = align_up((size_t)L.d_out * kc * 2, 1024), b_bytes = align_up((size_t)L.d_in * kc * 2, 1024);
    __nv_bfloat16 *At[2], *Bt[2];
    for (int i = 0; i < 2; ++i) {
        At[i] = reinterpret_cast<__nv_bfloat16 *>((unsigned char *)ws + kWsHeader + i * (a_bytes + b_bytes));
        Bt[i] = reinterpret_cast<__nv_bfloat16 *>((unsigned char *)At[i] + a_bytes);
    }
    SideStream *ss = side_stream();
    if (!ss) return EGR_ERR_CUDA;
    if (cudaMemsetAsync(status, 0, 8, st) != cudaSuccess) return EGR_ERR_CUDA;
    const NoiseKey key = make_noise_key(L.seed, L.layer_id);
    const int64_t n_chunks = (K + kc - 1) / kc;
    const bool narrow = narrow_tiles(L.d_out, L.d_in);
    // Short contractions (K <= 2048) are bound by the traffic of W, not by the tensor cores: there W_master += scale * acc
    // goes out as TMA reduce-add stores (no loads of W, no per-lane 16-byte accesses), provided the master can be
    // described by a tensor map and nothing else (dW_out, gradient only) needs the sums in registers; the shadow then
    // costs a separate streaming pass, which requires rows that are whole 16-byte pieces in both precisions.  Long
    // contractions keep the read-modify-write epilogue, which hides behind the main loop and keeps the sixth stage.
    CUtensorMap tw;
    bool reduce_path = K <= 2048 && W_master && !dW_out && (reinterpret_cast<uintptr_t>(W_master) & 15) == 0 && (L.ldw & 3) == 0 &&
                       (L.d_in & 3) == 0 && (!W_shadow || ((L.d_in & 7) == 0 && (L.ldw & 7) == 0));
    if (reduce_path &&
        cached_tmap_2d(&tw, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, W_master, L.d_out, L.d_in, L.ldw, 32, 32) != EGR_OK)
        reduce_path = false;

    FusedUpdateLayout fl;
    if (!reduce_path && fused_update_layout(L, &fl)) {
        // Reduce-add stores whenever the master can be described by a tensor map and nothing needs the sums in registers:
        // the register epilogue's loads and stores of W fill the queue that the generator's special-function instructions
        // share with memory instructions, and the staging warps then fall behind the tensor cores (2.1 ms against 1.6 ms
        // for 4096 x 4096 with 65536 noise vectors).
        CUtensorMap twf;
        bool fused_reduce = W_master && !dW_out && (reinterpret_cast<uintptr_t>(W_master) & 15) == 0 && (L.ldw & 3) == 0 &&
                            (L.d_in & 3) == 0 && (!W_shadow || ((L.d_in & 7) == 0 && (L.ldw & 7) == 0));
        if (fused_reduce &&
            cached_tmap_2d(&twf, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, W_master, L.d_out, L.d_in, L.ldw, 32, 32) != EGR_OK)
            fused_reduce = false;
        // one launch: the kernel's side warps stage the factors chunk by chunk while its tensor cores contract them
        unsigned char *base = (unsigned char *)ws;
        if (cudaMemsetAsync(ws, 0, fl.a_off, st) != cudaSuccess) return EGR_ERR_CUDA;       // status words and all counters
        const int64_t ldk = (int64_t)fl.n_slots * fl.kc;
        CUtensorMap ta, tb;
        int rc = cached_tmap_2d(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base + fl.a_off, L.d_out, ldk, ldk, BK, BM);
        if (rc != EGR_OK) return rc;
        rc = cached_tmap_2d(&tb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base + fl.b_off, L.d_in, ldk, ldk, BK, BNH);
        if (rc != EGR_OK) return rc;
        EpiParams ep = {};
        ep.Wm = W_master; ep.ldw = L.ldw; ep.Wsh = fused_reduce ? nullptr : reinterpret_cast<__nv_bfloat16 *>(W_shadow);
        ep.dW = dW_out; ep.lddw = L.d_in; ep.scale = scale;
        ep.rows = L.d_out; ep.cols = L.d_in; ep.K = (int)fl.Kpad; ep.status = status;
        ep.n_chunks = fl.n_chunks; ep.kc = (int)fl.kc; ep.n_slots = fl.n_slots; ep.K_total = fl.K; ep.fitness = fitness;
        ep.At = reinterpret_cast<__nv_bfloat16 *>(base + fl.a_off); ep.Bt = reinterpret_cast<__nv_bfloat16 *>(base + fl.b_off);
        ep.ldk = ldk; ep.ready_u = reinterpret_cast<int *>(base + fl.ready_off);
        ep.loaded = reinterpret_cast<int *>(base + fl.loaded_off); ep.done = reinterpret_cast<int *>(base + fl.done_off);
        ep.max_bands = fl.max_bands; ep.ipr = fl.ipr; ep.key = key; ep.flags = L.flags; ep.side_counter = status + 2;
        if (fused_reduce) {
            switch (L.rank) {
                case 1:  rc = launch_gemm<EPI_UPDATE_FUSED_REDUCE, 1>(ta, tb, ep, st, &twf); break;
                case 2:  rc = launch_gemm<EPI_UPDATE_FUSED_REDUCE, 2>(ta, tb, ep, st, &twf); break;
                case 4:  rc = launch_gemm<EPI_UPDATE_FUSED_REDUCE, 4>(ta, tb, ep, st, &twf); break;
                case 8:  rc = launch_gemm<EPI_UPDATE_FUSED_REDUCE, 8>(ta, tb, ep, st, &twf); break;
                case 16: rc = launch_gemm<EPI_UPDATE_FUSED_REDUCE, 16>(ta, tb, ep, st, &twf); break;
                default: rc = EGR_ERR_BADARG;
            }
            if (rc != EGR_OK || !W_shadow) return rc;
            return launch_shadow_bf16(W_master, L, W_shadow, st);
        }
        switch (L.rank) {
            case 1:  return launch_gemm<EPI_UPDATE_FUSED, 1>(ta, tb, ep, st);
            case 2:  return launch_gemm<EPI_UPDATE_FUSED, 2>(ta, tb, ep, st);
            case 4:  return launch_gemm<EPI_UPDATE_FUSED, 4>(ta, tb, ep, st);
            case 8:  return launch_gemm<EPI_UPDATE_FUSED, 8>(ta, tb, ep, st);
            case 16: return launch_gemm<EPI_UPDATE_FUSED, 16>(ta, tb, ep, st);
        }
        return EGR_ERR_BADARG;
    }

    auto stage = [&](int64_t c) -> int {
        const int64_t kc0 = c * kc;
        const int len = (int)((K - kc0 < kc) ? (K - kc0) : kc);
        int rc = launch_stage_r(L.rank, At[c & 1], kc, L.d_out, kc0, len, K, fitness, L.flags, key, kTagA, 1, ss->stream);
        if (rc != EGR_OK) return rc;
        rc = launch_stage_r(L.rank, Bt[c & 1], kc, L.d_in, kc0, len, K, fitness, L.flags, key, kTagB, 0, ss->stream);
        if (rc != EGR_OK) return rc;
        return cuda_ok(cudaEventRecord(ss->staged[c & 1], ss->stream));
    };

    // fork: the side stream starts after everything already queued on the caller's stream (fitness, status)
    if (cudaEventRecord(ss->fork, st) != cudaSuccess || cudaStreamWaitEvent(ss->stream, ss->fork, 0) != cudaSuccess)
        return EGR_ERR_CUDA;
    int rc = stage(0);
    if (rc != EGR_OK) return rc;
    for (int64_t c = 0; c < n_chunks; ++c) {
        const int64_t kc0 = c * kc;
        const int len = (int)((K - kc0 < kc) ? (K - kc0) : kc);
        const int len8 = (len + 7) / 8 * 8;
        if (c + 1 < n_chunks) {
            // buffer (c+1)&1 was last read by the contraction of chunk c-1
            if (c >= 1 && cudaStreamWaitEvent(ss->stream, ss->gemm_done[(c + 1) & 1], 0) != cudaSuccess) return EGR_ERR_CUDA;
            rc = stage(c + 1);
            if (rc != EGR_OK) return rc;
        }
        if (cudaStreamWaitEvent(st, ss->staged[c & 1], 0) != cudaSuccess) return EGR_ERR_CUDA;   // join for this chunk
        CUtensorMap ta, tb;
        rc = cached_tmap_2d(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, At[c & 1], L.d_out, len8, kc, BK, BM);
        if (rc != EGR_OK) return rc;
        rc = cached_tmap_2d(&tb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Bt[c & 1], L.d_in, len8, kc, BK, narrow ? BN_NARROW / 2 : BNH);
        if (rc != EGR_OK) return rc;
        EpiParams ep = {};
        ep.Wm = W_master; ep.ldw = L.ldw;
        ep.Wsh = (c + 1 == n_chunks && !reduce_path) ? reinterpret_cast<__nv_bfloat16 *>(W_shadow) : nullptr;
        ep.dW = dW_out; ep.lddw = L.d_in; ep.scale = scale; ep.dw_accumulate = (c > 0);
        ep.rows = L.d_out; ep.cols = L.d_in; ep.K = len8; ep.status = status;
        if (reduce_path)
            rc = narrow ? launch_gemm<EPI_UPDATE_REDUCE, 0, 1, false, BN_NARROW>(ta, tb, ep, st, &tw)
                        : launch_gemm<EPI_UPDATE_REDUCE, 0>(ta, tb, ep, st, &tw);
        else
            rc = narrow ? launch_gemm<EPI_UPDATE, 0, 1, false, BN_NARROW>(ta, tb, ep, st) : launch_gemm<EPI_UPDATE, 0>(ta, tb, ep, st);
        if (rc != EGR_OK) return rc;
        if (cudaEventRecord(ss->gemm_done[c & 1], st) != cudaSuccess) return EGR_ERR_CUDA;
    }
    if (reduce_path && W_shadow) return launch_shadow_bf16(W_master, L, W_shadow, st);
    return EGR_OK;
}

}  // namespace egr

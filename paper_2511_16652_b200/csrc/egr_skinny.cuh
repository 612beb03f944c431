// Warp-level skinny reduction s[rho][k] = sum_l X[rho][l] * B_p[l][k] for a group of up to four consecutive
// rows (Section 4.2: "a batch of N vector-vector dot products").  The caller's warp owns the rows; B_p is
// regenerated in registers and never stored.
//
// Lane `lane` takes Philox blocks q = lane, lane+32, ...  Because 128 is a multiple of r, the rank columns a
// lane touches are the same in every iteration: the partial sums stay in four registers per row and the final
// reduction is a handful of warp shuffles.  Rows that belong to the same member share one generated block;
// rows of different members (one token per member) run four independent Philox chains per iteration.
#pragma once
#include "egr_device.cuh"

namespace egr {

template <typename XT> struct XVec4;
template <> struct XVec4<float> {
    typedef float4 raw_t;
    static __device__ __forceinline__ raw_t load_raw(const float *p) { return *reinterpret_cast<const float4 *>(p); }
    static __device__ __forceinline__ void unpack(const raw_t &v, float (&x)[4]) { x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w; }
    static __device__ __forceinline__ void load(const float *p, float (&x)[4]) { unpack(load_raw(p), x); }
};
template <> struct XVec4<__nv_bfloat16> {
    typedef uint2 raw_t;
    static __device__ __forceinline__ raw_t load_raw(const __nv_bfloat16 *p) { return *reinterpret_cast<const uint2 *>(p); }
    static __device__ __forceinline__ void unpack(const raw_t &v, float (&x)[4]) {
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
    }
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&x)[4]) { unpack(load_raw(p), x); }
};

// rows row0 .. row0+nrows-1 (nrows <= 4), all inside the matrix.  s is dense [R][RANK].
// vec_ok: X rows are 4-element aligned (pitch multiple of 4 and base aligned), enabling vector loads for RANK 1.
// HALVES: only the first (half = 0) or second (half = 1) half of the rows' generator blocks, added to s (which the
// caller has zeroed) with atomics - two addends onto zero give the same bits in either order.  A template parameter,
// so that the whole-row form keeps its code.
template <typename XT, int RANK, bool PRECISE, bool HALVES = false>
__device__ __forceinline__ void skinny_rows4(const XT *__restrict__ X, int64_t ldx, int n, int T, int mbase, const int32_t *__restrict__ rowmap,
                                             uint32_t flags,
                                             const NoiseKey &key, int64_t row0, int nrows, float *__restrict__ s,
                                             int lane, int half = 0)
{
    uint32_t p[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        float sign;
        const int64_t row = row0 + (g < nrows ? g : 0);
        member_noise(member_of(rowmap, mbase, row, T), flags, p[g], sign);
    }
    // warp-uniform sharing pattern of the four rows
    const int pattern = (p[0] == p[1] && p[1] == p[2] && p[2] == p[3]) ? 0 : ((p[0] == p[1] && p[2] == p[3]) ? 1 : 2);
    float acc[4][4];
#pragma unroll
    for (int g = 0; g < 4; ++g)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[g][i] = 0.f;

    const int64_t total = (int64_t)n * RANK;
    const int nblocks = (int)((total + 3) >> 2);
    const int q_mid = min(((nblocks / 2 + 31) / 32) * 32, nblocks);            // whole trips of 32 blocks in the first half
    const int q_lo = (HALVES && half == 1) ? q_mid : 0;
    const int q_hi = (HALVES && half == 0) ? q_mid : nblocks;
    // Rank 1 with rows of whole blocks: the loads of the next trip are issued before this trip's normals are generated, so
    // that the memory latency (the rows come from DRAM) overlaps the generator instead of adding to every trip.
    const bool pipelined = (RANK == 1) && (n & 3) == 0;
    typename XVec4<XT>::raw_t xnext[4];
    if (RANK == 1 && pipelined && q_lo + lane < q_hi) {
#pragma unroll
        for (int g = 0; g < 4; ++g) xnext[g] = XVec4<XT>::load_raw(X + (row0 + (g < nrows ? g : 0)) * ldx + (q_lo + lane) * 4);
    }
    for (int q = q_lo + lane; q < q_hi; q += 32) {
        typename XVec4<XT>::raw_t xcur[4];
        if (RANK == 1 && pipelined) {
#pragma unroll
            for (int g = 0; g < 4; ++g) xcur[g] = xnext[g];
            if (q + 32 < q_hi) {
#pragma unroll
                for (int g = 0; g < 4; ++g) xnext[g] = XVec4<XT>::load_raw(X + (row0 + (g < nrows ? g : 0)) * ldx + (q + 32) * 4);
            }
        }
        // Rows with the same noise index (rows of one member, antithetic partners) reuse the block.  The common
        // patterns keep their generator calls in one basic block so that the independent chains interleave.
        float z[4][4];
        {
            const float4 z0 = noise_block<PRECISE>(key, p[0], kTagB, (uint32_t)q);
            z[0][0] = z0.x; z[0][1] = z0.y; z[0][2] = z0.z; z[0][3] = z0.w;
        }
        if (pattern == 0) {                                      // one member
#pragma unroll
            for (int g = 1; g < 4; ++g)
#pragma unroll
                for (int i = 0; i < 4; ++i) z[g][i] = z[0][i];
        } else if (pattern == 1) {                               // two pairs
            const float4 z2 = noise_block<PRECISE>(key, p[2], kTagB, (uint32_t)q);
#pragma unroll
            for (int i = 0; i < 4; ++i) z[1][i] = z[0][i];
            z[2][0] = z2.x; z[2][1] = z2.y; z[2][2] = z2.z; z[2][3] = z2.w;
#pragma unroll
            for (int i = 0; i < 4; ++i) z[3][i] = z[2][i];
        } else {                                                 // anything else: four generator calls
#pragma unroll
            for (int g = 1; g < 4; ++g) {
                const float4 zg = noise_block<PRECISE>(key, p[g], kTagB, (uint32_t)q);
                z[g][0] = zg.x; z[g][1] = zg.y; z[g][2] = zg.z; z[g][3] = zg.w;
            }
        }
        if (RANK >= 4) {
            const int l = (q * 4) / RANK;                       // one input column per block
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                if (g < nrows) {
                    const float x = load_as_float(X + (row0 + g) * ldx + l);
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[g][i] = fmaf(x, z[g][i], acc[g][i]);
                }
            }
        } else if (RANK == 1 && pipelined) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                if (g < nrows) {
                    float x[4];
                    XVec4<XT>::unpack(xcur[g], x);
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[g][0] = fmaf(x[i], z[g][i], acc[g][0]);
                }
            }
        } else if (RANK == 1 && (q * 4 + 3 < n)) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                if (g < nrows) {
                    float x[4];
                    XVec4<XT>::load(X + (row0 + g) * ldx + q * 4, x);
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[g][0] = fmaf(x[i], z[g][i], acc[g][0]);
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int e = q * 4 + i;
                const int l = e / RANK;
                if (l < n) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        if (g < nrows) {
                            const float x = load_as_float(X + (row0 + g) * ldx + l);
                            acc[g][i & (RANK - 1)] = fmaf(x, z[g][i], acc[g][i & (RANK - 1)]);
                        }
                    }
                }
            }
        }
    }
    // lanes whose (4*lane) % RANK agree hold partial sums of the same rank columns
    constexpr int kClasses = (RANK >= 4) ? RANK / 4 : 1;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float v = acc[g][i];
#pragma unroll
            for (int off = 16; off >= kClasses; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            acc[g][i] = v;
        }
    }
    if (lane < kClasses) {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            if (g < nrows) {
                if (RANK >= 4) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (!HALVES) s[(row0 + g) * RANK + lane * 4 + i] = acc[g][i];
                        else atomicAdd(s + (row0 + g) * RANK + lane * 4 + i, acc[g][i]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < RANK; ++i) {
                        if (!HALVES) s[(row0 + g) * RANK + i] = acc[g][i];
                        else atomicAdd(s + (row0 + g) * RANK + i, acc[g][i]);
                    }
                }
            }
        }
    }
}

// The halves form out of line: it runs for the first row-tile group only and must not cost the whole-row form its
// registers or its place in the instruction cache.
template <typename XT, int RANK>
__device__ __noinline__ void skinny_rows4_half(const XT *__restrict__ X, int64_t ldx, int n, int T, int mbase,
                                               const int32_t *__restrict__ rowmap, uint32_t flags, NoiseKey key, int64_t row0,
                                               int nrows, float *__restrict__ s, int lane, int half)
{
    skinny_rows4<XT, RANK, false, true>(X, ldx, n, T, mbase, rowmap, flags, key, row0, nrows, s, lane, half);
}

// Same reduction for NR consecutive rows that all see the same noise index (rows of one member, or of an antithetic
// pair): one generated block per iteration serves all of them.  Used when the run of equal rows is a multiple of NR.
// NW > 1: the run's blocks are dealt out to NW warps (warp `wslot` takes q = lane + 32 wslot, + 32 NW, ...) and this
// warp's partial sums go to part[wslot][NR][RANK] for the caller to add up in a fixed order.
template <typename XT, int RANK, bool PRECISE, int NR, int NW = 1>
__device__ __forceinline__ void skinny_rows_same(const XT *__restrict__ X, int64_t ldx, int n, uint32_t p, const NoiseKey &key,
                                                 int64_t row0, float *__restrict__ s, int lane, int wslot = 0,
                                                 float *__restrict__ part = nullptr)
{
    float acc[NR][4];
#pragma unroll
    for (int g = 0; g < NR; ++g)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[g][i] = 0.f;
    const int64_t total = (int64_t)n * RANK;
    const int nblocks = (int)((total + 3) >> 2);
    auto consume = [&](int q, const float4 &z4) {
        const float z[4] = {z4.x, z4.y, z4.z, z4.w};
        if (RANK >= 4) {
            const int l = (q * 4) / RANK;
#pragma unroll
            for (int g = 0; g < NR; ++g) {
                const float x = load_as_float(X + (row0 + g) * ldx + l);
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[g][i] = fmaf(x, z[i], acc[g][i]);
            }
        } else if (RANK == 1 && (q * 4 + 3 < n)) {
#pragma unroll
            for (int g = 0; g < NR; ++g) {
                float x[4];
                XVec4<XT>::load(X + (row0 + g) * ldx + q * 4, x);
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[g][0] = fmaf(x[i], z[i], acc[g][0]);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int e = q * 4 + i;
                const int l = e / RANK;
                if (l < n) {
#pragma unroll
                    for (int g = 0; g < NR; ++g) {
                        const float x = load_as_float(X + (row0 + g) * ldx + l);
                        acc[g][i & (RANK - 1)] = fmaf(x, z[i], acc[g][i & (RANK - 1)]);
                    }
                }
            }
        }
    };
    // two blocks per trip (q and q + 32, the same rank class), their generator chains walked in lock step
    for (int q = lane + 32 * wslot; q < nblocks; q += 64 * NW) {
        if (PRECISE) {
            consume(q, noise_block<true>(key, p, kTagB, (uint32_t)q));
            if (q + 32 * NW < nblocks) consume(q + 32 * NW, noise_block<true>(key, p, kTagB, (uint32_t)(q + 32 * NW)));
        } else {
            float4 z2[2];
            noise_blocks_lockstep<2>(key, p, kTagB, (uint32_t)q, (uint32_t)(32 * NW), z2);
            consume(q, z2[0]);
            if (q + 32 * NW < nblocks) consume(q + 32 * NW, z2[1]);
        }
    }
    constexpr int kClasses = (RANK >= 4) ? RANK / 4 : 1;
    float *dst = (NW > 1) ? part + (int64_t)wslot * NR * RANK : s + row0 * RANK;
    if constexpr (RANK >= 4 && (4 * NR) % (32 / kClasses) == 0) {
        // Lanes of one class (lane mod kClasses) hold partial sums of the same M = 4 NR accumulators.  Summing them with
        // one shuffle tree per accumulator costs 5 M shuffles; here every step halves the list instead: partners keep one
        // half each and add the other's copy of it, so that after the last step every lane owns M / (32 / kClasses)
        // finished sums (M - M / lanes shuffles in all).
        constexpr int M = 4 * NR;
        constexpr int kGroup = 32 / kClasses;                     // lanes that share a class
        float v[M];
#pragma unroll
        for (int g = 0; g < NR; ++g)
#pragma unroll
            for (int i = 0; i < 4; ++i) v[g * 4 + i] = acc[g][i];
        int first = 0;                                            // index of v[0] in the original list
#pragma unroll
        for (int off = 16, cnt = M; off >= kClasses; off >>= 1, cnt >>= 1) {
            const bool upper = (lane & off) != 0;
#pragma unroll
            for (int j = 0; j < cnt / 2; ++j) {
                const float mine = upper ? v[j + cnt / 2] : v[j];
                const float theirs = upper ? v[j] : v[j + cnt / 2];
                v[j] = mine + __shfl_xor_sync(0xffffffffu, theirs, off);
            }
            if (upper) first += cnt / 2;
        }
        constexpr int kMine = M / kGroup;
        const int cls = lane & (kClasses - 1);
#pragma unroll
        for (int j = 0; j < kMine; ++j) {
            const int idx = first + j;                            // accumulator (g, i) = (idx / 4, idx % 4)
            dst[(idx >> 2) * RANK + cls * 4 + (idx & 3)] = v[j];
        }
    } else {
#pragma unroll
        for (int g = 0; g < NR; ++g) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float v = acc[g][i];
#pragma unroll
                for (int off = 16; off >= kClasses; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
                acc[g][i] = v;
            }
        }
        if (lane < kClasses) {
#pragma unroll
            for (int g = 0; g < NR; ++g) {
                if (RANK >= 4) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) dst[g * RANK + lane * 4 + i] = acc[g][i];
                } else {
#pragma unroll
                    for (int i = 0; i < RANK; ++i) dst[g * RANK + i] = acc[g][i];
                }
            }
        }
    }
}

}  // namespace egr

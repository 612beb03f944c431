// fp32 path (plain FMA kernels) and the kernels every path shares: noise materialisation for tests,
// the skinny reduction s = X B_p (Section 4.2: "a batch of N vector-vector dot products"), the fp32
// perturbed forward and the fp32 EGGROLL update.
#include <type_traits>

#include "egr_device.cuh"
#include "egr_internal.h"
#include "egr_skinny.cuh"

namespace egr {

// ------------------------------------------------------------------------------------------------
// debug: Philox words and materialised factors
// ------------------------------------------------------------------------------------------------
__global__ void philox_kernel(const uint32_t *__restrict__ ctr, uint32_t k0, uint32_t k1, int64_t count,
                              uint32_t *__restrict__ out)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    const uint4 c = reinterpret_cast<const uint4 *>(ctr)[i];
    reinterpret_cast<uint4 *>(out)[i] = philox4x32_10(c.x, c.y, c.z, c.w, k0, k1);
}

int launch_philox_device(const uint32_t *ctr, uint32_t k0, uint32_t k1, int64_t count, uint32_t *out,
                         cudaStream_t st)
{
    if (count == 0) return EGR_OK;
    const int threads = 256;
    philox_kernel<<<(unsigned)((count + threads - 1) / threads), threads, 0, st>>>(ctr, k0, k1, count, out);
    return cuda_ok(cudaGetLastError());
}

template <bool PRECISE>
__global__ void noise_materialize_kernel(NoiseKey key, uint32_t p, uint32_t tag, int64_t count, float *__restrict__ out)
{
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q * 4 >= count) return;
    const float4 z = noise_block<PRECISE>(key, p, tag, (uint32_t)q);
    const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (q * 4 + i < count) out[q * 4 + i] = zz[i];
}

int launch_noise_materialize(const egr_layer &L, uint32_t p, int which, int precise, float *out, cudaStream_t st)
{
    const int64_t count = (int64_t)(which == 0 ? L.d_out : L.d_in) * L.rank;
    const int64_t blocks4 = (count + 3) / 4;
    const int threads = 256;
    const unsigned grid = (unsigned)((blocks4 + threads - 1) / threads);
    const NoiseKey key = make_noise_key(L.seed, L.layer_id);
    if (precise) noise_materialize_kernel<true><<<grid, threads, 0, st>>>(key, p, which ? kTagB : kTagA, count, out);
    else         noise_materialize_kernel<false><<<grid, threads, 0, st>>>(key, p, which ? kTagB : kTagA, count, out);
    return cuda_ok(cudaGetLastError());
}

// ------------------------------------------------------------------------------------------------
// skinny reduction as a stand-alone kernel (fp32 path): one warp per group of four consecutive rows.
// ------------------------------------------------------------------------------------------------
template <typename XT, int R, bool PRECISE>
__global__ void __launch_bounds__(256)
skinny_xb_kernel(const XT *__restrict__ X, int64_t ldx, int n, int64_t rows, int T, int mbase,
                 const int32_t *__restrict__ rowmap, uint32_t flags, NoiseKey key, float *__restrict__ s)
{
    const int lane = threadIdx.x & 31;
    const int64_t item = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t row0 = item * 4;
    if (row0 >= rows) return;
    const int nrows = (int)min((int64_t)4, rows - row0);
    skinny_rows4<XT, R, PRECISE>(X, ldx, n, T, mbase, rowmap, flags, key, row0, nrows, s, lane);
}

// Rows that come in aligned runs of NR rows with one noise index (the rows of a member, or of an antithetic pair): one
// block of four warps per run.  The warps split the run's generator blocks four ways (B_p is generated once per run, not
// once per four rows) and their partial sums are added in warp order, so the result does not depend on timing.
template <typename XT, int R, bool PRECISE, int NR>
__global__ void __launch_bounds__(128)
skinny_runs_kernel(const XT *__restrict__ X, int64_t ldx, int n, int64_t rows, int T, int mbase, uint32_t flags, NoiseKey key,
                   float *__restrict__ s, int xs_pitch)
{
    __shared__ float part[4 * NR * R];
    extern __shared__ __align__(16) unsigned char xs_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row0 = (int64_t)blockIdx.x * NR;
    if (row0 >= rows) return;
    uint32_t p; float sign;
    member_noise(member_of(nullptr, mbase, row0, T), flags, p, sign);
    if (xs_pitch > 0) {
        // the run's rows go through shared memory: 16-byte loads that cover whole rows, instead of one 2- or 4-byte load
        // per row and generator block (a lane's block stands for a single input element when r >= 4)
        XT *xs = reinterpret_cast<XT *>(xs_raw);
        constexpr int kVec = 16 / (int)sizeof(XT);
        const int nv = n / kVec;
        for (int i = threadIdx.x; i < NR * nv; i += 128) {
            const int g = i / nv, v = i % nv;
            reinterpret_cast<uint4 *>(xs + (int64_t)g * xs_pitch)[v] = reinterpret_cast<const uint4 *>(X + (row0 + g) * ldx)[v];
        }
        for (int i = threadIdx.x; i < NR * (n - nv * kVec); i += 128) {
            const int g = i / (n - nv * kVec), l = nv * kVec + i % (n - nv * kVec);
            xs[(int64_t)g * xs_pitch + l] = X[(row0 + g) * ldx + l];
        }
        __syncthreads();
        skinny_rows_same<XT, R, PRECISE, NR, 4>(xs, xs_pitch, n, p, key, 0, s, lane, warp, part);
    } else {
        skinny_rows_same<XT, R, PRECISE, NR, 4>(X, ldx, n, p, key, row0, s, lane, warp, part);
    }
    __syncthreads();
    for (int t = threadIdx.x; t < NR * R; t += 128)
        s[row0 * R + t] = ((part[t] + part[NR * R + t]) + part[2 * NR * R + t]) + part[3 * NR * R + t];
}

// The same for bf16 rows whose factor fits shared memory (n r floats, at most 32 KB): the block first generates B_p
// once into shared memory (every thread its share of the blocks, four generator chains in lock step), then each lane
// takes a few rows of the run and the columns of its warp's quarter that fall to its sub-lane, eight at a time (one
// 16-byte load per row, the factor's entries from shared memory).  A lane keeps 4 r partial sums instead of NR r and
// the rows are not staged, so more blocks are resident and the rows' loads overlap other blocks' generator phases.
// Partial sums are added over sub-lanes by shuffles and over warps in warp order.
template <int R, int NR>
__global__ void __launch_bounds__(128)
skinny_runs_smemB_kernel(const __nv_bfloat16 *__restrict__ X, int64_t ldx, int n, int64_t rows, int T, int mbase, uint32_t flags,
                         NoiseKey key, float *__restrict__ s)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *Bs = reinterpret_cast<float *>(smem_raw);                 // [n][R]
    __shared__ float part[4 * NR * R];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row0 = (int64_t)blockIdx.x * NR;
    if (row0 >= rows) return;
    uint32_t p; float sign;
    member_noise(member_of(nullptr, mbase, row0, T), flags, p, sign);
    // ---- the factor: element l R + k at Bs[l R + k + 4 (l / 8)], block q covers elements 4 q .. 4 q + 3 (one chunk of
    // eight columns).  The 16 bytes of padding per chunk put the entries that the sub-lanes of a quarter warp read at
    // the same time - the same column of consecutive chunks, 32 R bytes apart - into different banks.
    const int nb = (n * R + 3) >> 2;
    auto slot = [](int q) { return q + ((4 * q) / R) / 8; };
    for (int q = threadIdx.x; q < nb; q += 4 * 128) {
        if (q + 3 * 128 < nb) {
            float4 z[4];
            noise_blocks_lockstep<4>(key, p, kTagB, (uint32_t)q, 128u, z);
#pragma unroll
            for (int j = 0; j < 4; ++j) reinterpret_cast<float4 *>(Bs)[slot(q + j * 128)] = z[j];
        } else {
            for (int qq = q; qq < nb; qq += 128) reinterpret_cast<float4 *>(Bs)[slot(qq)] = noise_block<false>(key, p, kTagB, (uint32_t)qq);
        }
    }
    __syncthreads();
    // ---- the products: lane = (row group, sub-lane); a lane takes RPL rows of the run and those chunks of eight columns
    // of its warp's quarter that fall to its sub-lane (a factor entry read from shared memory serves RPL rows; the
    // sub-lanes of a quarter warp read different entries, so a load's passes carry different data)
    constexpr int RPL = (R <= 4) ? 4 : 2;
    constexpr int kGroups = NR / RPL, kSub = 32 / kGroups;
    const int grp = lane / kSub, sub = lane % kSub;
    const int chunks = n >> 3;                                       // n is a multiple of 8 (checked by the launcher)
    const int c_lo = (int)((int64_t)chunks * warp / 4), c_hi = (int)((int64_t)chunks * (warp + 1) / 4);
    float acc[RPL][R];
#pragma unroll
    for (int g = 0; g < RPL; ++g)
#pragma unroll
        for (int k = 0; k < R; ++k) acc[g][k] = 0.f;
    const __nv_bfloat16 *xrow = X + (row0 + grp * RPL) * ldx;
    for (int c = c_lo + sub; c < c_hi; c += kSub) {
        uint4 xv[RPL];
#pragma unroll
        for (int g = 0; g < RPL; ++g) xv[g] = *reinterpret_cast<const uint4 *>(xrow + g * ldx + 8 * c);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float x[RPL];
#pragma unroll
            for (int g = 0; g < RPL; ++g) {
                const uint32_t w = (j >> 1) == 0 ? xv[g].x : (j >> 1) == 1 ? xv[g].y : (j >> 1) == 2 ? xv[g].z : xv[g].w;
                x[g] = __uint_as_float((j & 1) ? (w & 0xffff0000u) : (w << 16));
            }
            const float *b = Bs + (size_t)(8 * c + j) * R + 4 * c;
            if constexpr (R % 4 == 0) {
#pragma unroll
                for (int k = 0; k < R; k += 4) {
                    const float4 b4 = *reinterpret_cast<const float4 *>(b + k);
#pragma unroll
                    for (int g = 0; g < RPL; ++g) {
                        acc[g][k] = fmaf(x[g], b4.x, acc[g][k]); acc[g][k + 1] = fmaf(x[g], b4.y, acc[g][k + 1]);
                        acc[g][k + 2] = fmaf(x[g], b4.z, acc[g][k + 2]); acc[g][k + 3] = fmaf(x[g], b4.w, acc[g][k + 3]);
                    }
                }
            } else if constexpr (R == 2) {
                const float2 b2 = *reinterpret_cast<const float2 *>(b);
#pragma unroll
                for (int g = 0; g < RPL; ++g) { acc[g][0] = fmaf(x[g], b2.x, acc[g][0]); acc[g][1] = fmaf(x[g], b2.y, acc[g][1]); }
            } else {
                const float b1 = b[0];
#pragma unroll
                for (int g = 0; g < RPL; ++g) acc[g][0] = fmaf(x[g], b1, acc[g][0]);
            }
        }
    }
    // the sub-lanes of a row group are consecutive lanes
#pragma unroll
    for (int g = 0; g < RPL; ++g)
#pragma unroll
        for (int k = 0; k < R; ++k) {
#pragma unroll
            for (int off = kSub / 2; off >= 1; off >>= 1) acc[g][k] += __shfl_xor_sync(0xffffffffu, acc[g][k], off);
        }
    if (sub == 0) {
#pragma unroll
        for (int g = 0; g < RPL; ++g)
#pragma unroll
            for (int k = 0; k < R; ++k) part[(warp * NR + grp * RPL + g) * R + k] = acc[g][k];
    }
    __syncthreads();
    for (int t = threadIdx.x; t < NR * R; t += 128)
        s[row0 * R + t] = ((part[t] + part[NR * R + t]) + part[2 * NR * R + t]) + part[3 * NR * R + t];
}

template <typename XT, int R, bool PRECISE>
static int launch_skinny_xb_r(const egr_layer &L, const XT *X, const int32_t *rowmap, float *s, cudaStream_t st)
{
    const int threads = 256;
    const int64_t rows = (int64_t)L.n_members * L.rows_per_member;
    const int64_t run = (int64_t)L.rows_per_member * ((L.flags & EGR_ANTITHETIC) ? 2 : 1);
    if (!rowmap && run % 8 == 0 && rows % 8 == 0 && rows / 8 < (int64_t)1 << 31) {
        const NoiseKey key = make_noise_key(L.seed, L.layer_id);
        // rows staged in shared memory when a run fits the 48 KB a kernel has without opting in for more
        const int nr = (run % 16 == 0) ? 16 : 8;
        if constexpr (std::is_same<XT, __nv_bfloat16>::value && !PRECISE) {
            // the form with the factor in shared memory: whole 16-byte pieces of every row, a factor of at most 32 KB
            const size_t b_bytes = (size_t)((L.d_in * R + 3) / 4) * 16 + (size_t)(L.d_in / 8) * 16;     // with the padding per chunk
            if ((L.d_in & 7) == 0 && (L.ldx & 7) == 0 && (reinterpret_cast<uintptr_t>(X) & 15) == 0 && b_bytes <= 32 * 1024) {
                if (nr == 16)
                    skinny_runs_smemB_kernel<R, 16><<<(unsigned)(rows / 16), 128, b_bytes, st>>>(
                        X, L.ldx, L.d_in, rows, L.rows_per_member, L.member_base, L.flags, key, s);
                else
                    skinny_runs_smemB_kernel<R, 8><<<(unsigned)(rows / 8), 128, b_bytes, st>>>(
                        X, L.ldx, L.d_in, rows, L.rows_per_member, L.member_base, L.flags, key, s);
                return cuda_ok(cudaGetLastError());
            }
        }
        const int pitch = (L.d_in + 7) / 8 * 8;                       // keeps every staged row 16-byte aligned
        const size_t xs_bytes = (size_t)nr * pitch * sizeof(XT);
        const bool staged = xs_bytes + 4 * 16 * 16 * sizeof(float) <= 48 * 1024;
        if (nr == 16)
            skinny_runs_kernel<XT, R, PRECISE, 16><<<(unsigned)(rows / 16), 128, staged ? xs_bytes : 0, st>>>(
                X, L.ldx, L.d_in, rows, L.rows_per_member, L.member_base, L.flags, key, s, staged ? pitch : 0);
        else
            skinny_runs_kernel<XT, R, PRECISE, 8><<<(unsigned)(rows / 8), 128, staged ? xs_bytes : 0, st>>>(
                X, L.ldx, L.d_in, rows, L.rows_per_member, L.member_base, L.flags, key, s, staged ? pitch : 0);
        return cuda_ok(cudaGetLastError());
    }
    const int64_t warps = (rows + 3) / 4;
    const unsigned grid = (unsigned)((warps * 32 + threads - 1) / threads);
    skinny_xb_kernel<XT, R, PRECISE><<<grid, threads, 0, st>>>(X, L.ldx, L.d_in, rows, L.rows_per_member, L.member_base, rowmap, L.flags,
                                                               make_noise_key(L.seed, L.layer_id), s);
    return cuda_ok(cudaGetLastError());
}

template <typename XT, bool PRECISE>
static int launch_skinny_xb_t(const egr_layer &L, const XT *X, const int32_t *rowmap, float *s, cudaStream_t st)
{
    switch (L.rank) {
        case 1:  return launch_skinny_xb_r<XT, 1, PRECISE>(L, X, rowmap, s, st);
        case 2:  return launch_skinny_xb_r<XT, 2, PRECISE>(L, X, rowmap, s, st);
        case 4:  return launch_skinny_xb_r<XT, 4, PRECISE>(L, X, rowmap, s, st);
        case 8:  return launch_skinny_xb_r<XT, 8, PRECISE>(L, X, rowmap, s, st);
        case 16: return launch_skinny_xb_r<XT, 16, PRECISE>(L, X, rowmap, s, st);
    }
    return EGR_ERR_BADARG;
}

int launch_skinny_xb(const egr_layer &L, const void *X, const int32_t *rowmap, float *s, bool precise, cudaStream_t st)
{
    if (L.x_dtype == EGR_F32)
        return precise ? launch_skinny_xb_t<float, true>(L, (const float *)X, rowmap, s, st)
                       : launch_skinny_xb_t<float, false>(L, (const float *)X, rowmap, s, st);
    if (L.x_dtype == EGR_BF16)
        return precise ? launch_skinny_xb_t<__nv_bfloat16, true>(L, (const __nv_bfloat16 *)X, rowmap, s, st)
                       : launch_skinny_xb_t<__nv_bfloat16, false>(L, (const __nv_bfloat16 *)X, rowmap, s, st);
    return EGR_ERR_UNSUPPORTED;
}

// ------------------------------------------------------------------------------------------------
// fp32 perturbed forward: 64x64 output tile per CTA, 4x4 outputs per thread, fp32 FMA, then the rank-r
// term with A_p regenerated per output row (Section 4.2: "batched scalar-vector multiplication").
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
forward_f32_kernel(const float *__restrict__ X, int64_t ldx, const float *__restrict__ W, int64_t ldw,
                   float *__restrict__ Y, int64_t ldy, int64_t R, int m, int n, int T, int mbase, int r, uint32_t flags,
                   NoiseKey key, float coef, const float *__restrict__ s, const int32_t *__restrict__ rowmap)
{
    __shared__ float sX[16][64 + 4];
    __shared__ float sW[16][64 + 4];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int64_t row_base = (int64_t)blockIdx.y * 64;
    const int col_base = blockIdx.x * 64;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < n; k0 += 16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = tid + i * 256;
            const int rr = idx >> 4, kk = idx & 15;
            const int64_t row = row_base + rr;
            const int col = col_base + rr;
            const int k = k0 + kk;
            sX[kk][rr] = (row < R && k < n) ? X[row * ldx + k] : 0.f;
            sW[kk][rr] = (col < m && k < n) ? W[(int64_t)col * ldw + k] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = sX[kk][ty * 4 + i]; b[i] = sW[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
    const int col0 = col_base + tx * 4;
    const int lr = ilog2_pow2(r);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t row = row_base + ty * 4 + i;
        if (row >= R) continue;
        float pert[4] = {0.f, 0.f, 0.f, 0.f};
        float c = 0.f;
        if (!(flags & EGR_NO_PERTURB)) {
            uint32_t p; float sign;
            member_noise(member_of(rowmap, mbase, row, T), flags, p, sign);
            c = coef * sign;
            const int e_end = min(col0 + 4, m) * r;
            for (int e = col0 * r; e < e_end; e += 4) {
                const float4 z4 = noise_block<true>(key, p, kTagA, (uint32_t)(e >> 2));
                const float z[4] = {z4.x, z4.y, z4.z, z4.w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int ee = e + u;
                    const int j = (ee >> lr) - col0, k = ee & (r - 1);
                    if (j < 4) {
                        const float sv = s[row * r + k];
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj)
                            if (jj == j) pert[jj] = fmaf(sv, z[u], pert[jj]);
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (col0 + j < m) Y[row * ldy + col0 + j] = apply_act<true>(fmaf(c, pert[j], acc[i][j]), flags & EGR_ACT_MASK);
    }
}

int launch_forward_f32(const egr_layer &L, const float *X, const float *W, float coef, const float *s,
                       const int32_t *rowmap, float *Y, cudaStream_t st)
{
    const int64_t R = (int64_t)L.n_members * L.rows_per_member;
    dim3 grid((unsigned)((L.d_out + 63) / 64), (unsigned)((R + 63) / 64));
    if (grid.y > 65535u) return EGR_ERR_UNSUPPORTED;
    forward_f32_kernel<<<grid, 256, 0, st>>>(X, L.ldx, W, L.ldw, Y, L.ldy, R, L.d_out, L.d_in,
                                             L.rows_per_member, L.member_base, L.rank, L.flags,
                                             make_noise_key(L.seed, L.layer_id), coef, s, rowmap);
    return cuda_ok(cudaGetLastError());
}

// ------------------------------------------------------------------------------------------------
// fp32 EGGROLL update: dW[j][l] = scale * sum_{p,k} g_p A_p[j][k] B_p[l][k], 64x64 tile per CTA.
// The contraction index kappa = p*r + k is walked in chunks of 16; each chunk's A and B slices are
// regenerated into shared memory (one Philox block per thread and side) and consumed by fp32 FMAs.
// Chunk sums are folded into the running total once per chunk (two-level summation).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
update_f32_kernel(float *__restrict__ W, int64_t ldw, const float *__restrict__ fitness, int P, int m, int n,
                  int r, uint32_t flags, NoiseKey key, float scale, float *__restrict__ dW_out)
{
    __shared__ __align__(16) float sA[16][64];
    __shared__ __align__(16) float sB[16][64];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int j0 = blockIdx.y * 64, l0 = blockIdx.x * 64;
    const int lr = ilog2_pow2(r);
    const int bpp = 16 * r;                 // Philox blocks per noise index inside a 64-row tile
    const int pl = tid / bpp, b = tid % bpp;
    const int p_per_chunk = 16 >> lr;       // noise indices per chunk (16 / r)
    const int64_t K = (int64_t)P * r;
    float tot[4][4] = {};
    for (int64_t kc = 0; kc < K; kc += 16) {
        const int64_t p64 = (kc >> lr) + pl;
        const bool live = p64 < P;
        const uint32_t p = (uint32_t)p64;
        float g = 0.f;
        if (live) g = (flags & EGR_ANTITHETIC) ? (fitness[2 * p64] - fitness[2 * p64 + 1]) : fitness[p64];
        float za[4] = {0.f, 0.f, 0.f, 0.f}, zb[4] = {0.f, 0.f, 0.f, 0.f};
        if (live) {
            const float4 a4 = noise_block<true>(key, p, kTagA, (uint32_t)(((int64_t)j0 * r >> 2) + b));
            const float4 b4 = noise_block<true>(key, p, kTagB, (uint32_t)(((int64_t)l0 * r >> 2) + b));
            za[0] = a4.x * g; za[1] = a4.y * g; za[2] = a4.z * g; za[3] = a4.w * g;
            zb[0] = b4.x; zb[1] = b4.y; zb[2] = b4.z; zb[3] = b4.w;
        }
        (void)p_per_chunk;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int el = 4 * b + i;
            const int jl = el >> lr, k = el & (r - 1);
            sA[pl * r + k][jl] = za[i];
            sB[pl * r + k][jl] = zb[i];
        }
        __syncthreads();
        float c[4][4] = {};
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            const float4 a4 = *reinterpret_cast<const float4 *>(&sA[kk][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4 *>(&sB[kk][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w}, bb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) c[i][j] = fmaf(a[i], bb[j], c[i][j]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) tot[i][j] += c[i][j];
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int j = j0 + ty * 4 + i;
        if (j >= m) continue;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const int l = l0 + tx * 4 + jj;
            if (l >= n) continue;
            const float d = scale * tot[i][jj];
            if (dW_out) dW_out[(int64_t)j * n + l] = d;
            W[(int64_t)j * ldw + l] += d;
        }
    }
}

int launch_update_f32(const egr_layer &L, float *W, const float *fitness, float scale, float *dW_out,
                      cudaStream_t st)
{
    const int P = (L.flags & EGR_ANTITHETIC) ? L.n_members / 2 : L.n_members;
    dim3 grid((unsigned)((L.d_in + 63) / 64), (unsigned)((L.d_out + 63) / 64));
    if (grid.y > 65535u) return EGR_ERR_UNSUPPORTED;
    update_f32_kernel<<<grid, 256, 0, st>>>(W, L.ldw, fitness, P, L.d_out, L.d_in, L.rank, L.flags,
                                            make_noise_key(L.seed, L.layer_id), scale, dW_out);
    return cuda_ok(cudaGetLastError());
}

}  // namespace egr

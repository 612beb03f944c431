// Fitness shaping kernels: centred ranks (HFT appendix), z-score, antithetic pair sign (integer
// appendix, "Fitness Shaping").  Element-wise passes use 128-bit accesses.
#include "egr_device.cuh"
#include "egr_internal.h"

namespace egr {

// Total order on fp32 as unsigned keys: NaN -> 0 (worst), -0 == +0, otherwise the usual sign flip.
__device__ __forceinline__ uint32_t order_key(float f)
{
    if (f != f) return 0u;
    f += 0.0f;                                   // -0 -> +0
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// asc_i = #{ j : (key_j, j) < (key_i, i) } is the position of element i after a stable sort by key, so the centred
// ranks come from a least-significant-digit radix sort of (key, index) pairs: four passes of 8-bit digits, each a
// stable counting sort.  Blocks own consecutive chunks of kSortChunk elements; a pass needs, per (digit, block), the
// number of elements with that digit in that block (counted by the previous pass's scatter, or by rank_hist_kernel for
// the first pass), per digit an exclusive scan of those counts over the blocks plus the digit's total, and a scatter
// that keeps the order of equal digits.  The cost is the same for every distribution of the values: all-equal, tied or clustered fitness (scores
// that differ in the last few mantissa bits) sort as fast as continuous ones.
constexpr int kSortThreads = 256;
constexpr int kSortItems = 4;                               // elements per thread
constexpr int kSortChunk = kSortThreads * kSortItems;       // elements per block
constexpr int kDigits = 256;

__host__ __device__ inline int sort_blocks(int N) { return (N + kSortChunk - 1) / kSortChunk; }

// counts of the first pass: hist[d * nblk + b] = #{ e in chunk b : key_e & 255 == d }
__global__ void __launch_bounds__(kSortThreads)
rank_hist_kernel(const float *__restrict__ raw, int N, unsigned int *__restrict__ hist, int nblk)
{
    __shared__ unsigned int h[kDigits];
    h[threadIdx.x] = 0u;
    __syncthreads();
    const int e0 = blockIdx.x * kSortChunk;
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) {
        const int e = e0 + j * kSortThreads + threadIdx.x;
        if (e < N) atomicAdd(&h[order_key(raw[e]) & 255u], 1u);
    }
    __syncthreads();
    hist[threadIdx.x * nblk + blockIdx.x] = h[threadIdx.x];
}

// One warp per digit: exclusive scan, in place, of the digit's counters over the blocks (cnt[d][0 .. nblk)), the digit's
// total, and the clearing of the next pass's counters of that digit.  Consecutive lanes read consecutive blocks.
__global__ void __launch_bounds__(256)
rank_rowscan_kernel(unsigned int *__restrict__ cnt, int nblk, unsigned int *__restrict__ total, unsigned int *__restrict__ next_cnt)
{
    const int lane = threadIdx.x & 31;
    const int d = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (d >= kDigits) return;
    unsigned int *row = cnt + (size_t)d * nblk;
    unsigned int carry = 0;
    for (int b0 = 0; b0 < nblk; b0 += 32) {
        const int b = b0 + lane;
        const unsigned int v = (b < nblk) ? row[b] : 0u;
        unsigned int incl = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int u = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += u;
        }
        if (b < nblk) {
            row[b] = carry + incl - v;
            if (next_cnt) next_cnt[(size_t)d * nblk + b] = 0u;
        }
        carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) total[d] = carry;
}

// Stable scatter of one pass.  PASS 0 reads the raw values (key from the value, index = position), later passes read
// the pairs the previous pass wrote.  A warp owns 32 kSortItems consecutive elements and walks them 32 at a time:
// lanes with the same digit find one another with match.any, the lowest of them advances the warp's counter of that
// digit, and a lane's place among its warp's elements of that digit is the old counter plus the number of lower lanes
// in its group.  The warps' counters are then turned into offsets (lower warps first, on top of the block's scanned
// global offset).  PASS 3 writes the centred rank of every element instead of the pairs; earlier passes also count the
// next pass's digits per destination block.
template <int PASS>
__global__ void __launch_bounds__(kSortThreads)
rank_scatter_kernel(const float *__restrict__ raw, const uint2 *__restrict__ in, int N, const unsigned int *__restrict__ offs,
                    const unsigned int *__restrict__ total, int nblk, uint2 *__restrict__ outp,
                    unsigned int *__restrict__ next_hist, float *__restrict__ out)
{
    constexpr int kWarps = kSortThreads / 32;
    __shared__ unsigned int wcnt[kWarps][kDigits];
    __shared__ unsigned int wsum[kWarps];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kWarps * kDigits; i += kSortThreads) (&wcnt[0][0])[i] = 0u;
    __syncthreads();
    const int e0 = blockIdx.x * kSortChunk + w * (32 * kSortItems);
    uint2 pr[kSortItems];
    unsigned int local[kSortItems];
    const unsigned int lt = (1u << lane) - 1u;
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) {                   // all loads first, so that they are in flight together
        const int e = e0 + j * 32 + lane;
        if (e < N) pr[j] = (PASS == 0) ? make_uint2(order_key(raw[e]), (unsigned int)e) : in[e];
        else pr[j] = make_uint2(0u, 0u);
    }
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) {
        const int e = e0 + j * 32 + lane;
        const bool valid = e < N;
        const unsigned int d = (pr[j].x >> (8 * PASS)) & 255u;
        const unsigned int grp = __match_any_sync(0xffffffffu, valid ? d : (256u + (unsigned int)lane));
        const int leader = __ffs(grp) - 1;
        unsigned int old = 0u;
        if (valid && lane == leader) { old = wcnt[w][d]; wcnt[w][d] = old + (unsigned int)__popc(grp); }
        old = __shfl_sync(0xffffffffu, old, leader);
        local[j] = old + (unsigned int)__popc(grp & lt);
        __syncwarp();
    }
    // one digit per thread: the digit's first position = the totals of all smaller digits (a scan over the 256 threads)
    // plus what the lower blocks hold of this digit
    const unsigned int tot = total[threadIdx.x];
    unsigned int incl = tot;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned int u = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += u;
    }
    if (lane == 31) wsum[w] = incl;
    __syncthreads();
    {
        const int d = threadIdx.x;
        unsigned int run = incl - tot + offs[(size_t)d * nblk + blockIdx.x];
#pragma unroll
        for (int ww = 0; ww < kWarps; ++ww) run += (ww < w) ? wsum[ww] : 0u;
#pragma unroll
        for (int ww = 0; ww < kWarps; ++ww) { const unsigned int c = wcnt[ww][d]; wcnt[ww][d] = run; run += c; }
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) {
        const int e = e0 + j * 32 + lane;
        const bool valid = e < N;
        const unsigned int d = (pr[j].x >> (8 * PASS)) & 255u;
        const unsigned int pos = valid ? wcnt[w][d] + local[j] : 0u;
        if (PASS == 3) {
            if (valid) {
                const float num = (float)(2 * (long long)pos - (long long)(N - 1));
                const float den = (float)(2 * (long long)(N - 1));
                out[pr[j].y] = (N == 1) ? 0.f : __fdiv_rn(num, den);
            }
        } else {
            if (valid) outp[pos] = pr[j];
            // the next pass's counter of this element: lanes that hit the same counter (equal or clustered keys land
            // side by side) add once for all of them
            const unsigned int dn = (pr[j].x >> (8 * (PASS + 1))) & 255u;
            const unsigned int slot = dn * (unsigned int)nblk + pos / kSortChunk;
            const unsigned int grp = __match_any_sync(0xffffffffu, valid ? slot : 0xffffffffu - (unsigned int)lane);
            if (valid && lane == __ffs(grp) - 1) atomicAdd(&next_hist[slot], (unsigned int)__popc(grp));
        }
    }
}

// ---- z-score: three streaming passes, fp64 statistics, deterministic summation order ----
// Each pass runs on up to kStatBlocks blocks (enough to fill the chip for populations of millions; one block per 1024
// members below that), reads with 128-bit loads, and leaves one fp64 partial sum per block; the next pass has every
// block add the partials up again in the same fixed order (thread t takes partials t, t + 256, ..., then the block's
// shuffle tree), so the result does not depend on scheduling.
constexpr int kStatBlocks = 1184;           // 8 blocks per SM on 148 SMs
__host__ __device__ inline int stat_blocks(int N) { const int b = (N + 1023) / 1024; return b < kStatBlocks ? (b < 1 ? 1 : b) : kStatBlocks; }

__device__ __forceinline__ double block_sum(double v)
{
    __shared__ double sh[32];
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += sh[w];
    return t;
}

// sum of `count` partials, the same value in every thread of the block
__device__ __forceinline__ double sum_partials(const double *__restrict__ part, int count)
{
    double v = 0.0;
    for (int b = threadIdx.x; b < count; b += blockDim.x) v += part[b];
    return block_sum(v);
}

// this block's share of sum_i f(raw[i]); f = identity (SQ = false) or squared deviation from `mean`
template <bool SQ>
__device__ __forceinline__ double stream_sum(const float *__restrict__ raw, int N, double mean)
{
    const int n4 = N >> 2;
    double v = 0.0;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += gridDim.x * blockDim.x) {
        const float4 x = reinterpret_cast<const float4 *>(raw)[i];
        if (SQ) {
            const double a = (double)x.x - mean, b = (double)x.y - mean, c = (double)x.z - mean, d = (double)x.w - mean;
            v += (a * a + b * b) + (c * c + d * d);
        } else {
            v += ((double)x.x + (double)x.y) + ((double)x.z + (double)x.w);
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < (N & 3)) {                 // the last one to three members
        const double x = (double)raw[(n4 << 2) + threadIdx.x];
        v += SQ ? (x - mean) * (x - mean) : x;
    }
    return block_sum(v);
}

__global__ void __launch_bounds__(256) zs_sum_kernel(const float *__restrict__ raw, int N, double *__restrict__ part)
{
    const double v = stream_sum<false>(raw, N, 0.0);
    if (threadIdx.x == 0) part[blockIdx.x] = v;
}

__global__ void __launch_bounds__(256) zs_var_kernel(const float *__restrict__ raw, int N, const double *__restrict__ part,
                                                      double *__restrict__ part2)
{
    const double mean = sum_partials(part, gridDim.x) / (double)N;
    const double v = stream_sum<true>(raw, N, mean);
    if (threadIdx.x == 0) part2[blockIdx.x] = v;
}

__global__ void __launch_bounds__(256) zs_apply_kernel(const float *__restrict__ raw, int N, const double *__restrict__ part,
                                                        const double *__restrict__ part2, int n_part, float *__restrict__ out)
{
    const double mean = sum_partials(part, n_part) / (double)N;
    const double var = sum_partials(part2, n_part) / (double)N;
    const double inv = 1.0 / (sqrt(var) + 1e-8);
    const int n4 = N >> 2;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += gridDim.x * blockDim.x) {
        const float4 v = reinterpret_cast<const float4 *>(raw)[i];
        float4 o;
        o.x = (float)(((double)v.x - mean) * inv); o.y = (float)(((double)v.y - mean) * inv);
        o.z = (float)(((double)v.z - mean) * inv); o.w = (float)(((double)v.w - mean) * inv);
        reinterpret_cast<float4 *>(out)[i] = o;
    }
    if (blockIdx.x == 0 && threadIdx.x < (N & 3)) {
        const int t = (n4 << 2) + threadIdx.x;
        out[t] = (float)(((double)raw[t] - mean) * inv);
    }
}

// ---- antithetic sign: two pairs (one float4) per thread ----
__device__ __forceinline__ float signf(float d) { return (d > 0.f) ? 1.f : ((d < 0.f) ? -1.f : 0.f); }

__global__ void __launch_bounds__(256) pair_sign_kernel(const float *__restrict__ raw, int N, float *__restrict__ out)
{
    const int i4 = blockIdx.x * blockDim.x + threadIdx.x;
    const int i = i4 * 4;
    if (i + 3 < N) {
        const float4 v = reinterpret_cast<const float4 *>(raw)[i4];
        const float s0 = signf(v.x - v.y), s1 = signf(v.z - v.w);
        reinterpret_cast<float4 *>(out)[i4] = make_float4(s0, -s0, s1, -s1);
    } else if (i + 1 < N) {
        const float s0 = signf(raw[i] - raw[i + 1]);
        out[i] = s0; out[i + 1] = -s0;
    }
}

// z-score partial sums, or (centred rank) two arrays of 256 counters per block of 1024 members and two of N pairs
size_t fitness_shape_workspace(int N)
{
    const size_t hist_bytes = align_up((size_t)kDigits * sort_blocks(N) * sizeof(unsigned int), 256);
    const size_t pair_bytes = align_up((size_t)N * sizeof(uint2), 256);
    const size_t zscore_bytes = 2 * kStatBlocks * sizeof(double);
    const size_t rank_bytes = 2 * hist_bytes + kDigits * sizeof(unsigned int) + 2 * pair_bytes;
    return kWsHeader + (rank_bytes > zscore_bytes ? rank_bytes : zscore_bytes);
}

int launch_fitness_shape(const float *raw, int N, int mode, float *out, void *ws, cudaStream_t st)
{
    unsigned char *base = (unsigned char *)ws + kWsHeader;
    switch (mode) {
        case EGR_SHAPE_NONE:
            return cuda_ok(cudaMemcpyAsync(out, raw, sizeof(float) * (size_t)N, cudaMemcpyDeviceToDevice, st));
        case EGR_SHAPE_CENTERED_RANK: {
            // scratch: two arrays of per-(digit, block) counters, the digit totals, then two arrays of N (key, index) pairs
            const int nblk = sort_blocks(N);
            const size_t hist_bytes = align_up((size_t)kDigits * nblk * sizeof(unsigned int), 256);
            const size_t pair_bytes = align_up((size_t)N * sizeof(uint2), 256);
            unsigned int *hist[2] = {reinterpret_cast<unsigned int *>(base), reinterpret_cast<unsigned int *>(base + hist_bytes)};
            unsigned int *total = reinterpret_cast<unsigned int *>(base + 2 * hist_bytes);
            unsigned char *pbase = base + 2 * hist_bytes + kDigits * sizeof(unsigned int);
            uint2 *pairs[2] = {reinterpret_cast<uint2 *>(pbase), reinterpret_cast<uint2 *>(pbase + pair_bytes)};
            const int sb = kDigits * 32 / 256;               // blocks of the row scan: one warp per digit
            rank_hist_kernel<<<nblk, kSortThreads, 0, st>>>(raw, N, hist[0], nblk);
            rank_rowscan_kernel<<<sb, 256, 0, st>>>(hist[0], nblk, total, hist[1]);
            rank_scatter_kernel<0><<<nblk, kSortThreads, 0, st>>>(raw, nullptr, N, hist[0], total, nblk, pairs[0], hist[1], nullptr);
            rank_rowscan_kernel<<<sb, 256, 0, st>>>(hist[1], nblk, total, hist[0]);
            rank_scatter_kernel<1><<<nblk, kSortThreads, 0, st>>>(nullptr, pairs[0], N, hist[1], total, nblk, pairs[1], hist[0], nullptr);
            rank_rowscan_kernel<<<sb, 256, 0, st>>>(hist[0], nblk, total, hist[1]);
            rank_scatter_kernel<2><<<nblk, kSortThreads, 0, st>>>(nullptr, pairs[1], N, hist[0], total, nblk, pairs[0], hist[1], nullptr);
            rank_rowscan_kernel<<<sb, 256, 0, st>>>(hist[1], nblk, total, nullptr);
            rank_scatter_kernel<3><<<nblk, kSortThreads, 0, st>>>(nullptr, pairs[0], N, hist[1], total, nblk, nullptr, nullptr, out);
            return cuda_ok(cudaGetLastError());
        }
        case EGR_SHAPE_ZSCORE: {
            double *part = reinterpret_cast<double *>(base);
            double *part2 = part + kStatBlocks;
            const int nb = stat_blocks(N);
            zs_sum_kernel<<<nb, 256, 0, st>>>(raw, N, part);
            zs_var_kernel<<<nb, 256, 0, st>>>(raw, N, part, part2);
            zs_apply_kernel<<<nb, 256, 0, st>>>(raw, N, part, part2, nb, out);
            return cuda_ok(cudaGetLastError());
        }
        case EGR_SHAPE_ANTITHETIC_SIGN: {
            const int n4 = (N + 3) / 4;
            pair_sign_kernel<<<(n4 + 255) / 256, 256, 0, st>>>(raw, N, out);
            return cuda_ok(cudaGetLastError());
        }
    }
    return EGR_ERR_BADARG;
}

// ---- integer pair sign: out[p] = sign(raw[2p] - raw[2p+1]); four pairs per thread ----
__global__ void __launch_bounds__(256) pair_sign_i8_kernel(const int32_t *__restrict__ raw, int P, int8_t *__restrict__ out)
{
    const int p4 = blockIdx.x * blockDim.x + threadIdx.x;
    const int p = p4 * 4;
    if (p + 3 < P) {
        const int4 a = reinterpret_cast<const int4 *>(raw)[2 * p4];
        const int4 b = reinterpret_cast<const int4 *>(raw)[2 * p4 + 1];
        char4 o;
        o.x = (signed char)((a.x > a.y) - (a.x < a.y)); o.y = (signed char)((a.z > a.w) - (a.z < a.w));
        o.z = (signed char)((b.x > b.y) - (b.x < b.y)); o.w = (signed char)((b.z > b.w) - (b.z < b.w));
        reinterpret_cast<char4 *>(out)[p4] = o;
    } else {
        for (int t = p; t < P; ++t) {
            const int32_t x = raw[2 * t], y = raw[2 * t + 1];
            out[t] = (int8_t)((x > y) - (x < y));
        }
    }
}

int launch_fitness_shape_i8(const int32_t *raw, int N, int8_t *out, cudaStream_t st)
{
    const int P = N / 2;
    if (P == 0) return EGR_OK;
    const int n4 = (P + 3) / 4;
    pair_sign_i8_kernel<<<(n4 + 255) / 256, 256, 0, st>>>(raw, P, out);
    return cuda_ok(cudaGetLastError());
}

}  // namespace egr

namespace egr {

// ---- per-question shaping: column statistics in two deterministic passes, then one row pass ----
constexpr int kQBlocks = 64;      // row slabs; partial sums are combined in slab order

// part[b][j] = sum over the rows of slab b of f(S[i][j]);  f = identity (mu == nullptr) or squared deviation
__global__ void __launch_bounds__(256)
q_colsum_kernel(const float *__restrict__ S, int N, int Q, const double *__restrict__ mu, double *__restrict__ part)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int b = blockIdx.y;
    if (j >= Q) return;
    const int rows_per = (N + kQBlocks - 1) / kQBlocks;
    const int i0 = b * rows_per, i1 = min(N, i0 + rows_per);
    const double m = mu ? mu[j] : 0.0;
    double acc = 0.0;
    for (int i = i0; i < i1; ++i) {
        const double v = (double)S[(int64_t)i * Q + j];
        acc += mu ? (v - m) * (v - m) : v;
    }
    part[(int64_t)b * Q + j] = acc;
}

// mu[j] = (sum_b part[b][j]) / N
__global__ void __launch_bounds__(256) q_mean_kernel(const double *__restrict__ part, int N, int Q, double *__restrict__ mu)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= Q) return;
    double acc = 0.0;
    for (int b = 0; b < kQBlocks; ++b) acc += part[(int64_t)b * Q + j];
    mu[j] = acc / (double)N;
}

// inv[0] = 1 / (sqrt(sum_{b,j} part[b][j] / (N Q)) + 1e-8), one block, fixed summation order
__global__ void __launch_bounds__(256) q_scale_kernel(const double *__restrict__ part, int N, int Q, double *__restrict__ inv)
{
    double acc = 0.0;
    for (int64_t t = threadIdx.x; t < (int64_t)kQBlocks * Q; t += blockDim.x) acc += part[t];
    acc = block_sum(acc);
    if (threadIdx.x == 0) inv[0] = 1.0 / (sqrt(acc / ((double)N * (double)Q)) + 1e-8);
}

// out[i] = (1/Q) sum_j (S[i][j] - mu[j]) * inv; one warp per member
__global__ void __launch_bounds__(256)
q_apply_kernel(const float *__restrict__ S, int N, int Q, const double *__restrict__ mu, const double *__restrict__ inv,
               float *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= N) return;
    double acc = 0.0;
    for (int j = lane; j < Q; j += 32) acc += ((double)S[i * Q + j] - mu[j]) * inv[0];
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) out[i] = (float)(acc / (double)Q);
}

int launch_fitness_shape_questions(const float *S, int N, int Q, float *out, void *ws, cudaStream_t st)
{
    double *part = reinterpret_cast<double *>((unsigned char *)ws + kWsHeader);
    double *mu = part + (size_t)kQBlocks * Q;
    double *inv = mu + Q;
    dim3 grid((Q + 255) / 256, kQBlocks);
    q_colsum_kernel<<<grid, 256, 0, st>>>(S, N, Q, nullptr, part);
    q_mean_kernel<<<(Q + 255) / 256, 256, 0, st>>>(part, N, Q, mu);
    q_colsum_kernel<<<grid, 256, 0, st>>>(S, N, Q, mu, part);
    q_scale_kernel<<<1, 256, 0, st>>>(part, N, Q, inv);
    q_apply_kernel<<<(unsigned)(((int64_t)N * 32 + 255) / 256), 256, 0, st>>>(S, N, Q, mu, inv, out);
    return cuda_ok(cudaGetLastError());
}

size_t fitness_shape_questions_ws(int Q) { return kWsHeader + ((size_t)kQBlocks * Q + Q + 8) * sizeof(double); }

// ---- base-3 packing of pair signs: five ternary digits per byte, one byte per thread ----
// ("Base-3 Fitness Packing and Bandwidth Efficiency": +1, 0, -1 -> digits 0, 1, 2; byte = sum digit_i 3^i)
__global__ void __launch_bounds__(256) pack3_kernel(const int8_t *__restrict__ F, int64_t count, uint8_t *__restrict__ packed,
                                                    int64_t n_bytes)
{
    const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= n_bytes) return;
    uint32_t byte = 0, pw = 1;
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        const int64_t e = 5 * b + i;
        const int v = (e < count) ? (int)F[e] : 0;
        byte += (uint32_t)(1 - v) * pw;           // +1 -> 0, 0 -> 1, -1 -> 2
        pw *= 3;
    }
    packed[b] = (uint8_t)byte;
}

__global__ void __launch_bounds__(256) unpack3_kernel(const uint8_t *__restrict__ packed, int64_t count, int8_t *__restrict__ F,
                                                      int64_t n_bytes)
{
    const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= n_bytes) return;
    uint32_t byte = packed[b];
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        const int64_t e = 5 * b + i;
        if (e < count) F[e] = (int8_t)(1 - (int)(byte % 3u));
        byte /= 3u;
    }
}

int launch_pack3(const int8_t *F, int64_t count, uint8_t *packed, cudaStream_t st)
{
    const int64_t n_bytes = (count + 4) / 5;
    if (n_bytes == 0) return EGR_OK;
    pack3_kernel<<<(unsigned)((n_bytes + 255) / 256), 256, 0, st>>>(F, count, packed, n_bytes);
    return cuda_ok(cudaGetLastError());
}

int launch_unpack3(const uint8_t *packed, int64_t count, int8_t *F, cudaStream_t st)
{
    const int64_t n_bytes = (count + 4) / 5;
    if (n_bytes == 0) return EGR_OK;
    unpack3_kernel<<<(unsigned)((n_bytes + 255) / 256), 256, 0, st>>>(packed, count, F, n_bytes);
    return cuda_ok(cudaGetLastError());
}

}  // namespace egr

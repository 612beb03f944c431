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

// asc_i = #{ j : (key_j, j) < (key_i, i) } without sorting everything:
//   1. histogram of the top 16 key bits (65536 buckets)
//   2. exclusive scan of the histogram              -> number of elements in lower buckets
//   3. scatter of (key, index) pairs into bucket order (order inside a bucket is arbitrary)
//   4. each element counts the smaller pairs inside its own bucket and adds the bucket's base
// For continuous fitness values a bucket holds a handful of elements, so step 4 is short; when many values are
// identical it degrades gracefully to the all-pairs count, which is still exact.
constexpr int kBuckets = 1 << 16;

__global__ void __launch_bounds__(256)
rank_hist_kernel(const float *__restrict__ raw, int N, unsigned int *__restrict__ hist)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N) atomicAdd(&hist[order_key(raw[i]) >> 16], 1u);
}

// one block of 32 warps: exclusive scan of 65536 counters.  Warp w owns the contiguous range [2048 w, 2048 (w+1))
// and walks it in 64 coalesced rows of 32, carrying the running sum; warp totals are then scanned in shared memory.
__global__ void __launch_bounds__(1024)
rank_scan_kernel(const unsigned int *__restrict__ hist, unsigned int *__restrict__ base, unsigned int *__restrict__ cursor)
{
    __shared__ unsigned int warp_tot[32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const unsigned int *h = hist + w * 2048;
    unsigned int excl[64];
    unsigned int carry = 0;
#pragma unroll
    for (int k = 0; k < 64; ++k) {
        const unsigned int v = h[k * 32 + lane];
        unsigned int incl = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int u = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += u;
        }
        excl[k] = carry + incl - v;
        carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) warp_tot[w] = carry;
    __syncthreads();
    if (w == 0) {
        const unsigned int t = warp_tot[lane];
        unsigned int incl = t;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int u = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += u;
        }
        warp_tot[lane] = incl - t;                      // exclusive offset of each warp's range
    }
    __syncthreads();
    const unsigned int woff = warp_tot[w];
#pragma unroll
    for (int k = 0; k < 64; ++k) {
        base[w * 2048 + k * 32 + lane] = woff + excl[k];
        cursor[w * 2048 + k * 32 + lane] = 0u;
    }
}

__global__ void __launch_bounds__(256)
rank_scatter_kernel(const float *__restrict__ raw, int N, const unsigned int *__restrict__ base,
                    unsigned int *__restrict__ cursor, uint2 *__restrict__ pairs)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const uint32_t k = order_key(raw[i]);
    const unsigned int slot = base[k >> 16] + atomicAdd(&cursor[k >> 16], 1u);
    pairs[slot] = make_uint2(k, (unsigned int)i);
}

__global__ void __launch_bounds__(256)
rank_finish_kernel(const float *__restrict__ raw, int N, const unsigned int *__restrict__ base,
                   const unsigned int *__restrict__ hist, const uint2 *__restrict__ pairs, float *__restrict__ out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    if (N == 1) { out[i] = 0.f; return; }
    const uint32_t k = order_key(raw[i]);
    const unsigned int b0 = base[k >> 16], cnt = hist[k >> 16];
    const unsigned long long ci = ((unsigned long long)k << 32) | (unsigned int)i;
    unsigned int asc = b0;
    for (unsigned int t = 0; t < cnt; ++t) {
        const uint2 pr = pairs[b0 + t];
        const unsigned long long cj = ((unsigned long long)pr.x << 32) | pr.y;
        asc += (cj < ci) ? 1u : 0u;
    }
    const float num = (float)(2 * (long long)asc - (long long)(N - 1));
    const float den = (float)(2 * (long long)(N - 1));
    out[i] = __fdiv_rn(num, den);
}

// ---- z-score: three small passes, fp64 statistics, deterministic summation order ----
constexpr int kStatBlocks = 128;

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

__global__ void __launch_bounds__(256) zs_sum_kernel(const float *__restrict__ raw, int N, double *__restrict__ part)
{
    double v = 0.0;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < N; i += gridDim.x * blockDim.x) v += (double)raw[i];
    v = block_sum(v);
    if (threadIdx.x == 0) part[blockIdx.x] = v;
}

__global__ void __launch_bounds__(256) zs_var_kernel(const float *__restrict__ raw, int N, const double *__restrict__ part,
                                                      double *__restrict__ part2)
{
    double mean = 0.0;
    for (int b = 0; b < kStatBlocks; ++b) mean += part[b];
    mean /= (double)N;
    double v = 0.0;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < N; i += gridDim.x * blockDim.x) {
        const double d = (double)raw[i] - mean;
        v += d * d;
    }
    v = block_sum(v);
    if (threadIdx.x == 0) part2[blockIdx.x] = v;
}

__global__ void __launch_bounds__(256) zs_apply_kernel(const float *__restrict__ raw, int N, const double *__restrict__ part,
                                                        const double *__restrict__ part2, float *__restrict__ out)
{
    double mean = 0.0, var = 0.0;
    for (int b = 0; b < kStatBlocks; ++b) { mean += part[b]; var += part2[b]; }
    mean /= (double)N; var /= (double)N;
    const double inv = 1.0 / (sqrt(var) + 1e-8);
    const int i4 = blockIdx.x * blockDim.x + threadIdx.x;
    const int i = i4 * 4;
    if (i + 3 < N) {
        const float4 v = reinterpret_cast<const float4 *>(raw)[i4];
        float4 o;
        o.x = (float)(((double)v.x - mean) * inv); o.y = (float)(((double)v.y - mean) * inv);
        o.z = (float)(((double)v.z - mean) * inv); o.w = (float)(((double)v.w - mean) * inv);
        reinterpret_cast<float4 *>(out)[i4] = o;
    } else {
        for (int t = i; t < N; ++t) out[t] = (float)(((double)raw[t] - mean) * inv);
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

int launch_fitness_shape(const float *raw, int N, int mode, float *out, void *ws, cudaStream_t st)
{
    unsigned char *base = (unsigned char *)ws + kWsHeader;
    switch (mode) {
        case EGR_SHAPE_NONE:
            return cuda_ok(cudaMemcpyAsync(out, raw, sizeof(float) * (size_t)N, cudaMemcpyDeviceToDevice, st));
        case EGR_SHAPE_CENTERED_RANK: {
            // scratch: histogram, bucket bases, cursors (65536 counters each), then N (key, index) pairs
            unsigned int *hist = reinterpret_cast<unsigned int *>(base);
            unsigned int *bbase = hist + kBuckets;
            unsigned int *cursor = bbase + kBuckets;
            uint2 *pairs = reinterpret_cast<uint2 *>(cursor + kBuckets);
            if (cudaMemsetAsync(hist, 0, sizeof(unsigned int) * kBuckets, st) != cudaSuccess) return EGR_ERR_CUDA;
            const int bx = (N + 255) / 256;
            rank_hist_kernel<<<bx, 256, 0, st>>>(raw, N, hist);
            rank_scan_kernel<<<1, 1024, 0, st>>>(hist, bbase, cursor);
            rank_scatter_kernel<<<bx, 256, 0, st>>>(raw, N, bbase, cursor, pairs);
            rank_finish_kernel<<<bx, 256, 0, st>>>(raw, N, bbase, hist, pairs, out);
            return cuda_ok(cudaGetLastError());
        }
        case EGR_SHAPE_ZSCORE: {
            double *part = reinterpret_cast<double *>(base);
            double *part2 = part + kStatBlocks;
            zs_sum_kernel<<<kStatBlocks, 256, 0, st>>>(raw, N, part);
            zs_var_kernel<<<kStatBlocks, 256, 0, st>>>(raw, N, part, part2);
            const int n4 = (N + 3) / 4;
            zs_apply_kernel<<<(n4 + 255) / 256, 256, 0, st>>>(raw, N, part, part2, out);
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

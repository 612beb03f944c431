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

// asc_i = #{ j : (key_j, j) < (key_i, i) }.  One thread per i, all j streamed through shared memory.
// The j range can be split over blockIdx.y; partial counts are then summed with atomics into `counts`.
constexpr int kRankTile = 2048;

__global__ void __launch_bounds__(256)
rank_count_kernel(const float *__restrict__ raw, int N, int j_per_slice, unsigned int *__restrict__ counts)
{
    __shared__ uint32_t sk[kRankTile];
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t ki = (i < N) ? order_key(raw[i]) : 0u;
    const unsigned long long ci = ((unsigned long long)ki << 32) | (unsigned int)i;
    const int j_lo = blockIdx.y * j_per_slice;
    const int j_hi = min(N, j_lo + j_per_slice);
    unsigned int cnt = 0;
    for (int j0 = j_lo; j0 < j_hi; j0 += kRankTile) {
        const int len = min(kRankTile, j_hi - j0);
        for (int t = threadIdx.x; t < len; t += blockDim.x) sk[t] = order_key(raw[j0 + t]);
        __syncthreads();
        if (i < N) {
#pragma unroll 8
            for (int t = 0; t < len; ++t) {
                const unsigned long long cj = ((unsigned long long)sk[t] << 32) | (unsigned int)(j0 + t);
                cnt += (cj < ci) ? 1u : 0u;
            }
        }
        __syncthreads();
    }
    if (i < N) {
        if (gridDim.y == 1) counts[i] = cnt;
        else atomicAdd(&counts[i], cnt);
    }
}

__global__ void rank_finish_kernel(const unsigned int *__restrict__ counts, int N, float *__restrict__ out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    if (N == 1) { out[i] = 0.f; return; }
    const float num = (float)(2 * (long long)counts[i] - (long long)(N - 1));
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
            // counts live in the output buffer itself (same size, overwritten by the finishing pass)
            unsigned int *counts = reinterpret_cast<unsigned int *>(out);
            const int bx = (N + 255) / 256;
            int slices = 1;
            while (bx * slices < 296 && (N / (slices * 2)) >= kRankTile) slices *= 2;
            const int j_per_slice = ((N + slices - 1) / slices + kRankTile - 1) / kRankTile * kRankTile;
            slices = (N + j_per_slice - 1) / j_per_slice;
            if (slices > 1) {
                cudaError_t e = cudaMemsetAsync(counts, 0, sizeof(unsigned int) * (size_t)N, st);
                if (e != cudaSuccess) return EGR_ERR_CUDA;
            }
            rank_count_kernel<<<dim3(bx, slices), 256, 0, st>>>(raw, N, j_per_slice, counts);
            rank_finish_kernel<<<bx, 256, 0, st>>>(counts, N, out);
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

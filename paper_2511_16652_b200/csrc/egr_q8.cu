// Per-channel-scaled int8 weights with a discretised Adam update (appendix "Fine-tuning of Integer Quantised
// Models").  Everything here is element-wise or a small reduction and therefore bound by HBM bandwidth: 128-bit
// accesses, one pass per tensor where the arithmetic allows it.  Whatever decides an integer (the quantised code,
// the unit step) is computed in fp32 with explicitly rounded operations (__fmul_rn and friends are never fused), so
// that the result is a pure function of the inputs.
#include <cuda_bf16.h>

#include "egr_device.cuh"
#include "egr_internal.h"

namespace egr {

namespace {

__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }
__device__ __forceinline__ uint32_t float_to_bf16_bits(float f)
{
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(f));
}

// ---------------------------------------------------------------- quantisation: one block per output channel
constexpr int QUANT_THREADS = 256;

__global__ void __launch_bounds__(QUANT_THREADS)
q8_quantize_kernel(const float *__restrict__ W, int n, int64_t ldw, float eps, int8_t *__restrict__ Q, int64_t ldq,
                   __nv_bfloat16 *__restrict__ scales)
{
    __shared__ float red[QUANT_THREADS / 32];
    __shared__ float s_shared;
    const float *w = W + (int64_t)blockIdx.x * ldw;
    // 128-bit accesses when the row allows them (enough bytes in flight to fill the memory pipeline)
    const bool vec = ((reinterpret_cast<uintptr_t>(w) & 15) == 0) && ((n & 3) == 0);
    float amax = 0.f;
    if (vec) {
        for (int j = threadIdx.x; j < n / 4; j += QUANT_THREADS) {
            const float4 v = reinterpret_cast<const float4 *>(w)[j];
            amax = fmaxf(fmaxf(amax, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
        }
    } else {
        for (int j = threadIdx.x; j < n; j += QUANT_THREADS) amax = fmaxf(amax, fabsf(w[j]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float a = red[0];
        for (int i = 1; i < QUANT_THREADS / 32; ++i) a = fmaxf(a, red[i]);
        const __nv_bfloat16 sb = __float2bfloat16_rn(fmaxf(__fdiv_rn(a, 127.0f), eps));
        scales[blockIdx.x] = sb;
        s_shared = __bfloat162float(sb);
    }
    __syncthreads();
    const float s = s_shared;
    int8_t *q = Q + (int64_t)blockIdx.x * ldq;
    // the second sweep over the row is served by L2
    auto code = [s](float x) { return (int)fminf(127.f, fmaxf(-127.f, rintf(__fdiv_rn(x, s)))); };
    if (vec && (reinterpret_cast<uintptr_t>(q) & 3) == 0) {
        for (int j = threadIdx.x; j < n / 4; j += QUANT_THREADS) {
            const float4 v = reinterpret_cast<const float4 *>(w)[j];
            const uint32_t packed = ((uint32_t)code(v.x) & 0xffu) | (((uint32_t)code(v.y) & 0xffu) << 8) |
                                    (((uint32_t)code(v.z) & 0xffu) << 16) | (((uint32_t)code(v.w) & 0xffu) << 24);
            reinterpret_cast<uint32_t *>(q)[j] = packed;
        }
    } else {
        for (int j = threadIdx.x; j < n; j += QUANT_THREADS) q[j] = (int8_t)code(w[j]);
    }
}

// ---------------------------------------------------------------- int8 codes -> bf16 (exact), 16 codes per thread
__global__ void __launch_bounds__(256)
q8_expand_kernel(const int8_t *__restrict__ Q, int m, int n16, int64_t ldq, __nv_bfloat16 *__restrict__ out, int64_t ldo)
{
    const int64_t total = (int64_t)m * n16;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / n16;
        const int c = (int)(i % n16) * 16;
        const int4 v = __ldg(reinterpret_cast<const int4 *>(Q + row * ldq + c));
        const int w[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int lo = (int)(int8_t)((w[k >> 1] >> (16 * (k & 1))) & 0xff);
            const int hi = (int)(int8_t)((w[k >> 1] >> (16 * (k & 1) + 8)) & 0xff);
            o[k] = float_to_bf16_bits((float)lo) | (float_to_bf16_bits((float)hi) << 16);
        }
        uint4 *dst = reinterpret_cast<uint4 *>(out + row * ldo + c);
        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

// ---------------------------------------------------------------- scale gradient g[j] = (1/N) sum_p g_p e_p[j]
constexpr int SG_THREADS = 128;
constexpr int SG_CHUNK = 64;        // noise indices per partial sum (small: enough blocks for small populations too)

__global__ void __launch_bounds__(SG_THREADS)
scale_gradient_partial_kernel(const float *__restrict__ fitness, int64_t P, uint32_t flags, NoiseKey key, int n_blocks,
                              int pitch, float *__restrict__ partial)
{
    const int q = blockIdx.x * SG_THREADS + threadIdx.x;
    if (q >= n_blocks) return;
    const int64_t p0 = (int64_t)blockIdx.y * SG_CHUNK;
    const int64_t p1 = (p0 + SG_CHUNK < P) ? p0 + SG_CHUNK : P;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t p = p0; p < p1; ++p) {
        const float gp = (flags & EGR_ANTITHETIC) ? __fsub_rn(__ldg(fitness + 2 * p), __ldg(fitness + 2 * p + 1)) : __ldg(fitness + p);
        const float4 z = noise_block<false>(key, (uint32_t)p, kTagScale, (uint32_t)q);
        acc.x = fmaf(gp, z.x, acc.x); acc.y = fmaf(gp, z.y, acc.y); acc.z = fmaf(gp, z.z, acc.z); acc.w = fmaf(gp, z.w, acc.w);
    }
    reinterpret_cast<float4 *>(partial + (int64_t)blockIdx.y * pitch)[q] = acc;
}

__global__ void __launch_bounds__(SG_THREADS)
scale_gradient_reduce_kernel(const float *__restrict__ partial, int chunks, int pitch, int len, float inv_n, float *__restrict__ g)
{
    const int j = blockIdx.x * SG_THREADS + threadIdx.x;
    if (j >= len) return;
    float acc = 0.f;
    for (int c = 0; c < chunks; ++c) acc += partial[(int64_t)c * pitch + j];
    g[j] = acc * inv_n;
}

// ---------------------------------------------------------------- Adam proposal (fp32, one rounding per operation)
// step = lr / (1 - b1^t) and rsb2 = 1 / sqrt(1 - b2^t) are rounded once to fp32 on the host
struct AdamConst { float b1, b2, c1, c2, eps, step, rsb2; };

__device__ __forceinline__ float adam_proposal(float g, float &m, float &v, const AdamConst &k)
{
    m = __fadd_rn(__fmul_rn(k.b1, m), __fmul_rn(k.c1, g));
    v = __fadd_rn(__fmul_rn(k.b2, v), __fmul_rn(k.c2, __fmul_rn(g, g)));
    const float den = __fadd_rn(__fmul_rn(__fsqrt_rn(v), k.rsb2), k.eps);
    return __fdiv_rn(__fmul_rn(k.step, m), den);
}

constexpr int ADAM_THREADS = 256;
constexpr int ADAM_MAX_BLOCKS = 148 * 8;

// Eight elements per thread and trip: g fp32 (2 x 128 bit), both moments and u bf16 (128 bit each).  Writes the
// rounded moments and u, and one (sum u, sum u^2) pair per block in fp64.
__global__ void __launch_bounds__(ADAM_THREADS)
adam_propose_kernel(const float *__restrict__ G, int64_t ldg, int n8, int64_t vecs, uint4 *__restrict__ mom1,
                    uint4 *__restrict__ mom2, uint4 *__restrict__ u_out, AdamConst k, double *__restrict__ partial)
{
    double s1 = 0.0, s2 = 0.0;
    for (int64_t i = (int64_t)blockIdx.x * ADAM_THREADS + threadIdx.x; i < vecs; i += (int64_t)gridDim.x * ADAM_THREADS) {
        const int64_t row = i / n8;
        const int c = (int)(i % n8) * 8;
        const float4 g0 = __ldg(reinterpret_cast<const float4 *>(G + row * ldg + c));
        const float4 g1 = __ldg(reinterpret_cast<const float4 *>(G + row * ldg + c) + 1);
        const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
        const uint4 mv = mom1[i], vv = mom2[i];
        const uint32_t mw[4] = {mv.x, mv.y, mv.z, mv.w}, vw[4] = {vv.x, vv.y, vv.z, vv.w};
        uint32_t mo[4], vo[4], uo[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            uint32_t mb[2], vb[2], ub[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float m = bf16_bits_to_float((mw[h] >> (16 * e)) & 0xffffu), v = bf16_bits_to_float((vw[h] >> (16 * e)) & 0xffffu);
                const float u = adam_proposal(g[2 * h + e], m, v, k);
                mb[e] = float_to_bf16_bits(m); vb[e] = float_to_bf16_bits(v); ub[e] = float_to_bf16_bits(u);
                const double ur = (double)bf16_bits_to_float(ub[e]);
                s1 += ur; s2 += ur * ur;
            }
            mo[h] = mb[0] | (mb[1] << 16); vo[h] = vb[0] | (vb[1] << 16); uo[h] = ub[0] | (ub[1] << 16);
        }
        mom1[i] = make_uint4(mo[0], mo[1], mo[2], mo[3]);
        mom2[i] = make_uint4(vo[0], vo[1], vo[2], vo[3]);
        u_out[i] = make_uint4(uo[0], uo[1], uo[2], uo[3]);
    }
    __shared__ double r1[ADAM_THREADS / 32], r2[ADAM_THREADS / 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { s1 += __shfl_xor_sync(0xffffffffu, s1, o); s2 += __shfl_xor_sync(0xffffffffu, s2, o); }
    if ((threadIdx.x & 31) == 0) { r1[threadIdx.x >> 5] = s1; r2[threadIdx.x >> 5] = s2; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0;
        for (int i = 0; i < ADAM_THREADS / 32; ++i) { a += r1[i]; b += r2[i]; }
        partial[2 * blockIdx.x] = a; partial[2 * blockIdx.x + 1] = b;
    }
}

// Every block first reduces the per-block sums of the proposal pass itself (same order everywhere, so every block
// arrives at the same bits): mean and population deviation of u in fp64 -> (mu, tau (sigma + 1e-8)) rounded once to
// fp32.  Then Delta = sign(u - mu) [|u - mu| >= threshold], Q <- clip(Q + Delta).
__global__ void __launch_bounds__(ADAM_THREADS)
adam_apply_q8_kernel(const uint4 *__restrict__ u_in, int n8, int64_t vecs, int8_t *__restrict__ Q, int64_t ldq,
                     const double *__restrict__ partial, int n_partial, double count, float tau,
                     unsigned long long *__restrict__ changed)
{
    __shared__ double r1[ADAM_THREADS / 32], r2[ADAM_THREADS / 32];
    __shared__ float stats[2];
    {
        double a = 0.0, b = 0.0;
        for (int i = threadIdx.x; i < n_partial; i += ADAM_THREADS) { a += partial[2 * i]; b += partial[2 * i + 1]; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { a += __shfl_xor_sync(0xffffffffu, a, o); b += __shfl_xor_sync(0xffffffffu, b, o); }
        if ((threadIdx.x & 31) == 0) { r1[threadIdx.x >> 5] = a; r2[threadIdx.x >> 5] = b; }
        __syncthreads();
        if (threadIdx.x == 0) {
            double s1 = 0.0, s2 = 0.0;
            for (int i = 0; i < ADAM_THREADS / 32; ++i) { s1 += r1[i]; s2 += r2[i]; }
            const double mu = s1 / count;
            double var = s2 / count - mu * mu;
            if (!(var > 0.0)) var = 0.0;
            stats[0] = (float)mu;
            stats[1] = (float)((double)tau * (sqrt(var) + 1e-8));
        }
        __syncthreads();
    }
    const float mu = stats[0], thr = stats[1];
    int moved = 0;
    // two vectors per trip, all four loads issued before the arithmetic (the kernel is latency-bound otherwise)
    const int64_t stride = (int64_t)gridDim.x * ADAM_THREADS;
    for (int64_t i0 = (int64_t)blockIdx.x * ADAM_THREADS + threadIdx.x; i0 < vecs; i0 += 2 * stride) {
        uint4 uv[2]; uint2 qv[2]; uint2 *qp[2]; bool live[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int64_t i = i0 + h * stride;
            live[h] = i < vecs;
            if (live[h]) {
                qp[h] = reinterpret_cast<uint2 *>(Q + (i / n8) * ldq + (int)(i % n8) * 8);
                uv[h] = __ldg(u_in + i);
                qv[h] = *qp[h];
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (!live[h]) continue;
            const uint32_t uw[4] = {uv[h].x, uv[h].y, uv[h].z, uv[h].w};
            const uint32_t qw[2] = {qv[h].x, qv[h].y};
            uint32_t qo[2] = {0u, 0u};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float u = bf16_bits_to_float((uw[e >> 1] >> (16 * (e & 1))) & 0xffffu);
                const float d = __fsub_rn(u, mu);
                const int step = (fabsf(d) >= thr) ? ((d > 0.f) - (d < 0.f)) : 0;
                const int q0 = (int)(int8_t)((qw[e >> 2] >> (8 * (e & 3))) & 0xffu);
                const int q1 = max(-127, min(127, q0 + step));
                moved += (q1 != q0);
                qo[e >> 2] |= ((uint32_t)q1 & 0xffu) << (8 * (e & 3));
            }
            if (qo[0] != qw[0] || qo[1] != qw[1]) *qp[h] = make_uint2(qo[0], qo[1]);      // the update is sparse
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) moved += __shfl_xor_sync(0xffffffffu, moved, o);
    if ((threadIdx.x & 31) == 0 && moved) atomicAdd(changed, (unsigned long long)moved);
}

__global__ void __launch_bounds__(ADAM_THREADS)
adam_step_bf16_kernel(__nv_bfloat16 *__restrict__ param, int64_t len, const float *__restrict__ g,
                      __nv_bfloat16 *__restrict__ mom1, __nv_bfloat16 *__restrict__ mom2, AdamConst k)
{
    const int64_t i = (int64_t)blockIdx.x * ADAM_THREADS + threadIdx.x;
    if (i >= len) return;
    float m = __bfloat162float(mom1[i]), v = __bfloat162float(mom2[i]);
    const float u = __bfloat162float(__float2bfloat16_rn(adam_proposal(g[i], m, v, k)));
    mom1[i] = __float2bfloat16_rn(m); mom2[i] = __float2bfloat16_rn(v);
    param[i] = __float2bfloat16_rn(__fadd_rn(__bfloat162float(param[i]), u));
}

AdamConst make_adam(float b1, float b2, float eps, float step, float rsb2)
{
    AdamConst k; k.b1 = b1; k.b2 = b2; k.c1 = 1.0f - b1; k.c2 = 1.0f - b2; k.eps = eps; k.step = step; k.rsb2 = rsb2;
    return k;
}

}  // namespace

// ---------------------------------------------------------------- launchers
int launch_q8_quantize(const float *W, int m, int n, int64_t ldw, float eps, int8_t *Q, int64_t ldq, void *scales, cudaStream_t st)
{
    q8_quantize_kernel<<<m, QUANT_THREADS, 0, st>>>(W, n, ldw, eps, Q, ldq, reinterpret_cast<__nv_bfloat16 *>(scales));
    return cuda_ok(cudaGetLastError());
}

// columns are expanded in groups of 16: the caller's output pitch covers n rounded up to 16 and Q's pitch does too
int launch_q8_expand(const int8_t *Q, int m, int n, int64_t ldq, void *out_bf16, int64_t ldo, cudaStream_t st)
{
    const int n16 = (n + 15) / 16;
    const int64_t total = (int64_t)m * n16;
    const int blocks = (int)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
    q8_expand_kernel<<<blocks, 256, 0, st>>>(Q, m, n16, ldq, reinterpret_cast<__nv_bfloat16 *>(out_bf16), ldo);
    return cuda_ok(cudaGetLastError());
}

static int sg_pitch(int d_out) { return ((d_out + 1 + 3) / 4) * 4; }

size_t scale_gradient_ws(int d_out, int64_t P)
{
    const int64_t chunks = (P + SG_CHUNK - 1) / SG_CHUNK;
    return kWsHeader + align_up((size_t)chunks * sg_pitch(d_out) * sizeof(float), 256);
}

int launch_scale_gradient(const egr_layer &L, const float *fitness, float *g, void *ws, cudaStream_t st)
{
    const int64_t P = (L.flags & EGR_ANTITHETIC) ? L.n_members / 2 : L.n_members;
    const int chunks = (int)((P + SG_CHUNK - 1) / SG_CHUNK);
    const int pitch = sg_pitch(L.d_out), n_blocks = pitch / 4;
    float *partial = reinterpret_cast<float *>((unsigned char *)ws + kWsHeader);
    if (cudaMemsetAsync(ws, 0, 8, st) != cudaSuccess) return EGR_ERR_CUDA;
    dim3 grid((n_blocks + SG_THREADS - 1) / SG_THREADS, chunks);
    scale_gradient_partial_kernel<<<grid, SG_THREADS, 0, st>>>(fitness, P, L.flags, make_noise_key(L.seed, L.layer_id), n_blocks,
                                                               pitch, partial);
    if (cudaGetLastError() != cudaSuccess) return EGR_ERR_CUDA;
    const int len = L.d_out + 1;
    scale_gradient_reduce_kernel<<<(len + SG_THREADS - 1) / SG_THREADS, SG_THREADS, 0, st>>>(partial, chunks, pitch, len,
                                                                                             1.0f / (float)L.n_members, g);
    return cuda_ok(cudaGetLastError());
}

// workspace: [header | changed counter | block partials | u]
size_t adam_q8_ws(int m, int n)
{
    return kWsHeader + 256 + align_up((size_t)ADAM_MAX_BLOCKS * 2 * sizeof(double), 256) + align_up((size_t)m * n * 2, 256);
}

int launch_adam_step_q8(int8_t *Q, int64_t ldq, int m, int n, const float *G, int64_t ldg, void *mom1, void *mom2,
                        float b1, float b2, float eps, float step, float rsb2, float tau, int64_t *n_changed,
                        void *ws, cudaStream_t st)
{
    unsigned char *base = reinterpret_cast<unsigned char *>(ws);
    unsigned long long *changed = reinterpret_cast<unsigned long long *>(base + kWsHeader);
    double *partial = reinterpret_cast<double *>(base + kWsHeader + 256);
    uint4 *u = reinterpret_cast<uint4 *>(base + kWsHeader + 256 + align_up((size_t)ADAM_MAX_BLOCKS * 2 * sizeof(double), 256));
    if (cudaMemsetAsync(ws, 0, kWsHeader + 256, st) != cudaSuccess) return EGR_ERR_CUDA;      // status and the counter
    const int n8 = n / 8;
    const int64_t vecs = (int64_t)m * n8;
    const int64_t want = (vecs + ADAM_THREADS - 1) / ADAM_THREADS;
    const int blocks = (int)(want < ADAM_MAX_BLOCKS ? (want > 0 ? want : 1) : ADAM_MAX_BLOCKS);
    const AdamConst k = make_adam(b1, b2, eps, step, rsb2);
    adam_propose_kernel<<<blocks, ADAM_THREADS, 0, st>>>(G, ldg, n8, vecs, reinterpret_cast<uint4 *>(mom1),
                                                         reinterpret_cast<uint4 *>(mom2), u, k, partial);
    if (cudaGetLastError() != cudaSuccess) return EGR_ERR_CUDA;
    adam_apply_q8_kernel<<<blocks, ADAM_THREADS, 0, st>>>(u, n8, vecs, Q, ldq, partial, blocks, (double)m * (double)n, tau, changed);
    if (cudaGetLastError() != cudaSuccess) return EGR_ERR_CUDA;
    if (n_changed &&
        cudaMemcpyAsync(n_changed, changed, sizeof(int64_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return EGR_ERR_CUDA;
    return EGR_OK;
}

int launch_adam_step_bf16(void *param, int64_t len, const float *g, void *mom1, void *mom2, float b1, float b2,
                          float eps, float step, float rsb2, cudaStream_t st)
{
    const AdamConst k = make_adam(b1, b2, eps, step, rsb2);
    const int blocks = (int)((len + ADAM_THREADS - 1) / ADAM_THREADS);
    adam_step_bf16_kernel<<<blocks, ADAM_THREADS, 0, st>>>(reinterpret_cast<__nv_bfloat16 *>(param), len, g,
                                                           reinterpret_cast<__nv_bfloat16 *>(mom1),
                                                           reinterpret_cast<__nv_bfloat16 *>(mom2), k);
    return cuda_ok(cudaGetLastError());
}

}  // namespace egr

// Device-side building blocks shared by the kernels: the counter-based noise generator
// (Philox4x32-10 + Box-Muller, the definition stated at the top of egr.h) and small helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/egr.h"

namespace egr {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

constexpr uint32_t kTagA = 0u, kTagB = 1u, kTagI8 = 2u, kTagScale = 3u;

__host__ __device__ __forceinline__ void philox_round(uint32_t &c0, uint32_t &c1, uint32_t &c2, uint32_t &c3,
                                                      uint32_t k0, uint32_t k1)
{
    // one 32x32->64 multiply per half (a single wide multiply-add on the device)
    const uint64_t p0 = (uint64_t)kPhiloxM0 * c0, p1 = (uint64_t)kPhiloxM1 * c2;
    const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
}

// Ten rounds; the key advances by the Weyl constants between rounds.
__host__ __device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                        uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int i = 0; i < 10; ++i) {
        philox_round(c0, c1, c2, c3, k0, k1);
        k0 += kPhiloxW0; k1 += kPhiloxW1;
    }
    return make_uint4(c0, c1, c2, c3);
}

struct NoiseKey {
    uint32_t k0, k1;      // seed words
    uint32_t layer_id;
};

__host__ __device__ __forceinline__ NoiseKey make_noise_key(uint64_t seed, uint32_t layer_id)
{
    NoiseKey k; k.k0 = (uint32_t)(seed & 0xffffffffu); k.k1 = (uint32_t)(seed >> 32); k.layer_id = layer_id;
    return k;
}

// Two uniforms -> two normals.  PRECISE: fp32 library functions (a few ulp); else hardware approximations
// (absolute error ~4e-7 on the trigonometric part, the argument is kept inside [-pi, pi)).
template <bool PRECISE>
__device__ __forceinline__ void box_muller(uint32_t xa, uint32_t xb, float &z_cos, float &z_sin)
{
    if (PRECISE) {
        const float u1 = (float)((xa >> 9) + 1u) * 0x1p-23f;      // (0, 1], exact
        const float u2x2 = (float)(xb >> 9) * 0x1p-22f;           // 2*u2 in [0, 2), exact
        const float rho = sqrtf(-2.0f * logf(u1));
        float s, c;
        sincospif(u2x2, &s, &c);
        z_cos = rho * c; z_sin = rho * s;
    } else {
        // mantissa trick instead of integer->float conversions: 1.m in [1,2) with m = x >> 9
        // x >> 9 as the high word of x * 2^23, plus the exponent bits: one multiply-add on the FMA pipe instead of a
        // shift and an OR on the (busier) integer ALU pipe
        const float f1 = __uint_as_float(__umulhi(xa, 0x00800000u) + 0x3f800000u);
        const float f2 = __uint_as_float(__umulhi(xb, 0x00800000u) + 0x3f800000u);
        const float u1f = f1 - 0.99999988079071044921875f;        // (m+1) 2^-23 in (0,1], exact
        const float v = f2 - 1.5f;                                // u2 - 1/2 in [-1/2, 1/2), exact
        // hardware approximations in their flush-to-zero forms (no denormal fix-up code): the inputs are normal floats
        float lg, rho, s, c;
        asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lg) : "f"(u1f));
        asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(rho) : "f"(-1.3862943611198906f * lg));        // sqrt(-2 ln u1)
        const float ang = 6.283185307179586f * v;
        asm("sin.approx.ftz.f32 %0, %1;" : "=f"(s) : "f"(ang));
        asm("cos.approx.ftz.f32 %0, %1;" : "=f"(c) : "f"(ang));
        z_cos = -rho * c; z_sin = -rho * s;                       // cos(2 pi u2) = -cos(2 pi v)
    }
}

// The four normals of block q of factor `tag` for noise index p: flat elements 4q .. 4q+3.
template <bool PRECISE>
__device__ __forceinline__ float4 noise_block(const NoiseKey &key, uint32_t p, uint32_t tag, uint32_t q)
{
    const uint4 x = philox4x32_10(q, p, key.layer_id, tag, key.k0, key.k1);
    float4 z;
    box_muller<PRECISE>(x.x, x.y, z.x, z.y);
    box_muller<PRECISE>(x.z, x.w, z.z, z.w);
    return z;
}

// Out-of-line copy for call sites that would otherwise unroll hundreds of generator bodies (instruction-cache
// pressure outweighs the call overhead there).
template <bool PRECISE>
__device__ __noinline__ float4 noise_block_call(NoiseKey key, uint32_t p, uint32_t tag, uint32_t q)
{
    return noise_block<PRECISE>(key, p, tag, q);
}

// sum_k w[k] * z[k] over the NB consecutive blocks q0 .. q0+NB-1 (4 NB normals), out of line.  The ten rounds of a
// Philox block are one dependent chain; walking NB chains in lock step gives the scheduler independent instructions,
// which a sequence of single-block calls does not.  `w` lives in local memory at the call site (a pointer argument),
// a handful of cached loads against several hundred generator instructions.
template <int NB>
__device__ __noinline__ float noise_dot_call(NoiseKey key, uint32_t p, uint32_t tag, uint32_t q0, const float *__restrict__ w)
{
    uint32_t c0[NB], c1[NB], c2[NB], c3[NB];
#pragma unroll
    for (int j = 0; j < NB; ++j) { c0[j] = q0 + (uint32_t)j; c1[j] = p; c2[j] = key.layer_id; c3[j] = tag; }
    uint32_t k0 = key.k0, k1 = key.k1;
#pragma unroll
    for (int i = 0; i < 10; ++i) {
#pragma unroll
        for (int j = 0; j < NB; ++j) philox_round(c0[j], c1[j], c2[j], c3[j], k0, k1);
        k0 += kPhiloxW0; k1 += kPhiloxW1;
    }
    float acc = 0.f;
#pragma unroll
    for (int j = 0; j < NB; ++j) {
        float z0, z1, z2, z3;
        box_muller<false>(c0[j], c1[j], z0, z1);
        box_muller<false>(c2[j], c3[j], z2, z3);
        acc = fmaf(w[4 * j], z0, acc); acc = fmaf(w[4 * j + 1], z1, acc);
        acc = fmaf(w[4 * j + 2], z2, acc); acc = fmaf(w[4 * j + 3], z3, acc);
    }
    return acc;
}

// NB blocks q0, q0 + stride, ... of one factor, their ten rounds walked in lock step (independent chains for the
// scheduler instead of NB dependent ones back to back)
template <int NB>
__device__ __forceinline__ void noise_blocks_lockstep(const NoiseKey &key, uint32_t p, uint32_t tag, uint32_t q0, uint32_t stride,
                                                      float4 (&z)[NB])
{
    uint32_t c0[NB], c1[NB], c2[NB], c3[NB];
#pragma unroll
    for (int j = 0; j < NB; ++j) { c0[j] = q0 + (uint32_t)j * stride; c1[j] = p; c2[j] = key.layer_id; c3[j] = tag; }
    uint32_t k0 = key.k0, k1 = key.k1;
#pragma unroll
    for (int i = 0; i < 10; ++i) {
#pragma unroll
        for (int j = 0; j < NB; ++j) philox_round(c0[j], c1[j], c2[j], c3[j], k0, k1);
        k0 += kPhiloxW0; k1 += kPhiloxW1;
    }
#pragma unroll
    for (int j = 0; j < NB; ++j) {
        box_muller<false>(c0[j], c1[j], z[j].x, z[j].y);
        box_muller<false>(c2[j], c3[j], z[j].z, z[j].w);
    }
}

// Out of line, results written to dst[0], dst[dst_stride], ... (shared memory at the call sites)
template <int NB>
__device__ __noinline__ void noise_blocks_store(NoiseKey key, uint32_t p, uint32_t tag, uint32_t q0, uint32_t stride,
                                                float4 *dst, int dst_stride)
{
    float4 z[NB];
    noise_blocks_lockstep<NB>(key, p, tag, q0, stride, z);
#pragma unroll
    for (int j = 0; j < NB; ++j) dst[j * dst_stride] = z[j];
}

// Element-wise function after the layer (flag bits EGR_ACT_*).  PRECISE: fp32 library functions, for fp32 outputs;
// otherwise tanh is the hardware approximation (relative error 2^-11, below the bf16 rounding that follows).
// GELU is x Phi(x) with Phi through erff in both forms.
template <bool PRECISE>
__device__ __forceinline__ float apply_act(float v, uint32_t act)
{
    if (act == EGR_ACT_RELU) return fmaxf(v, 0.f);
    if (act == EGR_ACT_TANH) {
        if (PRECISE) return tanhf(v);
        float t;
        asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(v));
        return t;
    }
    if (act == EGR_ACT_GELU) return 0.5f * v * (1.0f + erff(v * 0.70710678118654752f));
    return v;
}

// Four values at once, out of line: one copy of the function bodies per kernel instead of one per unrolled column
template <bool PRECISE>
__device__ __noinline__ float4 apply_act4(float4 v, uint32_t act)
{
    return make_float4(apply_act<PRECISE>(v.x, act), apply_act<PRECISE>(v.y, act), apply_act<PRECISE>(v.z, act),
                       apply_act<PRECISE>(v.w, act));
}

// member i -> noise index p and sign (+1 / -1)
__device__ __forceinline__ void member_noise(int member, uint32_t flags, uint32_t &p, float &sign)
{
    if (flags & EGR_ANTITHETIC) { p = (uint32_t)(member >> 1); sign = (member & 1) ? -1.0f : 1.0f; }
    else                        { p = (uint32_t)member;        sign = 1.0f; }
}

// population index of a row: explicit map if given, else member_base + row / rows_per_member
__device__ __forceinline__ int member_of(const int32_t *__restrict__ rowmap, int mbase, int64_t row, int T)
{
    if (rowmap) return __ldg(rowmap + row);
    // a 64-bit division is a subroutine of a few hundred cycles; rows fit in 32 bits almost always
    return mbase + (((uint64_t)row >> 32) == 0 ? (int)((uint32_t)row / (uint32_t)T) : (int)(row / T));
}

__device__ __forceinline__ int ilog2_pow2(int v) { return 31 - __clz(v); }

// Integer LM at width 256, one warp per member (8 values per lane): embedding row of the member's token with its
// rank-1 perturbation, y = sat127(emb[t][j] + ((sign B_p[t] A_p[j]) >> sigma_shift)), then the layer norm
// x = sat127(trunc(y w / max(sat127(sum|y| >> ln_shift), 1))).  emb_rows is the transposed embedding [256 tokens][256].
__device__ __forceinline__ void lm_embed_ln256_row(const int8_t *__restrict__ emb_rows, const uint8_t *__restrict__ tokens,
                                                   int seq_len, int pos, const int32_t *__restrict__ member_seq, int64_t member,
                                                   uint32_t flags, const NoiseKey &key, int sigma_shift,
                                                   const int8_t *__restrict__ table, uint32_t mask,
                                                   const int8_t *__restrict__ ln_w, int ln_shift, int8_t *y, int8_t *x, int lane)
{
    auto sat = [](int v) { return max(-127, min(127, v)); };
    uint32_t p; float sign;
    member_noise((int)member, flags, p, sign);
    const uint4 xw = philox4x32_10(0u, p, key.layer_id, kTagI8, key.k0, key.k1);
    const uint32_t off_a = xw.x & mask, off_b = xw.y & mask;
    const int t = tokens[(int64_t)member_seq[member] * seq_len + pos];
    const int bt = (sign < 0.f ? -1 : 1) * (int)table[(off_b + (uint32_t)t) & mask];
    // this lane's eight consecutive slice bytes (three words when the table is word-addressable) and embedding values
    int av[8];
    const uint32_t o = off_a + (uint32_t)lane * 8u;
    if (mask >= 3u && (reinterpret_cast<uintptr_t>(table) & 3) == 0) {
        const uint32_t *t32 = reinterpret_cast<const uint32_t *>(table);
        const uint32_t wm = mask >> 2, b = o >> 2, sh = (o & 3u) * 8u;
        const uint32_t w0 = __ldg(t32 + (b & wm)), w1 = __ldg(t32 + ((b + 1u) & wm)), w2 = __ldg(t32 + ((b + 2u) & wm));
        const uint32_t lo = __funnelshift_r(w0, w1, sh), hi = __funnelshift_r(w1, w2, sh);
#pragma unroll
        for (int i = 0; i < 4; ++i) { av[i] = (int)(int8_t)((lo >> (8 * i)) & 0xffu); av[4 + i] = (int)(int8_t)((hi >> (8 * i)) & 0xffu); }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) av[i] = (int)table[(o + (uint32_t)i) & mask];
    }
    const int2 e8 = __ldg(reinterpret_cast<const int2 *>(emb_rows + t * 256 + lane * 8));
    const int8_t *eb = reinterpret_cast<const int8_t *>(&e8);
    int yv[8], sum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        yv[i] = sat((int)eb[i] + ((bt * av[i]) >> sigma_shift));
        sum += abs(yv[i]);
    }
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    const int mav = max(1, sat(sum >> ln_shift));
    const int2 w8 = *reinterpret_cast<const int2 *>(ln_w + lane * 8);
    const int8_t *wb = reinterpret_cast<const int8_t *>(&w8);
    int2 oy, ox;
    int8_t *py = reinterpret_cast<int8_t *>(&oy), *px = reinterpret_cast<int8_t *>(&ox);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        py[i] = (int8_t)yv[i];
        px[i] = (int8_t)sat((yv[i] * (int)wb[i]) / mav);
    }
    *reinterpret_cast<int2 *>(y + member * 256 + lane * 8) = oy;
    *reinterpret_cast<int2 *>(x + member * 256 + lane * 8) = ox;
}

__device__ __forceinline__ float load_as_float(const float *p) { return *p; }
__device__ __forceinline__ float load_as_float(const __nv_bfloat16 *p) { return __bfloat162float(*p); }

}  // namespace egr

// Integer-only path ("EGG Pretraining with Integer EGGROLL"): int8 operands, int32 accumulation, exact.
// Perturbation vectors are slices of a caller-supplied table of round(16 z) values; the slice offsets come
// from one Philox block per (matrix, noise index).
#include "egr_device.cuh"
#include "egr_internal.h"

namespace egr {

__device__ __forceinline__ int sat127(int v) { return max(-127, min(127, v)); }

__device__ __forceinline__ void i8_offsets(const NoiseKey &key, uint32_t p, uint32_t mask, uint32_t &off_a, uint32_t &off_b)
{
    const uint4 x = philox4x32_10(0u, p, key.layer_id, kTagI8, key.k0, key.k1);
    off_a = x.x & mask; off_b = x.y & mask;
}

// ------------------------------------------------------------------------------------------------
// prepass: per row rho, t = sign_i * sum_l X[rho][l] B_p[l] and the A-slice offset.  One warp per row.
// aux[rho] = (t, off_A)
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
skinny_xb_i8_kernel(const int8_t *__restrict__ X, int64_t ldx, int n, int64_t R, int T, int mbase, uint32_t flags, NoiseKey key,
                    const int8_t *__restrict__ table, uint32_t mask, int2 *__restrict__ aux)
{
    const int lane = threadIdx.x & 31;
    const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= R) return;
    uint32_t p; float sign;
    member_noise(member_of(nullptr, mbase, row, T), flags, p, sign);
    uint32_t off_a, off_b;
    i8_offsets(key, p, mask, off_a, off_b);
    int acc = 0;
    const int words = n >> 2;
    for (int w = lane; w < words; w += 32) {
        const int xw = *reinterpret_cast<const int *>(X + row * ldx + 4 * w);
        const uint32_t o = off_b + 4u * (uint32_t)w;
        const uint32_t b0 = (uint8_t)table[o & mask], b1 = (uint8_t)table[(o + 1) & mask];
        const uint32_t b2 = (uint8_t)table[(o + 2) & mask], b3 = (uint8_t)table[(o + 3) & mask];
        acc = __dp4a(xw, (int)(b0 | (b1 << 8) | (b2 << 16) | (b3 << 24)), acc);
    }
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) aux[row] = make_int2(sign < 0.f ? -acc : acc, (int)off_a);
}

// ------------------------------------------------------------------------------------------------
// forward: 64x64 tile per CTA, 4x4 outputs per thread, dp4a over 64-byte K slices; epilogue applies the
// rank-1 term and the two floor shifts.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
forward_i8_kernel(const int8_t *__restrict__ X, int64_t ldx, const int8_t *__restrict__ W, int64_t ldw,
                  int8_t *__restrict__ Y, int64_t ldy, int64_t R, int m, int n, uint32_t flags,
                  int sigma_shift, int out_shift, const int8_t *__restrict__ table, uint32_t mask,
                  const int2 *__restrict__ aux)
{
    __shared__ int sX[64][17];
    __shared__ int sW[64][17];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int64_t row_base = (int64_t)blockIdx.y * 64;
    const int col_base = blockIdx.x * 64;
    int acc[4][4] = {};
    const int words = n >> 2;
    for (int w0 = 0; w0 < words; w0 += 16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int idx = tid + i * 256;
            const int rr = idx >> 4, ww = idx & 15;
            const int64_t row = row_base + rr;
            const int col = col_base + rr;
            const int w = w0 + ww;
            sX[rr][ww] = (row < R && w < words) ? *reinterpret_cast<const int *>(X + row * ldx + 4 * w) : 0;
            sW[rr][ww] = (col < m && w < words) ? *reinterpret_cast<const int *>(W + (int64_t)col * ldw + 4 * w) : 0;
        }
        __syncthreads();
#pragma unroll
        for (int ww = 0; ww < 16; ++ww) {
            int a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = sX[ty * 4 + i][ww]; b[i] = sW[tx * 4 + i][ww]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = __dp4a(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
    const int col0 = col_base + tx * 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t row = row_base + ty * 4 + i;
        if (row >= R) continue;
        int t = 0; uint32_t off_a = 0;
        if (!(flags & EGR_NO_PERTURB)) { const int2 a = aux[row]; t = a.x; off_a = (uint32_t)a.y; }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int col = col0 + j;
            if (col >= m) continue;
            int pert = 0;
            if (!(flags & EGR_NO_PERTURB)) pert = (t * (int)table[(off_a + (uint32_t)col) & mask]) >> sigma_shift;
            Y[row * ldy + col] = (int8_t)sat127((acc[i][j] + pert) >> out_shift);
        }
    }
}

int launch_forward_i8(const egr_layer &L, const int8_t *X, const int8_t *W, int sigma_shift, int out_shift,
                      const int8_t *table, uint32_t table_log2, int8_t *Y, void *ws, cudaStream_t st)
{
    const int64_t R = (int64_t)L.n_members * L.rows_per_member;
    const uint32_t mask = (table_log2 >= 32) ? 0xffffffffu : ((1u << table_log2) - 1u);
    int2 *aux = reinterpret_cast<int2 *>((unsigned char *)ws + kWsHeader);
    const NoiseKey key = make_noise_key(L.seed, L.layer_id);
    const bool tc = i8_tc_eligible(X, L.ldx, W, L.ldw);
    // Layers that are one tile wide and shallow let the tensor-core kernel's epilogue warps compute the skinny dot
    // products themselves; anything larger runs them once per row in a prepass (one warp per row).
    const bool inline_skinny = tc && L.d_out <= 256 && L.d_in <= 1024;
    if (!(L.flags & EGR_NO_PERTURB) && !inline_skinny) {
        const unsigned grid = (unsigned)((R * 32 + 255) / 256);
        skinny_xb_i8_kernel<<<grid, 256, 0, st>>>(X, L.ldx, L.d_in, R, L.rows_per_member, L.member_base, L.flags, key, table, mask, aux);
    }
    if (tc) {
        // tensor-core path: operands can be fed by TMA
        if (cudaMemsetAsync(ws, 0, 8, st) != cudaSuccess) return EGR_ERR_CUDA;
        return launch_forward_i8_tc(L, X, W, sigma_shift, out_shift, table, table_log2, Y, inline_skinny ? nullptr : aux,
                                    reinterpret_cast<int *>(ws), st);
    }
    dim3 grid((unsigned)((L.d_out + 63) / 64), (unsigned)((R + 63) / 64));
    if (grid.y > 65535u) return EGR_ERR_UNSUPPORTED;
    forward_i8_kernel<<<grid, 256, 0, st>>>(X, L.ldx, W, L.ldw, Y, L.ldy, R, L.d_out, L.d_in, L.flags, sigma_shift,
                                            out_shift, table, mask, aux);
    return cuda_ok(cudaGetLastError());
}

// ------------------------------------------------------------------------------------------------
// update: E[j][l] = sum_p F_p A_p[j] B_p[l] (int32) is one int8 contraction over the noise indices.  The stacked
// factors are gathered from the table into K-major int8 matrices (row = matrix row or column, contiguous in p,
// padded with zeros to a multiple of 128 noise indices), then contracted on the tensor cores; the epilogue of that
// kernel compares with the threshold and moves W by one bin.
//   out[r][p] = (F ? F[p] : 1) * table[(off(p) + r) & mask],  off = A offset (which == 0) or B offset (which == 1)
// One block gathers a 64 x 64 tile through shared memory so that both the table reads (contiguous in r) and the
// stores (contiguous in p) are coalesced.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
stage_factors_i8_kernel(int8_t *__restrict__ out, int rows, int64_t p_pad, int P, const int8_t *__restrict__ F, NoiseKey key,
                        int which, const int8_t *__restrict__ table, uint32_t mask)
{
    __shared__ __align__(16) int8_t tile[64][80];     // [r][p], rows 16-byte aligned
    const int tid = threadIdx.x;
    const int r0 = blockIdx.y * 64;
    const int64_t p0 = (int64_t)blockIdx.x * 64;
    {
        const int pl = tid >> 2, seg = tid & 3;      // this thread gathers 16 rows of noise index p0 + pl
        const int64_t p = p0 + pl;
        int f = 0; uint32_t off = 0;
        if (p < P) {
            uint32_t off_a, off_b;
            i8_offsets(key, (uint32_t)p, mask, off_a, off_b);
            off = which ? off_b : off_a;
            f = F ? (int)F[p] : 1;
        }
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {
            const int rr = seg * 16 + i;
            int v = 0;
            if (p < P && r0 + rr < rows) v = f * (int)table[(off + (uint32_t)(r0 + rr)) & mask];
            tile[rr][pl] = (int8_t)v;
        }
    }
    __syncthreads();
    {
        const int rr = tid >> 2, seg = tid & 3;      // 16 consecutive noise indices of row r0 + rr
        if (r0 + rr < rows)
            *reinterpret_cast<int4 *>(out + (int64_t)(r0 + rr) * p_pad + p0 + seg * 16) =
                *reinterpret_cast<const int4 *>(&tile[rr][seg * 16]);
    }
}

static int64_t update_i8_p_pad(const egr_layer &L)
{
    const int64_t P = (L.flags & EGR_ANTITHETIC) ? L.n_members / 2 : L.n_members;
    return (P + 127) / 128 * 128;
}

size_t update_i8_workspace(const egr_layer &L)
{
    const int64_t pp = update_i8_p_pad(L);
    return kWsHeader + align_up((size_t)L.d_out * pp, 1024) + align_up((size_t)L.d_in * pp, 1024);
}

int launch_update_i8(const egr_layer &L, int8_t *W, const int8_t *F, int32_t threshold, const int8_t *table,
                     uint32_t table_log2, int32_t *E_out, void *ws, cudaStream_t st)
{
    const int P = (L.flags & EGR_ANTITHETIC) ? L.n_members / 2 : L.n_members;
    const int64_t pp = update_i8_p_pad(L);
    const uint32_t mask = (table_log2 >= 32) ? 0xffffffffu : ((1u << table_log2) - 1u);
    int8_t *At = reinterpret_cast<int8_t *>((unsigned char *)ws + kWsHeader);
    int8_t *Bt = At + align_up((size_t)L.d_out * pp, 1024);
    if (cudaMemsetAsync(ws, 0, 8, st) != cudaSuccess) return EGR_ERR_CUDA;
    const NoiseKey key = make_noise_key(L.seed, L.layer_id);
    const unsigned gp = (unsigned)(pp / 64);
    if ((L.d_out + 63) / 64 > 65535 || (L.d_in + 63) / 64 > 65535) return EGR_ERR_UNSUPPORTED;
    stage_factors_i8_kernel<<<dim3(gp, (unsigned)((L.d_out + 63) / 64)), 256, 0, st>>>(At, L.d_out, pp, P, F, key, 0, table, mask);
    if (cudaGetLastError() != cudaSuccess) return EGR_ERR_CUDA;
    stage_factors_i8_kernel<<<dim3(gp, (unsigned)((L.d_in + 63) / 64)), 256, 0, st>>>(Bt, L.d_in, pp, P, nullptr, key, 1, table, mask);
    if (cudaGetLastError() != cudaSuccess) return EGR_ERR_CUDA;
    return launch_update_i8_tc(L, At, Bt, pp, W, threshold, E_out, reinterpret_cast<int *>(ws), st);
}

}  // namespace egr

// Building blocks of the sm_100a tensor-core kernels: mbarrier / TMA / tcgen05 wrappers (inline PTX), shared-memory
// and instruction descriptors, and the host helpers that encode tensor maps.  CTA pairs (cta_group::2) throughout;
// no cluster-multicast loads.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/egr.h"

namespace egr {

constexpr uint32_t WAIT_LIMIT = 1u << 22;        // try_wait attempts before giving up ...
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;  // ... or two seconds, whichever comes first
constexpr uint32_t WAIT_SUSPEND_NS = 20000;        // a failed attempt may park the warp for this long (it wakes on completion)

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// same with a suspend-time hint: the waiting warp is parked instead of re-issuing the instruction
__device__ __forceinline__ bool mbar_try_wait_parked(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(WAIT_SUSPEND_NS) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one ran out).  Waiting warps burn
// issue slots and power that the tensor cores could use, so after one plain attempt the warp parks itself and
// looks at the abort flag and the clock only now and then.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int where,
                                          uint64_t limit_ns = WAIT_LIMIT_NS)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        if (mbar_try_wait_parked(bar, parity)) return true;
        if ((it & 7u) == 7u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) break;
        }
    }
    if (*abort_flag) return false;
    *abort_flag = 1;
    if (status) { atomicExch(status, EGR_ERR_TIMEOUT); atomicExch(status + 1, where); }
    return false;
}

// The same for waits that are expected to last tens of microseconds (a whole phase of other warps' work): the
// waiting thread sleeps between polls instead of occupying its scheduler.
__device__ __forceinline__ bool mbar_wait_long(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int where,
                                               uint64_t limit_ns = WAIT_LIMIT_NS)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        __nanosleep(200);
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) break;
        }
    }
    if (*abort_flag) return false;
    *abort_flag = 1;
    if (status) { atomicExch(status, EGR_ERR_TIMEOUT); atomicExch(status + 1, where); }
    return false;
}

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on a barrier that may live in the peer CTA (cluster address)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}

// TMA tile load into this CTA's shared memory; completion bytes are signalled on `cluster_bar`, which may be the
// leader CTA's barrier (.cta_group::2 permits signalling the peer).  No multicast.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t cluster_bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(cluster_bar) : "memory");
}

// TMA tile stores read this CTA's shared memory and belong to the bulk async group of the issuing thread;
// out-of-range parts of the box are clipped by the tensor map
// TMA tile reduction: global[tile] += shared[tile] (element-wise add performed at L2; fp32 here)
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap *map, uint32_t src, int c0, int c1)
{
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all but the newest N groups of this thread have finished READING shared memory / have completed
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
// generic-proxy writes to shared memory become visible to the async proxy (TMA)
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// L2 eviction policy for data that is written once and not read again by this kernel
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tma_store_2d_hint(const CUtensorMap *map, uint32_t src, int c0, int c1, uint64_t policy)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%1, %2}], [%3], %4;"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(src), "l"(policy) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// completion of all MMAs issued so far arrives on the barrier at this offset in BOTH CTAs of the pair (a barrier
// arrival fanned out to the two CTAs, not a load; two separate commits measured 5 - 10 % slower on the bench shapes)
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}

__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// The four K = 16 steps of one 64-element stage in one sequence.  The operand descriptors of step k are those of the
// stage advanced by 32 k bytes inside the 128-byte swizzle span, i.e. low word + 2 k; the high word is constant.
// accumulate = 0 makes the first step overwrite the accumulator.
__device__ __forceinline__ void tc_mma_bf16_pair_x4(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                                    uint32_t accumulate)
{
    asm volatile(
        "{\n.reg .pred p, q;\n.reg .b64 da, db;\n.reg .b32 ta, tb;\n"
        "setp.ne.b32 p, %5, 0;\n"
        "setp.eq.b32 q, 0, 0;\n"
        "mov.b64 da, {%1, %3};\n mov.b64 db, {%2, %3};\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n"
        "add.u32 ta, %1, 2;\n add.u32 tb, %2, 2;\n mov.b64 da, {ta, %3};\n mov.b64 db, {tb, %3};\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, q;\n"
        "add.u32 ta, %1, 4;\n add.u32 tb, %2, 4;\n mov.b64 da, {ta, %3};\n mov.b64 db, {tb, %3};\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, q;\n"
        "add.u32 ta, %1, 6;\n add.u32 tb, %2, 6;\n mov.b64 da, {ta, %3};\n mov.b64 db, {tb, %3};\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, q;\n}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread t of the warp receives lane (base_lane + t)
__device__ __forceinline__ void tc_ld_32x32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major operand tile, 128-byte swizzle: rows are 128 bytes apart, 8-row groups 1024 bytes apart.
__host__ __device__ constexpr uint64_t make_kmajor_sw128_desc(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);          // start address
    d |= (uint64_t)0 << 16;                                // leading byte offset: unused for swizzled K-major
    d |= (uint64_t)(1024u >> 4) << 32;                     // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                                // descriptor version (Blackwell)
    d |= (uint64_t)2 << 61;                                // layout: 128-byte swizzle
    return d;
}

// kind::f16 instruction descriptor: D fp32, A/B bf16, both K-major, M x N
__host__ __device__ constexpr uint32_t make_idesc_bf16(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}


// kind::i8 instruction descriptor: D int32, A/B signed int8, both K-major, M x N
__host__ __device__ constexpr uint32_t make_idesc_i8(int M, int N)
{
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void tc_mma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// 2-D row-major matrix [rows][K] of `elem_bytes`-byte elements with pitch ld (elements); box = box_k x box_rows
// (box_k * elem_bytes = the swizzle span: 128 bytes by default), out-of-range elements read as zero / are not written.
inline int make_tmap_2d(CUtensorMap *map, CUtensorMapDataType dt, int elem_bytes, const void *base, int64_t rows,
                        int64_t K, int64_t ld, int box_k, int box_rows, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return EGR_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * (cuuint64_t)elem_bytes};
    cuuint32_t box[2] = {(cuuint32_t)box_k, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, dt, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? EGR_OK : EGR_ERR_CUDA;
}

// Tensor maps are pure functions of their arguments; callers that launch the same few shapes again and again (a
// training loop; the recurrent LM: 18 launches per position) look them up here instead of asking the driver to encode
// them every time.
inline int cached_tmap_2d(CUtensorMap *map, CUtensorMapDataType dt, int elem_bytes, const void *base, int64_t rows,
                          int64_t K, int64_t ld, int box_k, int box_rows, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B)
{
    struct Entry { const void *base; int64_t rows, K, ld; int dt, eb, bk, br, sw; CUtensorMap map; };
    constexpr int kSlots = 64;
    static Entry table[kSlots];
    static int used = 0, next = 0;
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < used; ++i) {
        const Entry &e = table[i];
        if (e.base == base && e.rows == rows && e.K == K && e.ld == ld && e.dt == (int)dt && e.eb == elem_bytes && e.bk == box_k &&
            e.br == box_rows && e.sw == (int)swizzle) { *map = e.map; return EGR_OK; }
    }
    const int rc = make_tmap_2d(map, dt, elem_bytes, base, rows, K, ld, box_k, box_rows, swizzle);
    if (rc != EGR_OK) return rc;
    Entry &e = table[next];
    e.base = base; e.rows = rows; e.K = K; e.ld = ld; e.dt = (int)dt; e.eb = elem_bytes; e.bk = box_k; e.br = box_rows;
    e.sw = (int)swizzle; e.map = *map;
    next = (next + 1) % kSlots;
    if (used < kSlots) ++used;
    return EGR_OK;
}

// One lock for the library's small per-device host state (kernel attributes set, SM count, side stream): host threads
// may make their first calls at the same time.
inline std::mutex &config_mutex()
{
    static std::mutex mu;
    return mu;
}

inline int sm_count()
{
    static int n[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    std::lock_guard<std::mutex> lock(config_mutex());
    if (n[dev] == 0 && cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n[dev] = 0;
    return n[dev];
}


}  // namespace egr

// Building blocks shared by the tcgen05 (5th-generation tensor core) kernels of libkvq: PTX wrappers for
// tensor memory, the MMA, TMA tensor copies, the shared-memory matrix descriptor, and the bounded
// mbarrier wait that lets a role give up without hanging its CTA.
#pragma once

#include <cuda.h>

#include "kvq_device.cuh"

namespace kvq {

// K-major operand with the 128-byte swizzle: start address >> 4 | LBO 0 | SBO 1024 B (8 rows x 128 B) | version 1 | swizzle
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// instruction descriptor of kind::f16: D = f32, A and B both f16 (bf16 = false) or both bf16, both K-major, M = 128
__host__ __device__ constexpr uint32_t umma_idesc_m128(int n, bool bf16)
{
    return (1u << 4) | ((bf16 ? 1u : 0u) << 7) | ((bf16 ? 1u : 0u) << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[tmem] * B[smem]
template <bool ACCUMULATE>
__device__ __forceinline__ void umma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(bdesc), "r"(idesc), "n"(ACCUMULATE ? 1 : 0)
        : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]
template <bool ACCUMULATE>
__device__ __forceinline__ void umma_f16_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "n"(ACCUMULATE ? 1 : 0)
        : "memory");
}

// the mbarrier gets one arrival when every tcgen05 operation this thread issued so far is complete
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 consecutive accumulator columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

// 16 consecutive accumulator columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 16 consecutive columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// 8 consecutive columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr), "r"(r[0]), "r"(r[1]),
                 "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}

__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// TMA tensor load, two coordinates, completion on an mbarrier: a per-CTA load of this GPU's own memory
__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap *tm, int c0, int c1, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                     dst_smem),
                 "l"(reinterpret_cast<uint64_t>(tm)), "r"(c0), "r"(c1), "r"(bar)
                 : "memory");
}

// TMA tensor store, three coordinates; joins the thread's current bulk group
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *tm, int c0, int c1, int c2, uint32_t src_smem)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(
                     reinterpret_cast<uint64_t>(tm)),
                 "r"(c0), "r"(c1), "r"(c2), "r"(src_smem)
                 : "memory");
}

// The A operand of the decode kernels, q sigma rho, is fp16.  A row whose G stored scales (packed 16-bit pairs in sc)
// would take it out of fp16's normal range -- sigma rho above max_t (the largest code times it must fit) or a non-zero
// sigma rho below 2^-14 -- is carried times a power of two instead: the function returns that factor (1 for every other
// row) and its inverse through inv, which the epilogue applies to the row's accumulators in fp32.  The factor takes
// 2^floor(log2(largest sigma rho)) to 2^7, so the largest operand lands in [7 * 128, 7 * 256) (byte codes: below 32512).
template <int G>
__device__ __forceinline__ float operand_rescue(const uint32_t (&sc)[(G + 1) / 2], float rho, float max_t, float &inv)
{
    uint32_t smax = 0u, smin = 0xFFFFu;
#pragma unroll
    for (int c = 0; c < G; ++c) {
        const uint32_t s = (sc[c >> 1] >> (16 * (c & 1))) & 0x7FFFu;   // fp16 bits of a non-negative number order like integers
        smax = max(smax, s);
        if (s != 0u) smin = min(smin, s);
    }
    const float tmax = __half2float(__ushort_as_half((unsigned short)smax)) * rho;
    const float tmin = __half2float(__ushort_as_half((unsigned short)(smin == 0xFFFFu ? 0u : smin))) * rho;
    inv = 1.0f;
    if (!(tmax > max_t || (tmin != 0.0f && tmin < 6.1035156e-5f))) return 1.0f;
    const int e = (int)((__float_as_uint(fminf(fmaxf(tmax, 1e-30f), 1e30f)) >> 23) & 0xFFu) - 127;
    inv = __uint_as_float((uint32_t)(127 - 7 + e) << 23);
    return __uint_as_float((uint32_t)(127 + 7 - e) << 23);
}

// 1 / max(lambda, 1e-6) for the channels this lane covers (4 i .. 4 i + 3, i = lane and, for D > 128, lane + 32),
// divided by rho, the power of two that brings the row's largest reciprocal into [1, 2).  Every lane gets rho.
template <int D>
struct RecipLambda {
    static constexpr int kPasses = (D / 4 + 31) / 32;
    float4 r[kPasses];
    float rho;
    bool wide;   // the reciprocals span more than 2^8: B, which carries them in fp16 next to each other, loses bits on the small ones
    __device__ __forceinline__ RecipLambda(const float *__restrict__ lam, int lane)
    {
        float mx = 0.0f, mn = 3.0e38f;
#pragma unroll
        for (int p = 0; p < kPasses; ++p) {
            const int i = lane + 32 * p;
            r[p] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (i < D / 4) {
                const float4 l = __ldg(reinterpret_cast<const float4 *>(lam) + i);
                r[p] = make_float4(__frcp_rn(fmaxf(l.x, 1e-6f)), __frcp_rn(fmaxf(l.y, 1e-6f)), __frcp_rn(fmaxf(l.z, 1e-6f)),
                                   __frcp_rn(fmaxf(l.w, 1e-6f)));
            }
            mx = fmaxf(mx, fmaxf(fmaxf(r[p].x, r[p].y), fmaxf(r[p].z, r[p].w)));
            if (i < D / 4) mn = fminf(mn, fminf(fminf(r[p].x, r[p].y), fminf(r[p].z, r[p].w)));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
            mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, o));
        }
        rho = __uint_as_float(__float_as_uint(mx) & 0x7F800000u);   // 2^floor(log2 max): exact to divide by
        wide = mn < rho * 0.00390625f;
#pragma unroll
        for (int p = 0; p < kPasses; ++p) r[p].x /= rho, r[p].y /= rho, r[p].z /= rho, r[p].w /= rho;
    }
};

// Bounded wait that also gives up when another role of the CTA has raised the abort flag.  On a
// time-out it raises the flag itself and records `reason` in the status word.
constexpr uint32_t kWaitPolls = 1u << 22;   // polls of a bounded wait before it gives up (seconds of wall time)

__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status,
                                              uint32_t reason, uint32_t limit = kWaitPolls)
{
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 32) {
            if (*abort_flag) return false;
            __nanosleep(32);
        }
    }
    *abort_flag = 1u;
    atomicOr(status, reason);
    return false;
}

// ---- host side: cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda)
typedef CUresult (*TensorMapEncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                           const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                           CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline TensorMapEncodeTiledFn tensor_map_encode_fn()
{
    // looked up once; the initialisation of a function-local static is thread-safe
    static const TensorMapEncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            return reinterpret_cast<TensorMapEncodeTiledFn>(p);
        (void)cudaGetLastError();
        return static_cast<TensorMapEncodeTiledFn>(nullptr);
    }();
    return fn;
}

// A tensor map over `rank` dimensions of `base`; strides in bytes for dimensions 1 .. rank - 1.
inline bool make_tensor_map(CUtensorMap *tm, CUtensorMapDataType type, int rank, const void *base, const cuuint64_t *dims,
                            const cuuint64_t *strides, const cuuint32_t *box, CUtensorMapSwizzle swizzle)
{
    TensorMapEncodeTiledFn enc = tensor_map_encode_fn();
    if (!enc) return false;
    const cuuint32_t es[5] = {1, 1, 1, 1, 1};
    return enc(tm, type, (cuuint32_t)rank, const_cast<void *>(base), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace kvq

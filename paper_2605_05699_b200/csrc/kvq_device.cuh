// Device-side building blocks shared by the libkvq kernels (sm_100a):
// compile-time trigonometry, compile-time loops, PTX wrappers for mbarrier and
// bulk asynchronous copies, and half-precision word helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include <type_traits>
#include <utility>

namespace kvq {

// Bits of the per-plan device status word.
enum : uint32_t {
    KVQ_DEV_LOAD_TIMEOUT = 1u,   // a bounded wait for a bulk load ran out
    KVQ_DEV_MMA_TIMEOUT = 2u,    // a bounded wait for a tensor-core commit ran out
    KVQ_DEV_SLOT_TIMEOUT = 4u,   // a bounded wait for a free pipeline slot ran out
    KVQ_DEV_RANGE = 8u,          // reserved: tiles outside the fp16 operands' range are redone in fp32 by the decode kernels themselves
    KVQ_DEV_POSITION = 16u,      // a cache position read from device memory was outside the cache: nothing was written
};

// ---------------------------------------------------------------------------
// compile-time loops: static_for<N>([&](auto i) { constexpr int I = decltype(i)::value; ... })
// ---------------------------------------------------------------------------
template <class F, int... I>
__device__ __forceinline__ void static_for_impl(F &&f, std::integer_sequence<int, I...>)
{
    (f(std::integral_constant<int, I>{}), ...);
}

template <int N, class F>
__device__ __forceinline__ void static_for(F &&f)
{
    static_for_impl(static_cast<F &&>(f), std::make_integer_sequence<int, N>{});
}

// ---------------------------------------------------------------------------
// compile-time trigonometry: cos / sin of 2 pi n / d with exact octant reduction
// on the integers and a Taylor series on [0, pi/4].  Evaluated by the compiler
// only; every twiddle factor becomes an immediate.
// ---------------------------------------------------------------------------
constexpr double kTwoPi = 6.283185307179586476925286766559;

constexpr double ct_cos_small(double x)
{
    double x2 = x * x, term = 1.0, sum = 1.0;
    for (int i = 1; i <= 13; ++i) {
        term *= -x2 / (double)((2 * i - 1) * (2 * i));
        sum += term;
    }
    return sum;
}

constexpr double ct_sin_small(double x)
{
    double x2 = x * x, term = x, sum = x;
    for (int i = 1; i <= 13; ++i) {
        term *= -x2 / (double)((2 * i) * (2 * i + 1));
        sum += term;
    }
    return sum;
}

constexpr double ct_cos2pi(long long n, long long d)
{
    n %= d;
    if (n < 0) n += d;
    long long a = 8 * n;            // angle = 2 pi a / (8 d); d <-> pi/4, 2d <-> pi/2, 4d <-> pi
    if (a > 4 * d) a = 8 * d - a;   // cos(2 pi - x) = cos x
    bool neg = false;
    if (a > 2 * d) {                // cos(pi - x) = -cos x
        a = 4 * d - a;
        neg = true;
    }
    double r = (a > d) ? ct_sin_small(kTwoPi * (double)(2 * d - a) / (double)(8 * d))   // cos x = sin(pi/2 - x)
                       : ct_cos_small(kTwoPi * (double)a / (double)(8 * d));
    return neg ? -r : r;
}

constexpr double ct_sin2pi(long long n, long long d) { return ct_cos2pi(4 * n - d, 4 * d); }

constexpr double ct_sqrt(double x)
{
    double r = x > 1.0 ? x : 1.0;
    for (int i = 0; i < 200; ++i) r = 0.5 * (r + x / r);
    return r;
}

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// One look at an mbarrier's phase without the hardware's suspend window: true if the phase with this parity is complete.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Waits for the given phase of an mbarrier, but never for ever: after `limit` polls it
// gives up and returns false, so that a lost copy turns into an error code, not a hang.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit = (1u << 22))
{
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 64) __nanosleep(64);
    }
    return false;
}

// global -> shared bulk copy (TMA, untiled); bytes % 16 == 0, both addresses 16-byte aligned.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src_gmem, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src_gmem), "r"(bytes), "r"(bar)
                 : "memory");
}

// shared -> global bulk copy (TMA, untiled); joins the thread's current bulk group.
__device__ __forceinline__ void bulk_store(void *dst_gmem, uint32_t src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst_gmem), "r"(src_smem), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }

// Waits until the shared-memory sources of all this thread's bulk stores have been read.
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// Waits until all this thread's bulk stores have completed.
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Makes generic-proxy writes to shared memory visible to the async proxy (TMA, tensor core).
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---------------------------------------------------------------------------
// Tiles of the tensor-core kernels.  Rows are cut into lambda segments of `rpl` rows, a segment into
// tiles of 128 rows (the last one of a segment may be short), tiles are numbered segment by segment.
// The cursor walks a CTA's tiles without a 64-bit division per step.
// ---------------------------------------------------------------------------
struct TileCursor {
    int64_t seg;   // lambda segment of the current tile
    int64_t tin;   // index of the tile within its segment
    int64_t tps;   // tiles per segment
    __device__ __forceinline__ TileCursor(int64_t tile, int64_t tiles_per_segment)
        : seg(tile / tiles_per_segment), tin(tile - (tile / tiles_per_segment) * tiles_per_segment), tps(tiles_per_segment)
    {
    }
    __device__ __forceinline__ void advance(int step)
    {
        tin += step;
        while (tin >= tps) {
            tin -= tps;
            ++seg;
        }
    }
    __device__ __forceinline__ bool first_of_segment() const { return tin == 0; }
    __device__ __forceinline__ int64_t row_in_segment() const { return tin * 128; }
};

// The contiguous share of a call's tiles that one CTA (or one CTA pair) of a persistent kernel takes: lambda segments of rpl
// rows are cut into tiles of 128 rows (a segment's last tile may be short), n_seg * tps tiles in all, `parts` shares.
// Contiguous, so that the B operand of a lambda row is rebuilt as rarely as possible.  A share that crosses into another
// lambda row pays a rebuild of B, about one tile's time, so with several rows and at least eight tiles per share the shares
// are equal in COST, each segment counting one unit more than its tiles (a share that would begin inside that unit begins
// at the segment's first tile); otherwise they are equal in tiles.
struct TileShare {
    int64_t tps;     // tiles per segment
    int64_t begin;   // first tile of this share
    int n;           // tiles in this share
    __device__ __forceinline__ TileShare(int64_t n_seg, int64_t rpl, unsigned part, unsigned parts)
    {
        tps = (rpl + 127) / 128;
        const int64_t n_tiles = n_seg * tps;
        const int64_t R = (n_seg > 1 && n_tiles >= 8 * (int64_t)parts) ? 1 : 0;   // cost units of a rebuild
        const int64_t C = tps + R, total = n_seg * C;
        const int64_t per = (total + parts - 1) / parts;
        auto tile_of = [&](int64_t u) -> int64_t {
            if (u >= total) return n_tiles;
            const int64_t seg = u / C, w = u - seg * C;
            return seg * tps + (w > R ? w - R : 0);
        };
        begin = tile_of((int64_t)part * per);
        const int64_t end = tile_of(((int64_t)part + 1) * per);
        n = end > begin ? (int)(end - begin) : 0;
    }
};

// ---------------------------------------------------------------------------
// half-precision words: two 16-bit values per 32-bit word, low half first
// ---------------------------------------------------------------------------
template <bool BF16>
__device__ __forceinline__ float2 widen2(uint32_t w)
{
    if constexpr (BF16) {
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
    } else {
        __half2 h = *reinterpret_cast<__half2 *>(&w);
        return __half22float2(h);
    }
}

template <bool BF16>
__device__ __forceinline__ uint32_t narrow2(float lo, float hi)
{
    if constexpr (BF16) {
        __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&b);
    } else {
        __half2 h = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&h);
    }
}

// ---------------------------------------------------------------------------
// round-to-nearest-even codes by the magic-number trick (Sec. 3.2 step 4): v / sigma + 1.5 * 2^23 (+ bias) has the
// biased code in its low mantissa bits, so eight nibbles (four bytes) are gathered with shifts and one subtraction
// ---------------------------------------------------------------------------
constexpr float kMagicRound = 12582912.0f + 8.0f;          // 1.5 * 2^23 + 8: (v + magic) has q + 8 in its low bits
constexpr uint32_t kMagicBits = 0x4B400000u;
constexpr uint32_t kMagicSum = kMagicBits * 0x11111111u;   // sum_i kMagicBits * 16^i  (mod 2^32)
constexpr float kMagicRound8 = 12582912.0f + 128.0f;       // byte codes: q + 128 in the low byte
constexpr uint32_t kMagicSum8 = kMagicBits * 0x01010101u;  // sum_i kMagicBits * 256^i (mod 2^32)

__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));   // (a & b) | c
    return d;
}

}  // namespace kvq

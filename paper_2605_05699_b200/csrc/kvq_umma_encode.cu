// Warp-specialised tcgen05 DFT-as-GEMM encode kernel of libkvq (sm_100a), D = 128, fp16 or bf16 input.
//
// The forward path v = lambda (.) M (s (.) x) (Sec. 3.1 Eq. 1-2, Sec. 5.1 item 1) is a dense D x D
// contraction per vector: v_c = sum_n W[c, n] x_n with W[c, n] = lambda_c M[c, n] s_n.  The codes must
// agree with an fp64 evaluation on all but ~1e-5 of the entries, so W cannot be rounded to 11 bits.
// x is exact in its 16-bit format; W is split into 16-bit terms whose sum carries ~22 bits,
//      fp16 input:  W 2^k = W1 + W2          (two fp16 terms)
//      bf16 input:  W 2^k = W1 + W2 + W3     (three bf16 terms)
// every product x_n W_i[c, n] is exact in fp32, and all terms accumulate in one fp32 accumulator in
// tensor memory.  2^k lifts the small terms clear of fp16's subnormal range; the epilogue undoes it in
// the scale computation, at no cost per element.
//
//   warp 0        producer   two TMA tensor loads per tile of 128 vectors (K blocks of 64 elements,
//                            128-byte swizzle): x lands in shared memory in the tensor core's
//                            canonical K-major layout, four tiles in flight, no thread touches it
//   warp 1        mma        one thread issues 8 K-steps per split term into one of four accumulator
//                            stages, then commits once: the epilogue reads it as "accumulator full",
//                            the producer as "x stage free"
//   warps 2-17    epilogue   two sets of eight warps on alternate tiles; thread = (row, half row).  Per group
//                            of 32 channels: tcgen05.ld of the 32 accumulator columns, abs-max, fp16 scale,
//                            round-to-nearest-even codes, nibble pack (Sec. 3.2 steps 3-4, per-group scales
//                            of Sec. 5.6 / 7.1): no shuffle, no shared memory; 32 bytes of codes and two
//                            scales per thread go straight to global memory.  The accumulator stage is
//                            released as soon as the values are in registers.  The set that meets the first
//                            tile of a new lambda row rebuilds the B operand (the mma warp waits for it on
//                            an mbarrier).
//
//   A [128 vectors, K = 128]   x in shared memory (TMA), K-major, 128-byte swizzle
//   B [N = 128 channels, K]    split terms of W 2^k in shared memory, same layout, one region per term
//   D [128, 128]               fp32 accumulator in tensor memory, four stages
//
// Every wait on an mbarrier is bounded: on a time-out the role records the reason in the status word,
// raises the CTA's abort flag and leaves its loop; the CTA then frees its tensor memory and returns.
#include <cuda.h>

#include "kvq_device.cuh"
#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kD = 128;
constexpr int kTile = 128;                 // vectors per tile = MMA M
constexpr int kGroup = 32;
constexpr int kInStages = 4;               // x tiles in flight (32 KB each)
constexpr int kAccStages = 4;              // accumulators in tensor memory
static_assert(kInStages == kAccStages, "the x stage of tile j is released by the accumulator barrier of tile j");
constexpr int kThreads = 576;              // producer, mma, 16 epilogue warps
constexpr int kEpiWarps = 16;

constexpr int kOpBytes = 2 * kTile * 128;  // 32 KB: one K-major operand, two K blocks of [128 rows x 128 B]
constexpr int kCtrlBytes = 256;
constexpr uint32_t kTmemCols = 512;

constexpr float kMagicRound = 12582912.0f + 8.0f;   // 1.5 * 2^23 + 8: (v + magic) has q + 8 in its low bits
constexpr uint32_t kMagicBits = 0x4B400000u;
constexpr uint32_t kMagicSum = kMagicBits * 0x11111111u;   // sum_i kMagicBits * 16^i  (mod 2^32)

template <bool BF16>
struct Cfg {
    static constexpr int kSplit = BF16 ? 3 : 2;
    static constexpr int kSmemBytes = kSplit * kOpBytes + kInStages * kOpBytes + kCtrlBytes + 1024;
    // instruction descriptor: D = f32, A = B = f16 (0) or bf16 (1), both K-major, N = 128, M = 128
    static constexpr uint32_t kIdesc = (1u << 4) | ((BF16 ? 1u : 0u) << 7) | ((BF16 ? 1u : 0u) << 10) |
                                       ((uint32_t)(kD >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
};

struct Ctrl {
    uint64_t in_full[kInStages];
    uint64_t acc_full[kAccStages], acc_empty[kAccStages];
    uint64_t b_first, b_ready;
    uint32_t tmem_base;
    volatile uint32_t abort;
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    // start address >> 4 | LBO 0 | SBO 1024 B (8 rows x 128 B) | version 1 | 128-byte swizzle
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
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

__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

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

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// TMA tensor load, two coordinates, completion on an mbarrier (no multicast)
__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap *tm, int c0, int c1, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                     dst_smem),
                 "l"(reinterpret_cast<uint64_t>(tm)), "r"(c0), "r"(c1), "r"(bar)
                 : "memory");
}

// byte offset of 16-byte chunk j (0..15 along K) of row r in a [2 K blocks][128 rows][128 B] swizzled operand
__device__ __forceinline__ uint32_t sw128_chunk(int r, int j)
{
    return (uint32_t)((j >> 3) * (kTile * 128) + r * 128 + (((j & 7) ^ (r & 7)) << 4));
}

// Bounded wait that also gives up when another role of the CTA has raised the abort flag.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status,
                                              uint32_t reason)
{
    for (uint32_t it = 0; it < (1u << 22); ++it) {
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

// 2^k for a lambda row: the power of two that brings max_c lambda_c sqrt(2 / D) into [2^13, 2^14), so that
// the first split term of W 2^k stays below fp16's maximum and the later ones above its subnormals.
// Every lane of the warp gets the same value.
__device__ __forceinline__ float lift_of(const float *__restrict__ lam, int lane)
{
    const float4 l = __ldg(reinterpret_cast<const float4 *>(lam) + lane);
    float mx = fmaxf(fmaxf(fabsf(l.x), fabsf(l.y)), fmaxf(fabsf(l.z), fabsf(l.w)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    mx = fminf(fmaxf(mx * 0.125f, 1e-30f), 1e30f);                       // sqrt(2 / 128) = 1 / 8
    const int e = (int)((__float_as_uint(mx) >> 23) & 0xFFu) - 127;      // floor(log2 mx)
    return __uint_as_float((uint32_t)(127 + 13 - e) << 23);
}

// Rows [c0, c1) of every split term of the B operand, by one warp: lane l reads the four table entries
// e0[c][4l .. 4l+3] (one coalesced 512-byte row per step), scales them by lambda_c 2^k, peels off 16-bit
// terms and writes 8 bytes of each term's swizzled row.
template <bool BF16>
__device__ __forceinline__ void build_b_rows(unsigned char *sB, const float *__restrict__ e0, const float *__restrict__ lam, float lift,
                                             int c0, int c1, int lane)
{
    constexpr int kSplit = Cfg<BF16>::kSplit;
#pragma unroll 8
    for (int c = c0; c < c1; ++c) {
        const float4 m = __ldg(reinterpret_cast<const float4 *>(e0 + (size_t)c * kD) + lane);
        const float f = __ldg(lam + c) * lift;
        float w[4] = {m.x * f, m.y * f, m.z * f, m.w * f};
        const uint32_t off = sw128_chunk(c, lane >> 1) + ((lane & 1) ? 8u : 0u);
#pragma unroll
        for (int t = 0; t < kSplit; ++t) {
            const uint32_t lo = narrow2<BF16>(w[0], w[1]), hi = narrow2<BF16>(w[2], w[3]);
            *reinterpret_cast<uint2 *>(sB + t * kOpBytes + off) = make_uint2(lo, hi);
            if (t + 1 < kSplit) {   // what the 16-bit term left behind (exact in fp32)
                const float2 a = widen2<BF16>(lo), b = widen2<BF16>(hi);
                w[0] -= a.x, w[1] -= a.y, w[2] -= b.x, w[3] -= b.y;
            }
        }
    }
}

}  // namespace

struct UmmaEncodeParams {
    const float *lambda;   // [n_lambda, D] fp32
    const float *e0;       // plan table [D, D] fp32: e0[c][n] = M[c][n] s_n
    unsigned char *packed; // [*, D/2] bytes out
    uint16_t *scales;      // [*, D/32] fp16 out
    int64_t N;
    int64_t n_lambda;
    int64_t rpl;           // rows per lambda segment (N when there is one lambda row)
    int64_t n_seg;
    int64_t out_mul, out_add;   // output row of input row r is r * out_mul + out_add
    uint32_t *status;
};

template <bool BF16>
__global__ void __launch_bounds__(kThreads, 1)
    kvq_encode_umma_d128_kernel(const __grid_constant__ UmmaEncodeParams prm, const __grid_constant__ CUtensorMap tm_x)
{
    using C = Cfg<BF16>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sB = smem;                                   // kSplit operands
    unsigned char *sIn = sB + C::kSplit * kOpBytes;             // kInStages x tiles
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(sIn + kInStages * kOpBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kInStages; ++s) {
            mbar_init(smem_u32(&ctrl->in_full[s]), 1);
        }
        for (int s = 0; s < kAccStages; ++s) {
            mbar_init(smem_u32(&ctrl->acc_full[s]), 1);
            mbar_init(smem_u32(&ctrl->acc_empty[s]), kEpiWarps / 2);
        }
        mbar_init(smem_u32(&ctrl->b_first), kEpiWarps);       // first B: all epilogue warps build it
        mbar_init(smem_u32(&ctrl->b_ready), kEpiWarps / 2);   // later rebuilds: the set that owns the tile
        ctrl->abort = 0u;
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    volatile uint32_t *abort_flag = &ctrl->abort;
    uint32_t *status = prm.status;

    // ---- tiles: lambda segments of rpl rows, cut into tiles of 128 rows; a contiguous range per CTA
    const int64_t N = prm.N, rpl = prm.rpl;
    const int64_t tps = (rpl + kTile - 1) / kTile;                 // tiles per segment
    const int64_t n_tiles = prm.n_seg * tps;
    const int64_t per_cta = (n_tiles + gridDim.x - 1) / gridDim.x;
    const int64_t tile_begin = (int64_t)blockIdx.x * per_cta;
    const int64_t tile_end = tile_begin + per_cta < n_tiles ? tile_begin + per_cta : n_tiles;
    const int n_my = tile_end > tile_begin ? (int)(tile_end - tile_begin) : 0;

    if (warp == 0) {
        // =========================== producer ===========================
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            TileCursor cur(tile_begin, tps);
            for (int j = 0; j < n_my; ++j, cur.advance(1)) {
                const int s = j % kInStages;
                // the x stage is free once the MMAs of the tile that used it last are complete: that tile's accumulator barrier
                if (j >= kInStages)
                    ok = wait_or_abort(smem_u32(&ctrl->acc_full[s]), (uint32_t)(j / kInStages - 1) & 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT);
                if (!ok) break;
                const int64_t row0 = cur.seg * rpl + cur.row_in_segment();
                const uint32_t bar = smem_u32(&ctrl->in_full[s]);
                mbar_arrive_expect_tx(bar, kOpBytes);
                tma_load_2d(smem_u32(sIn + s * kOpBytes), &tm_x, 0, (int)row0, bar);
                tma_load_2d(smem_u32(sIn + s * kOpBytes + kTile * 128), &tm_x, 64, (int)row0, bar);
                issued = j + 1;
            }
            if (!ok) {
                // give this thread's own copies in flight a bounded chance to land before the CTA goes away
                for (int j = issued > kInStages ? issued - kInStages : 0; j < issued; ++j)
                    (void)mbar_wait_bounded(smem_u32(&ctrl->in_full[j % kInStages]), (uint32_t)(j / kInStages) & 1u, 1u << 16);
            }
        }
    } else if (warp == 1) {
        // =========================== mma issuer ===========================
        if (lane == 0) {
            // Descriptors differ only in their 14-bit start-address field (bytes >> 4): one base per operand, one add per MMA.
            // The issuing thread is a single instruction stream: what it spends per MMA beyond the issue itself is time
            // the tensor core idles.
            const uint64_t b_desc = smem_desc_sw128(smem_u32(sB));
            const uint64_t a_desc = smem_desc_sw128(smem_u32(sIn));
            const uint32_t b_lo = (uint32_t)b_desc, b_hi = (uint32_t)(b_desc >> 32);
            const uint32_t a_lo = (uint32_t)a_desc, a_hi = (uint32_t)(a_desc >> 32);
            uint32_t builds = 0;
            TileCursor cur(tile_begin, tps);
            for (int j = 0; j < n_my; ++j, cur.advance(1)) {
                const int s = j % kInStages, sc = j % kAccStages;
                if (j == 0) {   // all epilogue warps build the first B while the first x tiles are in flight
                    if (!wait_or_abort(smem_u32(&ctrl->b_first), 0u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                } else if (cur.first_of_segment()) {   // an epilogue set rebuilds B for this lambda row
                    if (!wait_or_abort(smem_u32(&ctrl->b_ready), builds & 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                    ++builds;
                }
                if (!wait_or_abort(smem_u32(&ctrl->in_full[s]), (uint32_t)(j / kInStages) & 1u, abort_flag, status, KVQ_DEV_LOAD_TIMEOUT)) break;
                if (!wait_or_abort(smem_u32(&ctrl->acc_empty[sc]), ((uint32_t)(j / kAccStages) & 1u) ^ 1u, abort_flag, status,
                                   KVQ_DEV_SLOT_TIMEOUT))
                    break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)sc * kD;
                const uint32_t a_lo_s = a_lo + (uint32_t)s * (kOpBytes >> 4);
#pragma unroll
                for (int t = 0; t < C::kSplit; ++t) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        constexpr uint32_t kBlk = (kTile * 128) >> 4;
                        const uint32_t koff = (uint32_t)(ks >> 2) * kBlk + (uint32_t)(ks & 3) * 2u;   // (bytes >> 4) of K-step ks
                        const uint64_t ad = ((uint64_t)a_hi << 32) | (uint64_t)(a_lo_s + koff);
                        const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + (uint32_t)t * (kOpBytes >> 4) + koff);
                        if (t > 0 || ks > 0) umma_f16_ss<true>(d_tmem, ad, bd, C::kIdesc);
                        else umma_f16_ss<false>(d_tmem, ad, bd, C::kIdesc);
                    }
                }
                umma_commit(smem_u32(&ctrl->acc_full[sc]));   // to the epilogue; the producer takes it as "x stage free"
            }
        }
    } else {
        // =========================== epilogue: accumulator -> scales, codes, nibbles ===========================
        // Two sets of eight warps take alternate tiles, so that one set's waits (barrier, tensor-memory load)
        // hide behind the other set's arithmetic.  Thread = (row, half row): groups 2h and 2h + 1.
        const int set = (warp - 2) >> 3;        // this set takes tiles set, set + 2, ...
        const int q = warp & 3;                 // tensor-memory lane quarter this warp may touch
        const int h = ((warp - 2) >> 2) & 1;    // half of the row: channels 64 h .. 64 h + 63
        const int r = q * 32 + lane;            // tile row of this thread
        const int bw = (warp - 2) & 7;          // position within the set: 16 rows of B per warp when the set rebuilds B
        const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(h * 2 * kGroup);
        int64_t cached_seg = -1;
        float unlift = 1.0f;
        if (n_my > 0) {   // B for the CTA's first lambda row: eight rows per warp, all sixteen warps
            TileCursor first(tile_begin, tps);
            const float *lam = prm.lambda + (prm.n_lambda == 1 ? 0 : first.seg) * kD;
            const float lift = lift_of(lam, lane);
            build_b_rows<BF16>(sB, prm.e0, lam, lift, (warp - 2) * 8, (warp - 2) * 8 + 8, lane);
            fence_proxy_async();   // B is read by the tensor core through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->b_first));
            unlift = 1.0f / lift;
            cached_seg = first.seg;
        }
        TileCursor cur(tile_begin + set, tps);
        for (int j = set; j < n_my; j += 2, cur.advance(2)) {
            __syncwarp();
            const int64_t seg = cur.seg;
            const int64_t off = cur.row_in_segment();

            // ---- a new lambda row.  Every set needs its lift; the set that owns the row's first tile rebuilds B,
            // ---- once every MMA that read the old B is complete (the previous tile's accumulator is full), and
            // ---- tells the mma warp.
            if (seg != cached_seg) {
                const float *lam = prm.lambda + (prm.n_lambda == 1 ? 0 : seg) * kD;
                const float lift = lift_of(lam, lane);
                if (j > 0 && cur.first_of_segment()) {
                    if (!wait_or_abort(smem_u32(&ctrl->acc_full[(j - 1) % kAccStages]), (uint32_t)((j - 1) / kAccStages) & 1u,
                                       abort_flag, status, KVQ_DEV_MMA_TIMEOUT))
                        break;
                    build_b_rows<BF16>(sB, prm.e0, lam, lift, bw * 16, bw * 16 + 16, lane);
                    fence_proxy_async();   // B is read by the tensor core through the async proxy
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctrl->b_ready));
                }
                unlift = 1.0f / lift;
                cached_seg = seg;
            }

            const int sc = j % kAccStages;
            if (!wait_or_abort(smem_u32(&ctrl->acc_full[sc]), (uint32_t)(j / kAccStages) & 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT)) break;
            tc_fence_after();

            // ---- rows of the tile that exist: the segment (and with it the tensor) may end inside the tile
            int64_t seg_rows = N - seg * rpl;
            if (seg_rows > rpl) seg_rows = rpl;
            const bool live = off + r < seg_rows;
            const int64_t orow = (seg * rpl + off + r) * prm.out_mul + prm.out_add;
            uint32_t sbits = 0;
#pragma unroll
            for (int gg = 0; gg < 2; ++gg) {
                uint32_t vb[32];
                tmem_ld32(t_addr + (uint32_t)sc * kD + (uint32_t)(gg * kGroup), vb);
                tmem_ld_wait();
                if (gg == 1) {   // both groups are in registers: hand the accumulator back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctrl->acc_empty[sc]));
                }
                // ---- scale: sigma = fp16(absmax / 7); codes are taken against the stored value
                float amax = 0.0f;
#pragma unroll
                for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(__uint_as_float(vb[i])));
                amax *= unlift;
                const float sig = fminf(__fdiv_rn(amax, 7.0f), 65504.0f);
                const __half hs = __float2half_rn(sig);
                const float sg = __half2float(hs);
                const float rs1 = sg > 0.0f ? __frcp_rn(sg) : 0.0f;
                const bool clamp = !(amax * rs1 < 7.25f);   // saturated or subnormal scale: codes could leave [-7, 7]
                const float rs = rs1 * unlift;              // applies to the lifted accumulator values
                sbits |= (uint32_t)__half_as_ushort(hs) << (16 * gg);

                // ---- round, bias to unsigned nibbles, pack 8 codes per word
                uint32_t words[4];
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    uint32_t acc = 0;
                    if (!clamp) {
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            acc += __float_as_uint(fmaf(__uint_as_float(vb[8 * w + e]), rs, kMagicRound)) << (4 * e);
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            acc += __float_as_uint(fminf(fmaxf(__uint_as_float(vb[8 * w + e]) * rs, -7.0f), 7.0f) + kMagicRound) << (4 * e);
                    }
                    words[w] = (acc - kMagicSum) ^ 0x88888888u;
                }
                if (live)
                    *reinterpret_cast<uint4 *>(prm.packed + orow * (kD / 2) + (2 * h + gg) * 16) =
                        make_uint4(words[0], words[1], words[2], words[3]);
            }
            if (live) *reinterpret_cast<uint32_t *>(prm.scales + orow * (kD / kGroup) + 2 * h) = sbits;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        if (*abort_flag) __nanosleep(20000);   // let tensor-core work that was already issued drain
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            (void)cudaGetLastError();
    }
    return fn;
}

template <bool BF16>
cudaError_t launch(const UmmaEncodeParams &prm, const CUtensorMap &tm_x, int64_t tiles, cudaStream_t stream)
{
    static int sms = 0;
    if (sms == 0) {
        cudaError_t e = cudaFuncSetAttribute(kvq_encode_umma_d128_kernel<BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg<BF16>::kSmemBytes);
        if (e != cudaSuccess) return e;
        int dev = 0;
        if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    }
    const int grid = (int)(tiles < sms ? tiles : sms);
    kvq_encode_umma_d128_kernel<BF16><<<grid, kThreads, Cfg<BF16>::kSmemBytes, stream>>>(prm, tm_x);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t umma_encode_d128(bool bf16, int64_t N, const FftParams &f, const float *e0, cudaStream_t stream)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return cudaErrorNotSupported;
    if (N >= (int64_t)1 << 31) return cudaErrorInvalidValue;   // tensor-map coordinates are 32-bit

    UmmaEncodeParams prm;
    prm.lambda = f.lambda;
    prm.e0 = e0;
    prm.packed = static_cast<unsigned char *>(f.packed);
    prm.scales = static_cast<uint16_t *>(f.scales);
    prm.N = N;
    prm.n_lambda = f.n_lambda;
    prm.rpl = f.n_lambda == 1 ? N : f.rows_per_lambda;
    prm.n_seg = (N + prm.rpl - 1) / prm.rpl;
    prm.out_mul = f.out_mul;
    prm.out_add = f.out_add;
    prm.status = f.status;

    CUtensorMap tm_x;
    const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)N};
    const cuuint64_t strides[1] = {(cuuint64_t)(2 * kD)};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    const cuuint32_t es[2] = {1, 1};
    if (enc(&tm_x, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(f.in), dims, strides,
            box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;

    const int64_t tiles = prm.n_seg * ((prm.rpl + kTile - 1) / kTile);
    return bf16 ? launch<true>(prm, tm_x, tiles, stream) : launch<false>(prm, tm_x, tiles, stream);
}

}  // namespace kvq

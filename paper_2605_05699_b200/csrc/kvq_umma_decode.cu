// Warp-specialised tcgen05 DFT-as-GEMM decode kernel of libkvq (sm_100a), D = 128, fp16 output.
//
// The inverse path x^ = diag(s) M^T diag(1 / max(lambda, 1e-6)) (q (.) sigma) (Sec. 3.1 "unpack, irfft,
// apply s"; Sec. 5.1 item 1) is a dense D x D contraction per vector.  A tile of 128 vectors is one
// 128 x 128 x 128 GEMM on the 5th-generation tensor core, a quarter of the time the tile's bytes need
// to cross HBM, so the kernel's job is to keep HBM busy: one persistent CTA per SM runs four roles that
// hand tiles to one another through mbarriers and never wait for one another's latency.
//
//   warp 0        producer   one TMA tensor load per tile: 128 packed rows (8 KB) into a ring of
//                            shared-memory stages (64-byte swizzle, so that row-per-thread reads
//                            are free of bank conflicts)
//   warps 2-9     dequant    two groups of four warps that take alternate tiles.  Thread t of a group
//                            owns row t: nibbles -> fp16 codes -> times sigma * rho, two codes per
//                            half2 instruction, stored straight into TENSOR MEMORY as the A operand
//                            (tcgen05.st); the group scales come by plain loads, one tile ahead.
//                            The group that meets the first tile of a new lambda row rebuilds B.
//   warp 1        mma        one thread issues 8 K-steps of tcgen05.mma (A from tensor memory, B from
//                            shared memory) into one of two accumulator stages and commits
//   warps 10-17   epilogue   two groups of four warps, alternate tiles.  Thread t reads accumulator
//                            row t (tcgen05.ld), rounds to fp16, writes a 128-byte-swizzled staging
//                            tile; one lane per warp issues two TMA tensor stores (32 rows x 128 B
//                            each).  The output tensor map is three-dimensional (column, row within
//                            lambda segment, segment), so the hardware clips a tile that ends with
//                            its segment or with the tensor: no per-row tail code.
//
//   A [128 vectors, K = 128]  fp16 in tensor memory: lane = vector, 64 columns of two codes each
//   B [N = 128 outputs, K]    fp16 in shared memory, K-major, 128-byte swizzle:
//                             W'[n, c] = s_n M[c, n] / max(lambda_c, 1e-6) / rho, rho a power of two
//   D [128, 128]              fp32 accumulator in tensor memory, two stages
//
// The K order inside a word of 8 codes is (0,4,1,5,2,6,3,7): that is how the half2 nibble trick
// delivers them, and B is built in the same order, so no instruction is spent on reordering.
//
// Precision: A and B are each rounded once to fp16, accumulation is fp32: about 3e-4 relative L2 per
// vector before the output rounding.  Every wait on an mbarrier is bounded: on a time-out the role
// records the reason in the status word, raises the CTA's abort flag and leaves its loop; the CTA
// then frees its tensor memory and returns.
#include <cuda.h>

#include "kvq_device.cuh"
#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kD = 128;
constexpr int kTile = 128;                 // vectors per tile = MMA M
constexpr int kInStages = 6;               // packed tiles in flight
constexpr int kAStages = 4;                // A operands in tensor memory
constexpr int kAccStages = 2;              // accumulators in tensor memory
constexpr int kThreads = 576;              // producer, mma, 2 x 4 dequant, 2 x 4 epilogue warps

constexpr int kBBytes = 2 * kTile * 128;               // 32 KB: two K blocks of [128 rows x 128 B]
constexpr int kInBytes = kTile * (kD / 2);             // 8 KB per packed tile
constexpr int kOutWarpBytes = 2 * 32 * 128;            // 8 KB: two column halves of [32 rows x 128 B]
constexpr int kOutBytes = 8 * kOutWarpBytes;           // one staging tile per epilogue warp
constexpr int kCtrlBytes = 256;
constexpr int kSmemBytes = kBBytes + kInStages * kInBytes + kOutBytes + kCtrlBytes + 1024;

constexpr uint32_t kAccCol0 = 0;                       // 2 x 128 accumulator columns
constexpr uint32_t kACol0 = kAccStages * kD;           // then 4 x 64 columns of A
constexpr uint32_t kTmemCols = 512;

// instruction descriptor: D = f32, A = B = f16, both K-major, N = 128, M = 128
constexpr uint32_t kIdesc = (1u << 4) | ((uint32_t)(kD >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);

struct Ctrl {
    uint64_t in_full[kInStages], in_empty[kInStages];
    uint64_t a_full[kAStages], a_empty[kAStages];
    uint64_t acc_full[kAccStages], acc_empty[kAccStages];
    uint64_t b_first;
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

// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void umma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
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

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// TMA tensor load, two coordinates, completion on an mbarrier (no multicast)
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


__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));   // (a & b) | c
    return d;
}

// byte offset of 16-byte chunk j (0..15 along K) of row r in a [2 K blocks][128 rows][128 B] swizzled operand
__device__ __forceinline__ uint32_t sw128_chunk(int r, int j)
{
    return (uint32_t)((j >> 3) * (kTile * 128) + r * 128 + (((j & 7) ^ (r & 7)) << 4));
}

// 1 / max(lambda, 1e-6) for the four channels 4 lane .. 4 lane + 3 of lambda row `lam`, divided by rho, the
// power of two that brings the row's largest reciprocal into [1, 2).  Every lane of the warp gets rho.
__device__ __forceinline__ float4 recip_lambda4(const float *__restrict__ lam, int lane, float &rho)
{
    const float4 l = __ldg(reinterpret_cast<const float4 *>(lam) + lane);
    float4 r = make_float4(__frcp_rn(fmaxf(l.x, 1e-6f)), __frcp_rn(fmaxf(l.y, 1e-6f)), __frcp_rn(fmaxf(l.z, 1e-6f)),
                           __frcp_rn(fmaxf(l.w, 1e-6f)));
    float mx = fmaxf(fmaxf(r.x, r.y), fmaxf(r.z, r.w));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    rho = __uint_as_float(__float_as_uint(mx) & 0x7F800000u);   // 2^floor(log2 max): exact to divide by
    r.x /= rho, r.y /= rho, r.z /= rho, r.w /= rho;
    return r;
}

// Rows [n0, n1) of the B operand, by one warp: lane l reads the four table entries b0[n][4l .. 4l+3]
// (one coalesced 512-byte row per step), scales them, trades two values with its neighbour so that each
// lane holds two K-ordered pairs, and writes 8 bytes of the swizzled row.
__device__ __forceinline__ void build_b_rows(unsigned char *sB, const float *__restrict__ b0, float4 rl, int n0, int n1, int lane)
{
    const bool odd = lane & 1;
    const int w = lane >> 1;   // word of 8 codes = 16-byte chunk of the K-major row
#pragma unroll 8
    for (int n = n0; n < n1; ++n) {
        const float4 m = __ldg(reinterpret_cast<const float4 *>(b0 + (size_t)n * kD) + lane);
        auto sat = [](float v) { return fminf(fmaxf(v, -65504.0f), 65504.0f); };
        const float vx = sat(m.x * rl.x), vy = sat(m.y * rl.y), vz = sat(m.z * rl.z), vw = sat(m.w * rl.w);
        // even lane holds codes 8w .. 8w+3, odd lane 8w+4 .. 8w+7; K order of the word is (0,4,1,5,2,6,3,7)
        const float r0 = __shfl_xor_sync(0xFFFFFFFFu, odd ? vx : vz, 1);
        const float r1 = __shfl_xor_sync(0xFFFFFFFFu, odd ? vy : vw, 1);
        uint2 o;
        o.x = odd ? narrow2<false>(r0, vz) : narrow2<false>(vx, r0);   // odd: (2, 6)   even: (0, 4)
        o.y = odd ? narrow2<false>(r1, vw) : narrow2<false>(vy, r1);   // odd: (3, 7)   even: (1, 5)
        *reinterpret_cast<uint2 *>(sB + sw128_chunk(n, w) + (odd ? 8 : 0)) = o;
    }
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

}  // namespace

struct UmmaDecodeParams {
    GemmParams g;
    int64_t rpl;        // rows per lambda segment (N when there is one lambda row)
    int64_t n_seg;      // segments
    int64_t n_full;     // segments of exactly rpl rows, covered by the main output map; a shorter last one uses the tail map
};

__global__ void __launch_bounds__(kThreads, 1)
    kvq_decode_umma_d128_kernel(const __grid_constant__ UmmaDecodeParams prm, const __grid_constant__ CUtensorMap tm_packed,
                                const __grid_constant__ CUtensorMap tm_out, const __grid_constant__ CUtensorMap tm_out_tail)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sB = smem;
    unsigned char *sIn = sB + kBBytes;
    unsigned char *sOut = sIn + kInStages * kInBytes;
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(sOut + kOutBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kInStages; ++s) {
            mbar_init(smem_u32(&ctrl->in_full[s]), 1);
            mbar_init(smem_u32(&ctrl->in_empty[s]), 4);
        }
        for (int s = 0; s < kAStages; ++s) {
            mbar_init(smem_u32(&ctrl->a_full[s]), 4);
            mbar_init(smem_u32(&ctrl->a_empty[s]), 1);
        }
        for (int s = 0; s < kAccStages; ++s) {
            mbar_init(smem_u32(&ctrl->acc_full[s]), 1);
            mbar_init(smem_u32(&ctrl->acc_empty[s]), 4);
        }
        mbar_init(smem_u32(&ctrl->b_first), 16);   // first B: the sixteen dequant and epilogue warps build it
        ctrl->abort = 0u;
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);

    // ---- tiles: lambda segments of rpl rows, cut into tiles of 128 rows; a contiguous range of tiles
    // ---- per CTA, so that the B operand is rebuilt as rarely as possible
    const int64_t N = prm.g.N, rpl = prm.rpl;
    const int64_t tps = (rpl + kTile - 1) / kTile;                 // tiles per segment
    const int64_t n_tiles = prm.n_seg * tps;
    const int64_t per_cta = (n_tiles + gridDim.x - 1) / gridDim.x;
    const int64_t tile_begin = (int64_t)blockIdx.x * per_cta;
    const int64_t tile_end = tile_begin + per_cta < n_tiles ? tile_begin + per_cta : n_tiles;
    const int n_my = tile_end > tile_begin ? (int)(tile_end - tile_begin) : 0;
    const int64_t seg_first = n_my > 0 ? tile_begin / tps : 0;
    auto lambda_row = [&](int64_t seg) -> const float * { return prm.g.lambda + (prm.g.n_lambda == 1 ? 0 : seg) * kD; };

    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    volatile uint32_t *abort_flag = &ctrl->abort;
    uint32_t *status = prm.g.status;

    // ---- B for the first tile's lambda row: the sixteen dequant and epilogue warps build eight rows each while the
    // ---- producer's first loads are in flight; the mma warp waits for all of them
    if (n_my > 0 && warp >= 2) {
        float rho;
        const float4 rl = recip_lambda4(lambda_row(seg_first), lane, rho);
        build_b_rows(sB, prm.g.b0, rl, (warp - 2) * 8, (warp - 2) * 8 + 8, lane);
        fence_proxy_async();   // B is read by the tensor core through the async proxy
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->b_first));
    }

    if (warp == 0) {
        // =========================== producer ===========================
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            TileCursor cur(tile_begin, tps);
            for (int j = 0; j < n_my; ++j, cur.advance(1)) {
                const int s = j % kInStages;
                const uint32_t use = (uint32_t)(j / kInStages);
                ok = wait_or_abort(smem_u32(&ctrl->in_empty[s]), (use & 1u) ^ 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT);
                if (!ok) break;
                const int64_t row0 = cur.seg * rpl + cur.row_in_segment();
                const uint32_t bar = smem_u32(&ctrl->in_full[s]);
                mbar_arrive_expect_tx(bar, kInBytes);
                tma_load_2d(smem_u32(sIn + s * kInBytes), &tm_packed, 0, (int)row0, bar);
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
            const uint32_t b_addr = smem_u32(sB);
            int n_mma = n_my;
            if (n_my > 0 && !wait_or_abort(smem_u32(&ctrl->b_first), 0u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) n_mma = 0;
            for (int j = 0; j < n_mma; ++j) {
                const int sa = j % kAStages, sc = j % kAccStages;
                if (!wait_or_abort(smem_u32(&ctrl->a_full[sa]), (uint32_t)(j / kAStages) & 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                if (!wait_or_abort(smem_u32(&ctrl->acc_empty[sc]), ((uint32_t)(j / kAccStages) & 1u) ^ 1u, abort_flag, status,
                                   KVQ_DEV_SLOT_TIMEOUT))
                    break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + kAccCol0 + (uint32_t)sc * kD;
                const uint32_t a_tmem = tmem_base + kACol0 + (uint32_t)sa * (kD / 2);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t koff = (uint32_t)((ks >> 2) * (kTile * 128) + (ks & 3) * 32);
                    umma_f16_ts(d_tmem, a_tmem + (uint32_t)ks * 8u, smem_desc_sw128(b_addr + koff), kIdesc, ks > 0 ? 1u : 0u);
                }
                umma_commit(smem_u32(&ctrl->acc_full[sc]));
                umma_commit(smem_u32(&ctrl->a_empty[sa]));
            }
        }
    } else if (warp < 10) {
        // =========================== dequant: packed codes -> A in tensor memory ===========================
        const int grp = (warp - 2) >> 2;        // this group takes tiles grp, grp + 2, ...
        const int q = warp & 3;                 // tensor-memory lane quarter this warp may touch
        const int r = q * 32 + lane;            // tile row and tensor-memory lane of this thread
        const uint2 *scales = static_cast<const uint2 *>(prm.g.scales);   // 4 fp16 scales per row
        const uint32_t swz = (uint32_t)((r >> 1) & 3);
        int64_t cached_seg = n_my > 0 ? seg_first : -1;   // B holds this row's table (built above)
        float rho;
        (void)recip_lambda4(lambda_row(seg_first), lane, rho);

        TileCursor cur(tile_begin + grp, tps), ahead(tile_begin + grp, tps);   // this tile; the tile whose scales are fetched
        auto load_scales = [&](int j) -> uint2 {
            if (j >= n_my) return make_uint2(0u, 0u);
            const int64_t row = ahead.seg * rpl + ahead.row_in_segment() + r;
            return row < N ? __ldg(scales + row) : make_uint2(0u, 0u);
        };

        uint2 sc_next = load_scales(grp);
        for (int j = grp; j < n_my; j += 2, cur.advance(2)) {
            const uint2 sc = sc_next;
            ahead.advance(2);
            sc_next = load_scales(j + 2);
            const int64_t seg = cur.seg;

            // ---- a new lambda row: this group needs its rho; the group that meets the row's first tile rebuilds B
            if (seg != cached_seg) {
                const float4 rl = recip_lambda4(lambda_row(seg), lane, rho);
                if (cur.first_of_segment()) {
                    // Every MMA issued so far has read B: the commit of the previous tile (the other group's) covers them
                    // all.  A parity wait can only tell a phase from its neighbours, and the other group may lag by more
                    // than one of its tiles, so first wait for this group's own last tile (its barrier is at most one
                    // phase behind, this group waited on it before writing that tile): MMAs complete in order, so after it
                    // the previous tile's barrier is at most one phase behind too.
                    if (j >= 2 && !wait_or_abort(smem_u32(&ctrl->a_empty[(j - 2) % kAStages]), (uint32_t)((j - 2) / kAStages) & 1u,
                                                 abort_flag, status, KVQ_DEV_MMA_TIMEOUT))
                        break;
                    if (!wait_or_abort(smem_u32(&ctrl->a_empty[(j - 1) % kAStages]), (uint32_t)((j - 1) / kAStages) & 1u, abort_flag,
                                       status, KVQ_DEV_MMA_TIMEOUT))
                        break;
                    build_b_rows(sB, prm.g.b0, rl, q * 32, q * 32 + 32, lane);
                    fence_proxy_async();   // B is read by the tensor core through the async proxy
                }
                cached_seg = seg;
            }

            // ---- this tile's packed rows have landed; the A stage is free again
            const int s = j % kInStages, sa = j % kAStages;
            if (!wait_or_abort(smem_u32(&ctrl->in_full[s]), (uint32_t)(j / kInStages) & 1u, abort_flag, status, KVQ_DEV_LOAD_TIMEOUT)) break;
            uint4 pk[4];
            {
                const unsigned char *row = sIn + s * kInBytes + r * (kD / 2);
#pragma unroll
                for (int c = 0; c < 4; ++c) pk[c] = *reinterpret_cast<const uint4 *>(row + (((uint32_t)c ^ swz) << 4));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->in_empty[s]));   // the values are in registers
            if (!wait_or_abort(smem_u32(&ctrl->a_empty[sa]), ((uint32_t)(j / kAStages) & 1u) ^ 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT))
                break;
            tc_fence_after();

            // ---- nibbles -> fp16 codes -> times sigma * rho, two codes per instruction
            const uint32_t a_row = tmem_base + ((uint32_t)(q * 32) << 16) + kACol0 + (uint32_t)sa * (kD / 2);
            const __half2 sa2 = *reinterpret_cast<const __half2 *>(&sc.x), sb2 = *reinterpret_cast<const __half2 *>(&sc.y);
            const float2 fa = __half22float2(sa2), fb = __half22float2(sb2);
            const float sg[4] = {fa.x * rho, fa.y * rho, fb.x * rho, fb.y * rho};
            const __half2 h1032 = __float2half2_rn(1032.0f);
#pragma unroll
            for (int c = 0; c < 4; ++c) {   // chunk c = group c: 32 codes, 16 tensor-memory columns
                const __half2 s2 = __float2half2_rn(sg[c]);
                const uint32_t words[4] = {pk[c].x, pk[c].y, pk[c].z, pk[c].w};
                uint32_t a[16];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t u = words[i] ^ 0x88888888u;   // nibbles now hold q + 8
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const uint32_t m = lop3_and_or(u >> (4 * e), 0x000F000Fu, 0x64006400u);   // {1024 + n_e, 1024 + n_{e+4}}
                        const __half2 h = __hmul2(__hsub2(*reinterpret_cast<const __half2 *>(&m), h1032), s2);   // exact q, one rounding
                        a[4 * i + e] = *reinterpret_cast<const uint32_t *>(&h);
                    }
                }
                tmem_st16(a_row + 16u * (uint32_t)c, a);
            }
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->a_full[sa]));
        }
    } else {
        // =========================== epilogue: accumulator -> fp16 -> TMA store ===========================
        const int grp = (warp - 10) >> 2;
        const int q = warp & 3;
        unsigned char *stg = sOut + (warp - 10) * kOutWarpBytes;   // this warp's staging tile: two [32 rows x 128 B] halves
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16) + kAccCol0;
        TileCursor cur(tile_begin + grp, tps);
        for (int j = grp; j < n_my; j += 2, cur.advance(2)) {
            const int sc = j % kAccStages;
            if (!wait_or_abort(smem_u32(&ctrl->acc_full[sc]), (uint32_t)(j / kAccStages) & 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT)) break;
            tc_fence_after();
            if (lane == 0) bulk_wait_read_all();   // this warp's previous stores have read the staging tile
            __syncwarp();
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {   // 32 accumulator columns = 64 bytes of the output row
                uint32_t v[32];
                tmem_ld32(lane_addr + (uint32_t)sc * kD + (uint32_t)cc * 32u, v);
                tmem_ld_wait();
                unsigned char *half_base = stg + (cc >> 1) * (32 * 128) + lane * 128;   // column half = one store box
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    uint4 o;
                    o.x = narrow2<false>(__uint_as_float(v[8 * k]), __uint_as_float(v[8 * k + 1]));
                    o.y = narrow2<false>(__uint_as_float(v[8 * k + 2]), __uint_as_float(v[8 * k + 3]));
                    o.z = narrow2<false>(__uint_as_float(v[8 * k + 4]), __uint_as_float(v[8 * k + 5]));
                    o.w = narrow2<false>(__uint_as_float(v[8 * k + 6]), __uint_as_float(v[8 * k + 7]));
                    const int chunk = (cc & 1) * 4 + k;   // 16-byte chunk of the 128-byte half row
                    *reinterpret_cast<uint4 *>(half_base + ((chunk ^ (lane & 7)) << 4)) = o;
                }
            }
            tc_fence_before();
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&ctrl->acc_empty[sc]));
                const int64_t seg = cur.seg;
                const int row_in_seg = (int)cur.row_in_segment() + q * 32;
                const bool tail = seg >= prm.n_full;
                const CUtensorMap *tm = tail ? &tm_out_tail : &tm_out;
                const int segc = tail ? 0 : (int)seg;
                tma_store_3d(tm, 0, row_in_seg, segc, smem_u32(stg));
                tma_store_3d(tm, 64, row_in_seg, segc, smem_u32(stg + 32 * 128));
                bulk_commit();
            }
        }
        if (lane == 0) bulk_wait_all();
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

}  // namespace

cudaError_t umma_decode_d128(int64_t N, const GemmParams &g, cudaStream_t stream)
{
    static int sms = 0;
    if (sms == 0) {
        cudaError_t e = cudaFuncSetAttribute(kvq_decode_umma_d128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        int dev = 0;
        if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    }
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return cudaErrorNotSupported;
    if (N >= (int64_t)1 << 31) return cudaErrorInvalidValue;   // tensor-map coordinates are 32-bit

    UmmaDecodeParams prm;
    prm.g = g;
    prm.rpl = g.n_lambda == 1 ? N : g.rows_per_lambda;
    prm.n_seg = (N + prm.rpl - 1) / prm.rpl;
    prm.n_full = N / prm.rpl;

    CUtensorMap tm_packed, tm_out, tm_tail;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)(kD / 2), (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)(kD / 2)};
        const cuuint32_t box[2] = {(cuuint32_t)(kD / 2), (cuuint32_t)kTile};
        const cuuint32_t es[2] = {1, 1};
        if (enc(&tm_packed, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(g.packed), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    auto out_map = [&](CUtensorMap *tm, void *base, int64_t rows, int64_t segs) -> bool {
        const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)rows, (cuuint64_t)segs};
        const cuuint64_t strides[2] = {(cuuint64_t)(2 * kD), (cuuint64_t)(2 * kD) * (cuuint64_t)rows};
        const cuuint32_t box[3] = {64, 32, 1};
        const cuuint32_t es[3] = {1, 1, 1};
        return enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    const int64_t tail_rows = N - prm.n_full * prm.rpl;
    if (prm.n_full > 0) {
        if (!out_map(&tm_out, g.out, prm.rpl, prm.n_full)) return cudaErrorInvalidValue;
    }
    if (tail_rows > 0) {
        unsigned char *base = static_cast<unsigned char *>(g.out) + (size_t)prm.n_full * prm.rpl * (2 * kD);
        if (!out_map(&tm_tail, base, tail_rows, 1)) return cudaErrorInvalidValue;
    } else {
        tm_tail = tm_out;
    }
    if (prm.n_full == 0) tm_out = tm_tail;

    const int64_t tiles = prm.n_seg * ((prm.rpl + kTile - 1) / kTile);
    const int grid = (int)(tiles < sms ? tiles : sms);
    kvq_decode_umma_d128_kernel<<<grid, kThreads, kSmemBytes, stream>>>(prm, tm_packed, tm_out, tm_tail);
    count_launch();
    return cudaGetLastError();
}

}  // namespace kvq

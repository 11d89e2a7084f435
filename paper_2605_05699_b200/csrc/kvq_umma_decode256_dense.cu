// Warp-specialised tcgen05 decode kernel of libkvq (sm_100a) for D = 256 with a DENSE 256 x 256 table, fp16 or
// bf16 output.  It serves plans that carry a rotation (Sec. 5.1 item 2): their table R-rotated has no even / odd
// structure left, so the radix-2 kernel of kvq_umma_decode256.cu does not apply.
//
// Same contraction as kvq_umma_decode.cu, x^ = diag(s) M^T diag(1 / max(lambda, 1e-6)) (q (.) sigma) (Sec. 3.1,
// Sec. 5.1 item 1), with two changes that D = 256 forces:
//
//   * the B operand (256 x 256) does not fit one CTA's shared memory next to the staging buffers once it
//     is split for precision, so CTAs work in pairs on the same tiles and each computes one half of the
//     output columns: B is [128 outputs, K = 256] per CTA.  The two CTAs of a pair share nothing and never
//     wait for each other; the packed tile is read twice (the second read hits L2).
//   * bf16 output has a rounding step 8x coarser than fp16, and a result that is off by 1e-4 of the
//     vector's rms already lands on the other side of enough rounding boundaries to miss the 1e-3
//     tolerance.  So for bf16 both operands are carried in two fp16 terms: a = q sigma rho has 15
//     significant bits and splits exactly into a_hi + a_lo (one half2 FMA), W' = W_hi + W_lo, and
//     x^ = a_hi W_hi + a_lo W_hi + a_hi W_lo accumulates in fp32 (the a_lo W_lo term is below 1e-7).
//     fp16 output needs one term.
//
// The A operand lives in tensor memory by K halves (128 codes: 64 columns, twice that with a_lo), two
// stages; the accumulator (128 columns) has two stages.  Roles as in kvq_umma_decode.cu: producer (TMA),
// two dequant groups, one mma thread, two epilogue groups; every wait is bounded.
#include "kvq_decode_fp32.cuh"
#include "kvq_internal.h"
#include "kvq_umma.cuh"

namespace kvq {

namespace {

constexpr int kD = 256;
constexpr int kG = kD / 32;
constexpr int kTile = 128;       // vectors per tile = MMA M
constexpr int kHalfN = 128;      // output columns per CTA = MMA N
constexpr int kThreads = 576;    // producer, mma, 2 x 4 dequant, 2 x 4 epilogue warps
constexpr int kInStages = 4;     // packed tiles in flight (16 KB each); even, so that a stage always serves the same dequant group
constexpr int kAStages = 2;      // K halves of A in tensor memory
constexpr int kAccStages = 2;
constexpr int kInBytes = kTile * (kD / 2);             // 16 KB
constexpr int kBBlock = kHalfN * 128;                  // one K block of 64: 128 rows x 128 B
constexpr int kBTerm = 4 * kBBlock;                    // 64 KB: K = 256
constexpr int kOutWarpBytes = 32 * 128;                // one 64-column box per epilogue warp
constexpr int kCtrlBytes = 256;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kACol0 = 256;                       // accumulators at 0 and 128; A stages of 128 columns behind them
constexpr uint32_t kIdesc = umma_idesc_m128(kHalfN, false);

template <bool BF16OUT>
struct Cfg {
    static constexpr int kBTerms = BF16OUT ? 2 : 1;    // W_hi (, W_lo)
    static constexpr int kSmemBytes = kBTerms * kBTerm + kInStages * kInBytes + 8 * kOutWarpBytes + kCtrlBytes + 1024;
};

struct Ctrl {
    uint64_t in_full[kInStages], in_empty[kInStages];
    uint64_t a_full[kAStages], a_empty[2][kAStages];   // a_empty[g][s]: a unit of dequant group g has been read from stage s
    uint64_t acc_full[kAccStages], acc_empty[kAccStages];
    uint64_t b_first;
    uint32_t tmem_base;
    volatile uint32_t abort;
    volatile uint32_t any_wide;  // a lambda row too wide for the fp16 B operand, or a scale outside A's range: tiles redone in fp32 at the end
    volatile uint32_t b_epoch;   // lambda rows whose last MMA is complete, counted from the CTA's first one
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

// Rows [n0, n1) of this CTA's half of the B operand (output column 128 half + n), by one warp.  A lane reads four
// table entries per pass, scales them, trades two values with its neighbour so that each lane holds two K-ordered
// pairs (the K order of a word of 8 codes is (0,4,1,5,2,6,3,7)), peels off fp16 terms and writes 8 bytes of each
// term's swizzled row.
template <int TERMS>
__device__ __forceinline__ void build_b_rows(unsigned char *sB, const float *__restrict__ b0, const RecipLambda<kD> &rl, int half, int n0,
                                             int n1, int lane)
{
    const bool odd = lane & 1;
#pragma unroll 2
    for (int n = n0; n < n1; ++n) {
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            const int i = lane + 32 * p;
            const float4 m = __ldg(reinterpret_cast<const float4 *>(b0 + (size_t)(half * kHalfN + n) * kD) + i);
            auto sat = [](float v) { return fminf(fmaxf(v, -65504.0f), 65504.0f); };
            const float vx = sat(m.x * rl.r[p].x), vy = sat(m.y * rl.r[p].y), vz = sat(m.z * rl.r[p].z), vw = sat(m.w * rl.r[p].w);
            const float r0 = __shfl_xor_sync(0xFFFFFFFFu, odd ? vx : vz, 1);
            const float r1 = __shfl_xor_sync(0xFFFFFFFFu, odd ? vy : vw, 1);
            float w[4];   // two K-ordered pairs: odd lane (2, 6), (3, 7); even lane (0, 4), (1, 5)
            w[0] = odd ? r0 : vx, w[1] = odd ? vz : r0, w[2] = odd ? r1 : vy, w[3] = odd ? vw : r1;
            const int ch = i >> 1;   // 16-byte chunk of the K-major row: K block ch / 8, chunk ch % 8
            const uint32_t off = (uint32_t)((ch >> 3) * kBBlock + n * 128 + (((ch & 7) ^ (n & 7)) << 4) + (odd ? 8 : 0));
#pragma unroll
            for (int t = 0; t < TERMS; ++t) {
                const uint32_t lo = narrow2<false>(w[0], w[1]), hi = narrow2<false>(w[2], w[3]);
                *reinterpret_cast<uint2 *>(sB + t * kBTerm + off) = make_uint2(lo, hi);
                if (t + 1 < TERMS) {   // what the fp16 term left behind (exact in fp32)
                    const float2 a = widen2<false>(lo), b = widen2<false>(hi);
                    w[0] -= a.x, w[1] -= a.y, w[2] -= b.x, w[3] -= b.y;
                }
            }
        }
    }
}

}  // namespace

struct UmmaDecode256DenseParams {
    GemmParams g;
    int64_t rpl;        // rows per lambda segment (N when there is one lambda row)
    int64_t n_seg;      // segments
    int64_t n_full;     // segments of exactly rpl rows, covered by the main output map; a shorter last one uses the tail map
};

struct UmmaDecode256DenseMaps {
    CUtensorMap packed;       // [N, 128] bytes, box 128 rows, 128-byte swizzle
    CUtensorMap out, tail;    // output, boxes of 64 columns x 32 rows (128-byte swizzle)
};

template <bool BF16OUT>
__global__ void __launch_bounds__(kThreads, 1)
    kvq_decode_umma_d256_dense_kernel(const __grid_constant__ UmmaDecode256DenseParams prm, const __grid_constant__ UmmaDecode256DenseMaps maps)
{
    using C = Cfg<BF16OUT>;
    constexpr int kATerms = BF16OUT ? 2 : 1;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sB = smem;
    unsigned char *sIn = sB + C::kBTerms * kBTerm;
    unsigned char *sOut = sIn + kInStages * kInBytes;
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(sOut + 8 * kOutWarpBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int half = blockIdx.x & 1;            // which 128 output columns this CTA computes
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kInStages; ++s) {
            mbar_init(smem_u32(&ctrl->in_full[s]), 1);
            mbar_init(smem_u32(&ctrl->in_empty[s]), 4);
        }
        for (int s = 0; s < kAStages; ++s) {
            mbar_init(smem_u32(&ctrl->a_full[s]), 4);
            mbar_init(smem_u32(&ctrl->a_empty[0][s]), 1);
            mbar_init(smem_u32(&ctrl->a_empty[1][s]), 1);
        }
        for (int s = 0; s < kAccStages; ++s) {
            mbar_init(smem_u32(&ctrl->acc_full[s]), 1);
            mbar_init(smem_u32(&ctrl->acc_empty[s]), 4);
        }
        mbar_init(smem_u32(&ctrl->b_first), 16);
        ctrl->abort = 0u;
        ctrl->any_wide = 0u;
        ctrl->b_epoch = 0u;
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);

    // ---- tiles: lambda segments of rpl rows, cut into tiles of 128 rows; a contiguous range of tiles per CTA pair
    const int64_t N = prm.g.N, rpl = prm.rpl;
    const TileShare share(prm.n_seg, rpl, (unsigned)pair, (unsigned)n_pairs);
    const int64_t tps = share.tps, tile_begin = share.begin;
    const int n_my = share.n;
    const int64_t seg_first = n_my > 0 ? tile_begin / tps : 0;
    auto lambda_row = [&](int64_t seg) -> const float * { return prm.g.lambda + prm.g.lambda_index(seg) * kD; };

    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    volatile uint32_t *abort_flag = &ctrl->abort;
    uint32_t *status = prm.g.status;

    // ---- B for the first tile's lambda row: the sixteen dequant and epilogue warps build eight rows each
    if (n_my > 0 && warp >= 2) {
        const RecipLambda<kD> rl(lambda_row(seg_first), lane);
        if (rl.wide) ctrl->any_wide = 1u;
        build_b_rows<C::kBTerms>(sB, prm.g.b0, rl, half, (warp - 2) * 8, (warp - 1) * 8, lane);
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
                ok = wait_or_abort(smem_u32(&ctrl->in_empty[s]), ((uint32_t)(j / kInStages) & 1u) ^ 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT);
                if (!ok) break;
                const int64_t row0 = cur.seg * rpl + cur.row_in_segment();
                const uint32_t bar = smem_u32(&ctrl->in_full[s]);
                mbar_arrive_expect_tx(bar, kInBytes);
                tma_load_2d(smem_u32(sIn + s * kInBytes), &maps.packed, 0, (int)row0, bar);
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
            const uint64_t b_desc = smem_desc_sw128(smem_u32(sB));
            const uint32_t b_lo = (uint32_t)b_desc, b_hi = (uint32_t)(b_desc >> 32);
            int n_mma = n_my;
            if (n_my > 0 && !wait_or_abort(smem_u32(&ctrl->b_first), 0u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) n_mma = 0;
            bool ok = true;
            TileCursor cur(tile_begin, tps);
            for (int j = 0; j < n_mma && ok; ++j, cur.advance(1)) {
                const int sc = j % kAccStages;
                // A new lambda row: a dequant group will overwrite B once every MMA issued so far has read the old one.  This
                // thread waits for the previous tile's accumulator barrier itself (it is at most one phase behind: the stage
                // was free when that tile was issued) and publishes a count; a counter, unlike a parity, cannot be misread
                // by a group that skipped a rebuild.  The tensor core drains once per lambda row.
                if (j > 0 && cur.first_of_segment()) {
                    if (!wait_or_abort(smem_u32(&ctrl->acc_full[(j - 1) % kAccStages]), (uint32_t)((j - 1) / kAccStages) & 1u, abort_flag,
                                       status, KVQ_DEV_MMA_TIMEOUT))
                        break;
                    ctrl->b_epoch = (uint32_t)(cur.seg - seg_first);
                    __threadfence_block();
                }
                if (!wait_or_abort(smem_u32(&ctrl->acc_empty[sc]), ((uint32_t)(j / kAccStages) & 1u) ^ 1u, abort_flag, status,
                                   KVQ_DEV_SLOT_TIMEOUT))
                    break;
                const uint32_t d_tmem = tmem_base + (uint32_t)sc * kHalfN;
#pragma unroll
                for (int kh = 0; kh < 2; ++kh) {   // K halves arrive one after the other
                    const int u = 2 * j + kh, sa = u % kAStages;
                    if (!wait_or_abort(smem_u32(&ctrl->a_full[sa]), (uint32_t)(u / kAStages) & 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_tmem = tmem_base + kACol0 + (uint32_t)sa * 128u;
                    // terms: a_hi W_hi (, a_lo W_hi, a_hi W_lo)
#pragma unroll
                    for (int t = 0; t < (BF16OUT ? 3 : 1); ++t) {
                        const uint32_t a_base = a_tmem + (t == 1 ? 64u : 0u);
                        const uint32_t b_term = (t == 2 ? (uint32_t)(kBTerm >> 4) : 0u);
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            // (bytes >> 4) of K-step 8 kh + ks: K block 2 kh + ks / 4
                            const uint32_t koff = (uint32_t)(2 * kh + (ks >> 2)) * (kBBlock >> 4) + (uint32_t)(ks & 3) * 2u;
                            const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + b_term + koff);
                            if (kh > 0 || t > 0 || ks > 0) umma_f16_ts<true>(d_tmem, a_base + (uint32_t)ks * 8u, bd, kIdesc);
                            else umma_f16_ts<false>(d_tmem, a_base, bd, kIdesc);
                        }
                    }
                    umma_commit(smem_u32(&ctrl->a_empty[j & 1][sa]));   // tile j belongs to dequant group j & 1
                }
                if (ok) umma_commit(smem_u32(&ctrl->acc_full[sc]));
            }
        }
    } else if (warp < 10) {
        // =========================== dequant: packed codes -> A in tensor memory ===========================
        const int grp = (warp - 2) >> 2;        // this group takes tiles grp, grp + 2, ...
        const int q = warp & 3;                 // tensor-memory lane quarter this warp may touch
        const int r = q * 32 + lane;            // tile row and tensor-memory lane of this thread
        const uint4 *scales = static_cast<const uint4 *>(prm.g.scales);   // 8 fp16 scales per row
        int64_t cached_seg = n_my > 0 ? seg_first : -1;   // B holds this row's table (built above)
        float rho = RecipLambda<kD>(lambda_row(seg_first), lane).rho;

        TileCursor cur(tile_begin + grp, tps), ahead(tile_begin + grp, tps);
        auto fetch_scales = [&](int j) -> uint4 {
            if (j >= n_my) return make_uint4(0u, 0u, 0u, 0u);
            const int64_t row = ahead.seg * rpl + ahead.row_in_segment() + r;
            if (row >= N) return make_uint4(0u, 0u, 0u, 0u);
            if (prm.g.per_vector) {   // one scale per vector: the same value in every group's slot
                const uint32_t s1 = (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(prm.g.scales) + row);
                const uint32_t s2 = s1 | (s1 << 16);
                return make_uint4(s2, s2, s2, s2);
            }
            return __ldg(scales + row);
        };
        uint4 sc_next = fetch_scales(grp);
        bool ok = true;
        for (int j = grp; j < n_my && ok; j += 2, cur.advance(2)) {
            const uint4 sc4 = sc_next;
            const uint32_t sc[4] = {sc4.x, sc4.y, sc4.z, sc4.w};
            ahead.advance(2);
            sc_next = fetch_scales(j + 2);
            const int64_t seg = cur.seg;

            // ---- a new lambda row: this group needs its rho; the group that meets the row's first tile rebuilds B
            if (seg != cached_seg) {
                const RecipLambda<kD> rl(lambda_row(seg), lane);
                if (rl.wide) ctrl->any_wide = 1u;
                rho = rl.rho;
                if (cur.first_of_segment()) {
                    // every MMA issued so far must have read B: the mma thread says so by raising b_epoch to this row's index
                    {
                        const uint32_t need = (uint32_t)(seg - seg_first);
                        bool freed = false;
                        for (uint32_t it = 0; it < (1u << 22); ++it) {
                            if (ctrl->b_epoch >= need) {
                                freed = true;
                                break;
                            }
                            if (*abort_flag) break;
                            __nanosleep(64);
                        }
                        if (!freed) {
                            if (!*abort_flag) {
                                *abort_flag = 1u;
                                atomicOr(status, KVQ_DEV_MMA_TIMEOUT);
                            }
                            break;
                        }
                    }
                    build_b_rows<C::kBTerms>(sB, prm.g.b0, rl, half, q * 32, q * 32 + 32, lane);
                    fence_proxy_async();   // B is read by the tensor core through the async proxy
                }
                cached_seg = seg;
            }

            // ---- this tile's packed rows have landed
            const int s = j % kInStages;
            if (!wait_or_abort(smem_u32(&ctrl->in_full[s]), (uint32_t)(j / kInStages) & 1u, abort_flag, status, KVQ_DEV_LOAD_TIMEOUT)) break;
            uint4 pk[kG];
            {
                const unsigned char *row = sIn + s * kInBytes + r * 128;
#pragma unroll
                for (int c = 0; c < kG; ++c) pk[c] = *reinterpret_cast<const uint4 *>(row + ((c ^ (r & 7)) << 4));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->in_empty[s]));   // the values are in registers

            const __half2 h1032 = __float2half2_rn(1032.0f);
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {   // K half kh: groups 4 kh .. 4 kh + 3
                const int u = 2 * j + kh, sa = u % kAStages;
                // The stage was last used by unit u - 2, a K half of the other group's tile j - 1.  Each (group, stage)
                // pair has a barrier of its own, so that this group sees its phases one by one: a parity wait cannot
                // tell a phase from the one two before it.
                if (j >= 1 && !wait_or_abort(smem_u32(&ctrl->a_empty[(j - 1) & 1][sa]), (uint32_t)((u - 2) / 4) & 1u, abort_flag, status,
                                             KVQ_DEV_MMA_TIMEOUT)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t a_row = tmem_base + ((uint32_t)(q * 32) << 16) + kACol0 + (uint32_t)sa * 128u;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    const int c = 4 * kh + cc;   // group: 32 codes, 16 tensor-memory columns
                    const float sig = __half2float(__ushort_as_half((unsigned short)((sc[c >> 1] >> (16 * (c & 1))) & 0xFFFFu)));
                    const float sr = sig * rho;
                const __half2 s2 = __float2half2_rn(sr);
                // the A operand q sigma rho is fp16: it overflows beyond 7 sr = 65504 and loses bits once sr is subnormal
                if (sr != 0.0f && (sr > 9357.0f || sr < 6.1035156e-5f)) ctrl->any_wide = 1u;   // the tile is redone in fp32 at the end
                    const uint32_t words[4] = {pk[c].x, pk[c].y, pk[c].z, pk[c].w};
                    uint32_t a_hi[16], a_lo[16];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t w = words[i] ^ 0x88888888u;   // nibbles now hold q + 8
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint32_t m = lop3_and_or(w >> (4 * e), 0x000F000Fu, 0x64006400u);   // {1024 + n_e, 1024 + n_{e+4}}
                            const __half2 qq = __hsub2(*reinterpret_cast<const __half2 *>(&m), h1032);   // exact codes
                            const __half2 hi = __hmul2(qq, s2);                                          // one rounding
                            a_hi[4 * i + e] = *reinterpret_cast<const uint32_t *>(&hi);
                            if constexpr (kATerms == 2) {
                                const __half2 lo = __hfma2(qq, s2, __hneg2(hi));   // q s - hi: exact, the product has 15 bits
                                a_lo[4 * i + e] = *reinterpret_cast<const uint32_t *>(&lo);
                            }
                        }
                    }
                    tmem_st16(a_row + 16u * (uint32_t)cc, a_hi);
                    if constexpr (kATerms == 2) tmem_st16(a_row + 64u + 16u * (uint32_t)cc, a_lo);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->a_full[sa]));
            }
        }
    } else {
        // =========================== epilogue: accumulator -> 16-bit -> TMA store ===========================
        const int grp = (warp - 10) >> 2;
        const int q = warp & 3;
        unsigned char *stg = sOut + (warp - 10) * kOutWarpBytes;   // one [32 rows][128 B] box
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        TileCursor cur(tile_begin + grp, tps);
        for (int j = grp; j < n_my; j += 2, cur.advance(2)) {
            const int sc = j % kAccStages;
            if (!wait_or_abort(smem_u32(&ctrl->acc_full[sc]), (uint32_t)(j / kAccStages) & 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT)) break;
            tc_fence_after();
            const int64_t seg = cur.seg;
            const int row_in_seg = (int)cur.row_in_segment() + q * 32;
            const bool tail = seg >= prm.n_full;
            const CUtensorMap *tm = tail ? &maps.tail : &maps.out;
            const int segc = tail ? 0 : (int)seg;
#pragma unroll
            for (int b = 0; b < 2; ++b) {   // two boxes of 64 columns through the same staging tile
                if (lane == 0) bulk_wait_read_all();   // the previous store has read the staging tile
                __syncwarp();
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    uint32_t v[32];
                    tmem_ld32(lane_addr + (uint32_t)sc * kHalfN + (uint32_t)(2 * b + cc) * 32u, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        uint4 o;
                        o.x = narrow2<BF16OUT>(__uint_as_float(v[8 * k]), __uint_as_float(v[8 * k + 1]));
                        o.y = narrow2<BF16OUT>(__uint_as_float(v[8 * k + 2]), __uint_as_float(v[8 * k + 3]));
                        o.z = narrow2<BF16OUT>(__uint_as_float(v[8 * k + 4]), __uint_as_float(v[8 * k + 5]));
                        o.w = narrow2<BF16OUT>(__uint_as_float(v[8 * k + 6]), __uint_as_float(v[8 * k + 7]));
                        const int chunk = cc * 4 + k;
                        *reinterpret_cast<uint4 *>(stg + lane * 128 + ((chunk ^ (lane & 7)) << 4)) = o;
                    }
                }
                if (b == 1) tc_fence_before();
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    if (b == 1) mbar_arrive(smem_u32(&ctrl->acc_empty[sc]));
                    tma_store_3d(tm, half * kHalfN + 64 * b, row_in_seg, segc, smem_u32(stg));
                    bulk_commit();
                }
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
    // ---- tiles of a lambda row too wide for the fp16 B operand, or with a scale outside the A operand's range: this CTA's
    // ---- output columns decoded again in fp32
    if (ctrl->any_wide && !*abort_flag)
        redo_tiles_fp32<kD, BF16OUT, 4, kTile, kHalfN, true>(prm.g, tile_begin, n_my, tps, rpl, reinterpret_cast<float *>(smem), half * kHalfN);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
namespace {

template <bool BF16OUT>
cudaError_t launch(int64_t N, const GemmParams &g, cudaStream_t stream)
{
    using C = Cfg<BF16OUT>;
    static DeviceSlots slots;
    int dev = 0;
    cudaError_t e = current_device_slot(&dev);
    if (e != cudaSuccess) return e;
    int &sms = slots.sms[dev];
    if (sms == 0) {
        int n = 0;
        if ((e = cudaFuncSetAttribute(kvq_decode_umma_d256_dense_kernel<BF16OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        sms = n;
    }
    if (!tensor_map_encode_fn()) return cudaErrorNotSupported;
    if (N == 0) return cudaSuccess;   // kvq_plan_prepare: the launch attributes are set, there is nothing to run
    if (N >= (int64_t)1 << 31) return cudaErrorInvalidValue;   // tensor-map coordinates are 32-bit

    UmmaDecode256DenseParams prm;
    prm.g = g;
    prm.rpl = g.n_lambda == 1 ? N : g.rows_per_lambda;
    prm.n_seg = (N + prm.rpl - 1) / prm.rpl;
    prm.n_full = N / prm.rpl;

    UmmaDecode256DenseMaps maps;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)(kD / 2), (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)(kD / 2)};
        const cuuint32_t box[2] = {(cuuint32_t)(kD / 2), (cuuint32_t)kTile};
        if (!make_tensor_map(&maps.packed, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, g.packed, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
            return cudaErrorInvalidValue;
    }
    auto out_map = [&](CUtensorMap *tm, void *base, int64_t rows, int64_t segs) -> bool {
        const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)rows, (cuuint64_t)segs};
        const cuuint64_t strides[2] = {(cuuint64_t)(2 * kD), (cuuint64_t)(2 * kD) * (cuuint64_t)rows};
        const cuuint32_t box[3] = {64u, 32u, 1u};
        return make_tensor_map(tm, BF16OUT ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base, dims, strides, box,
                               CU_TENSOR_MAP_SWIZZLE_128B);
    };
    const int64_t tail_rows = N - prm.n_full * prm.rpl;
    unsigned char *tail_base = static_cast<unsigned char *>(g.out) + (size_t)prm.n_full * prm.rpl * (2 * kD);
    if (prm.n_full > 0 && !out_map(&maps.out, g.out, prm.rpl, prm.n_full)) return cudaErrorInvalidValue;
    if (tail_rows > 0 && !out_map(&maps.tail, tail_base, tail_rows, 1)) return cudaErrorInvalidValue;
    if (tail_rows == 0) maps.tail = maps.out;
    if (prm.n_full == 0) maps.out = maps.tail;

    const int64_t tiles = prm.n_seg * ((prm.rpl + kTile - 1) / kTile);
    const int64_t pairs = tiles < sms / 2 ? tiles : sms / 2;
    kvq_decode_umma_d256_dense_kernel<BF16OUT><<<(int)(2 * pairs), kThreads, C::kSmemBytes, stream>>>(prm, maps);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t umma_decode_d256_dense(bool bf16, int64_t N, const GemmParams &g, cudaStream_t stream)
{
    return bf16 ? launch<true>(N, g, stream) : launch<false>(N, g, stream);
}

}  // namespace kvq

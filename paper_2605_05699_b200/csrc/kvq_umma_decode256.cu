// Warp-specialised tcgen05 DFT-as-GEMM decode kernel of libkvq (sm_100a) for D = 256, fp16 or bf16 output.
//
// Same contraction as kvq_umma_decode.cu, x^ = diag(s) M^T diag(1 / max(lambda, 1e-6)) (q (.) sigma) (Sec. 3.1,
// Sec. 5.1 item 1), with two changes that D = 256 forces:
//
//   * One radix-2 step of the transform is taken out of the GEMM.  Every row of M is cos or sin of 2 pi k n / D,
//     so moving n by D / 2 multiplies the row by (-1)^k, and in the packing of Eq. 2 the parity of k is the parity
//     of the channel c.  With E_n the sum over the even channels and O_n the sum over the odd ones (n < 128),
//         x^_n = s_n (E_n + O_n),      x^_{n+128} = s_{n+128} (E_n - O_n) = (s_n s_{n+128}) s_n (E_n - O_n).
//     E and O are two 128 x 128 x 128 GEMMs instead of one 128 x 256 x 256: half the tensor-core work, and a B
//     operand (64 KB per fp16 term) that fits one CTA's shared memory even when it is split for precision.  The
//     half2 nibble trick already delivers the codes in pairs (c, c + 4) of equal parity, so routing them to the
//     two A operands costs nothing; the +- and the signs are a few instructions per output in the epilogue.
//   * bf16 output has a rounding step 8x coarser than fp16, and a result that is off by 1e-4 of the vector's rms
//     already lands on the other side of enough rounding boundaries to miss the 1e-3 tolerance.  So for bf16 both
//     operands are carried in two fp16 terms: a = q sigma rho has 15 significant bits and splits exactly into
//     a_hi + a_lo (one half2 FMA), W' = W_hi + W_lo, and a_hi W_hi + a_lo W_hi + a_hi W_lo accumulates in fp32
//     (the a_lo W_lo term is below 1e-7).  fp16 output needs one term.
//
//   warp 0        producer   one TMA tensor load per tile: 128 packed rows x 128 B, 128-byte swizzle, 4 stages (2 for bf16);
//                            byte codes (template BITS = 8): rows of 256 B as two such boxes, 2 stages (1 for bf16)
//   warps 2-9     dequant    two groups of four warps, thread = row, both on every tile: group 0 turns the even
//                            channels of the row's packed words into the A operand of the E GEMM, group 1 the
//                            odd ones into that of the O GEMM (tensor memory; two stages each for fp16 output,
//                            one with a_lo beside a_hi for bf16).  Each group also owns the B operand of its
//                            GEMM and rebuilds it when the lambda row changes, behind its own barriers.
//   warp 1        mma        per tile: E GEMM into accumulator columns 0-127, O GEMM into 128-255 (8 K-steps per
//                            term each, A from tensor memory, B from shared memory)
//   warps 10-17   epilogue   all eight warps on every tile (the accumulator has one stage): thread = (row, 64 of the
//                            128 column pairs); E + O and E - O, sign, 16-bit rounding, 64-byte-swizzled staging,
//                            TMA tensor stores of 32 x 32 boxes; the accumulator is released as soon as the last
//                            values are in registers
//
// Every wait is bounded: on a time-out the role records the reason in the status word, raises the CTA's abort
// flag and leaves its loop; the CTA then frees its tensor memory and returns.
#include "kvq_decode_fp32.cuh"
#include "kvq_internal.h"
#include "kvq_umma.cuh"

namespace kvq {

namespace {

constexpr int kD = 256;
constexpr int kG = kD / 32;
constexpr int kTile = 128;       // vectors per tile = MMA M
constexpr int kHalf = 128;       // outputs n < 128 per GEMM = MMA N; also K of each GEMM (channels of one parity)
constexpr int kThreads = 576;    // producer, mma, 2 x 4 dequant, 8 epilogue warps
constexpr int kMaxInStages = 4;
constexpr int kBBlock = kHalf * 128;                   // one K block of 64: 128 rows x 128 B
constexpr int kBPart = 2 * kBBlock;                    // 32 KB: one parity of one term, K = 128
constexpr int kOutWarpBytes = 2 * 2 * 32 * 64;         // per epilogue warp: two chunks x two [32 rows][64 B] boxes
constexpr int kCtrlBytes = 512;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kACol0 = 256;                       // accumulator E at 0, O at 128; A of parity p at 256 + 128 p (hi, then lo)
constexpr uint32_t kIdesc = umma_idesc_m128(kHalf, false);

// BITS = 8: byte codes (Sec. 3.2 step 4's int8 output).  A packed row is then 256 B, loaded as two boxes of 128 B.
template <bool BF16OUT, int BITS = 4>
struct Cfg {
    static constexpr int kInRow = kD * BITS / 8;       // bytes of a packed row
    static constexpr int kInBytes = kTile * kInRow;    // 16 KB (32 KB for byte codes)
    static constexpr int kTerms = BF16OUT ? 2 : 1;     // fp16 terms per operand
    static constexpr int kAStages = BF16OUT ? 1 : 2;   // per parity: 128 columns hold a_hi | a_lo, or two stages of a_hi
    static constexpr int kBBytes = kTerms * 2 * kBPart;
    // packed tiles in flight: what the split B and the 64 KB of output staging leave room for (byte codes with bf16 output:
    // one 32 KB tile, reloaded while the MMAs and the epilogue of the tile before run)
    static constexpr int kInStages = BITS == 8 ? (BF16OUT ? 1 : 2) : BF16OUT ? 2 : 4;
    // per-row output scales of the tiles between a dequant group and the epilogue: as many slots as a group can run ahead
    static constexpr int kScaleSlots = 2 * kAStages;
    static constexpr int kScaleBytes = kScaleSlots * kTile * (int)sizeof(float);
    static constexpr int kSmemBytes = kBBytes + kInStages * kInBytes + 8 * kOutWarpBytes + kCtrlBytes + kScaleBytes + 1024;
    static_assert(kSmemBytes <= 232448, "shared memory over the per-CTA limit");
};

struct Ctrl {
    uint64_t in_full[kMaxInStages], in_empty[kMaxInStages];
    uint64_t a_full[2][2], a_empty[2][2];   // [parity][stage]
    uint64_t acc_full, acc_empty;
    uint64_t b_first;
    uint32_t tmem_base;
    volatile uint32_t abort;
    volatile uint32_t any_wide;   // some lambda row of this CTA's tiles is too wide for the fp16 B operand: redone in fp32 at the end
    uint32_t pad;
    uint4 flip[16];   // sign-bit masks of s_n s_{n+128} for the output pairs (n, n + 1), n = 0, 2, .. 126
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

// Rows [n0, n1) (outputs n < 128) of the B operand of parity p (0: E GEMM, even channels; 1: O GEMM), by one warp.
// The table row b0[n][c] = s_n M[c][n] is used as it is: the accumulators then hold s_n E_n and s_n O_n.  Lanes 2w and 2w + 1 hold
// channels 8w .. 8w + 7; the K order inside a word is the one the nibble trick produces, pairs (c, c + 4): the even
// lane assembles the pair (8w + p, 8w + p + 4), the odd lane (8w + p + 2, 8w + p + 6), each from one value of its
// own and one of its neighbour's.  Terms: fp16(W'), then what that left behind.
template <int TERMS>
__device__ __forceinline__ void build_b_rows(unsigned char *sB, const float *__restrict__ b0, const RecipLambda<kD> &rl, int p, int n0, int n1, int lane)
{
    const bool odd = lane & 1;
#pragma unroll 8   // 16 row quads in flight per lane: the build is a chain of L2 round trips, not arithmetic
    for (int n = n0; n < n1; ++n) {
#pragma unroll
        for (int ps = 0; ps < 2; ++ps) {
            const int i = lane + 32 * ps;
            const float4 m = __ldg(reinterpret_cast<const float4 *>(b0 + (size_t)n * kD) + i);
            auto sat = [](float v) { return fminf(fmaxf(v, -65504.0f), 65504.0f); };
            // this lane's two channels of parity p: 4 i + p and 4 i + p + 2
            const float v0 = sat((p ? m.y : m.x) * (p ? rl.r[ps].y : rl.r[ps].x));
            const float v2 = sat((p ? m.w : m.z) * (p ? rl.r[ps].w : rl.r[ps].z));
            // even lane (channels 8w ..): keeps v0 = 8w + p, needs the odd lane's v0 = 8w + p + 4
            // odd lane (channels 8w + 4 ..): keeps v2 = 8w + p + 6, needs the even lane's v2 = 8w + p + 2
            const float got = __shfl_xor_sync(0xFFFFFFFFu, odd ? v0 : v2, 1);
            float w0 = odd ? got : v0, w1 = odd ? v2 : got;
            const int wd = i >> 1;   // word of 8 codes: columns 2 wd (even lane) and 2 wd + 1 (odd lane) of the K-major row
            const int ch = wd >> 1;  // 16-byte chunk: K block ch / 8, chunk ch % 8
            const uint32_t off = (uint32_t)(p * kBPart + (ch >> 3) * kBBlock + n * 128 + (((ch & 7) ^ (n & 7)) << 4) + ((wd & 1) ? 8 : 0) + (odd ? 4 : 0));
#pragma unroll
            for (int t = 0; t < TERMS; ++t) {
                const uint32_t h = narrow2<false>(w0, w1);
                *reinterpret_cast<uint32_t *>(sB + t * (2 * kBPart) + off) = h;
                if (t + 1 < TERMS) {   // what the fp16 term left behind (exact in fp32)
                    const float2 a = widen2<false>(h);
                    w0 -= a.x, w1 -= a.y;
                }
            }
        }
    }
}

}  // namespace

struct UmmaDecode256Params {
    GemmParams g;
    int64_t rpl;        // rows per lambda segment (N when there is one lambda row)
    int64_t n_seg;      // segments
    int64_t n_full;     // segments of exactly rpl rows, covered by the main output map; a shorter last one uses the tail map
    int64_t phys_rows;  // rows of the packed / scales arrays (N, or the whole cache for a cache view)
    uint32_t sign_xor[128];   // word m: bit 15 set if s_{2m} = -1, bit 31 set if s_{2m+1} = -1
};

struct UmmaDecode256Maps {
    CUtensorMap packed;       // [N, 128] bytes, box 128 rows, 128-byte swizzle
    CUtensorMap out, tail;    // output, boxes of 32 columns x 32 rows (64-byte swizzle)
};

template <bool BF16OUT, int BITS>
__global__ void __launch_bounds__(kThreads, 1)
    kvq_decode_umma_d256_kernel(const __grid_constant__ UmmaDecode256Params prm, const __grid_constant__ UmmaDecode256Maps maps)
{
    using C = Cfg<BF16OUT, BITS>;
    constexpr int kTerms = C::kTerms, kInStages = C::kInStages, kInBytes = C::kInBytes;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sB = smem;                           // [term][parity][2 K blocks][128 rows][128 B]
    unsigned char *sIn = sB + C::kBBytes;
    unsigned char *sOut = sIn + kInStages * kInBytes;
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(sOut + 8 * kOutWarpBytes);
    float *row_scale = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(ctrl) + kCtrlBytes);   // [slot][row]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kInStages; ++s) {
            mbar_init(smem_u32(&ctrl->in_full[s]), 1);
            mbar_init(smem_u32(&ctrl->in_empty[s]), 8);   // both dequant groups read every tile
        }
        for (int p = 0; p < 2; ++p)
            for (int st = 0; st < 2; ++st) {
                mbar_init(smem_u32(&ctrl->a_full[p][st]), 4);
                mbar_init(smem_u32(&ctrl->a_empty[p][st]), 1);
            }
        mbar_init(smem_u32(&ctrl->acc_full), 1);
        mbar_init(smem_u32(&ctrl->acc_empty), 8);
        mbar_init(smem_u32(&ctrl->b_first), 16);
        ctrl->abort = 0u;
        ctrl->any_wide = 0u;
        mbar_init_fence();
    }
    if (threadIdx.x >= 32 && threadIdx.x < 96) {   // sign of s_n s_{n+128}: the xor of the two sign bits
        const int m = threadIdx.x - 32;
        reinterpret_cast<uint32_t *>(ctrl->flip)[m] = prm.sign_xor[m] ^ prm.sign_xor[m + 64];
    }
    if (warp == 0) tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);

    // ---- tiles: lambda segments of rpl rows, cut into tiles of 128 rows; a contiguous range of tiles per CTA
    const int64_t N = prm.g.N, rpl = prm.rpl;
    const TileShare share(prm.n_seg, rpl, blockIdx.x, gridDim.x);
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

    // ---- B for the first tile's lambda row: of the sixteen dequant and epilogue warps, eight build the E operand
    // ---- and eight the O operand, sixteen rows each
    // ---- (the dequant warps request their first tile's scales before the build and keep rho from it, so that neither
    // ---- costs a round trip to L2 after it)
    float rho_first = 1.0f;
    uint4 sc_first = make_uint4(0u, 0u, 0u, 0u);
    if (n_my > 0 && warp >= 2) {
        if (warp < 10) {
            const TileCursor first(tile_begin, tps);
            const int64_t row = prm.g.phys_row(first.seg, first.row_in_segment(), rpl) + (warp & 3) * 32 + lane;
            if (row < prm.phys_rows) {
                if (prm.g.per_vector) {
                    const uint32_t s1 = (uint32_t)__ldg(static_cast<const uint16_t *>(prm.g.scales) + row);
                    sc_first = make_uint4(s1 | (s1 << 16), s1 | (s1 << 16), s1 | (s1 << 16), s1 | (s1 << 16));
                } else {
                    sc_first = __ldg(static_cast<const uint4 *>(prm.g.scales) + row);
                }
            }
        }
        const RecipLambda<kD> rl(lambda_row(seg_first), lane);
        rho_first = rl.rho;
        if (rl.wide) ctrl->any_wide = 1u;
        const int bp = ((warp - 2) >> 2) & 1, bw = ((warp - 2) & 3) + 4 * ((warp - 2) >> 3);   // parity, position among its eight
        build_b_rows<kTerms>(sB, prm.g.b0, rl, bp, bw * 16, bw * 16 + 16, lane);
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
                const int64_t row0 = prm.g.phys_row(cur.seg, cur.row_in_segment(), rpl);   // rows past the segment are read and never stored
                const uint32_t bar = smem_u32(&ctrl->in_full[s]);
                mbar_arrive_expect_tx(bar, kInBytes);
                tma_load_2d(smem_u32(sIn + s * kInBytes), &maps.packed, 0, (int)row0, bar);
                if constexpr (BITS == 8) tma_load_2d(smem_u32(sIn + s * kInBytes + kInBytes / 2), &maps.packed, 128, (int)row0, bar);   // bytes 128 .. 255 of the rows
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
            for (int j = 0; j < n_mma && ok; ++j) {
                // the epilogue has taken the previous tile's E and O out of tensor memory
                if (!wait_or_abort(smem_u32(&ctrl->acc_empty), ((uint32_t)j & 1u) ^ 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                const int sa = j % C::kAStages;
#pragma unroll
                for (int p = 0; p < 2; ++p) {   // E GEMM, then O GEMM
                    if (!wait_or_abort(smem_u32(&ctrl->a_full[p][sa]), (uint32_t)(j / C::kAStages) & 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)p * kHalf;
                    const uint32_t a_tmem = tmem_base + kACol0 + (uint32_t)p * 128u + (uint32_t)sa * 64u;
                    // terms: a_hi W_hi (, a_lo W_hi, a_hi W_lo)
#pragma unroll
                    for (int t = 0; t < (BF16OUT ? 3 : 1); ++t) {
                        const uint32_t a_base = a_tmem + (t == 1 ? 64u : 0u);
                        const uint32_t b_part = (uint32_t)((t == 2 ? 2 * kBPart : 0) + p * kBPart) >> 4;
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t koff = (uint32_t)(ks >> 2) * (kBBlock >> 4) + (uint32_t)(ks & 3) * 2u;   // (bytes >> 4) of K-step ks
                            const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + b_part + koff);
                            if (t > 0 || ks > 0) umma_f16_ts<true>(d_tmem, a_base + (uint32_t)ks * 8u, bd, kIdesc);
                            else umma_f16_ts<false>(d_tmem, a_base, bd, kIdesc);
                        }
                    }
                    umma_commit(smem_u32(&ctrl->a_empty[p][sa]));
                }
                if (ok) umma_commit(smem_u32(&ctrl->acc_full));
            }
        }
    } else if (warp < 10) {
        // =========================== dequant: packed codes -> A operands in tensor memory ===========================
        const int p = (warp - 2) >> 2;          // this group's parity: 0 = even channels (E GEMM), 1 = odd channels (O GEMM)
        const int q = warp & 3;                 // tensor-memory lane quarter this warp may touch
        const int r = q * 32 + lane;            // tile row and tensor-memory lane of this thread
        const uint4 *scales = static_cast<const uint4 *>(prm.g.scales);   // 8 fp16 scales per row
        int64_t cached_seg = n_my > 0 ? seg_first : -1;   // B holds this row's table (built above)
        float rho = rho_first;

        TileCursor cur(tile_begin, tps), ahead(tile_begin, tps);
        auto fetch_scales = [&](int j) -> uint4 {
            if (j >= n_my) return make_uint4(0u, 0u, 0u, 0u);
            const int64_t row = prm.g.phys_row(ahead.seg, ahead.row_in_segment(), rpl) + r;
            if (row >= prm.phys_rows) return make_uint4(0u, 0u, 0u, 0u);
            if (prm.g.per_vector) {   // one scale per vector: the same value in every group's slot
                const uint32_t s1 = (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(prm.g.scales) + row);
                const uint32_t s2 = s1 | (s1 << 16);
                return make_uint4(s2, s2, s2, s2);
            }
            return __ldg(scales + row);
        };
        uint4 sc_next = sc_first;   // requested before the first B build
        for (int j = 0; j < n_my; ++j, cur.advance(1)) {
            const uint4 sc4 = sc_next;
            const uint32_t sc[4] = {sc4.x, sc4.y, sc4.z, sc4.w};
            ahead.advance(1);
            sc_next = fetch_scales(j + 1);
            const int64_t seg = cur.seg;
            const int sa = j % C::kAStages;

            // ---- a new lambda row: new rho, and this group rebuilds the B operand of its own GEMM once every MMA of that
            // ---- GEMM issued so far is complete: the previous tile's, on this group's own barriers (it sees every phase)
            if (seg != cached_seg) {
                const RecipLambda<kD> rl(lambda_row(seg), lane);
                if (rl.wide) ctrl->any_wide = 1u;
                rho = rl.rho;
                if (!wait_or_abort(smem_u32(&ctrl->a_empty[p][(j - 1) % C::kAStages]), (uint32_t)((j - 1) / C::kAStages) & 1u, abort_flag,
                                   status, KVQ_DEV_MMA_TIMEOUT))
                    break;
                build_b_rows<kTerms>(sB, prm.g.b0, rl, p, q * 32, q * 32 + 32, lane);
                fence_proxy_async();   // B is read by the tensor core through the async proxy
                cached_seg = seg;
            }

            // ---- this tile's packed rows have landed
            const int s = j % kInStages;
            if (!wait_or_abort(smem_u32(&ctrl->in_full[s]), (uint32_t)(j / kInStages) & 1u, abort_flag, status, KVQ_DEV_LOAD_TIMEOUT)) break;
            uint4 pk[BITS == 4 ? kG : 1];
            const unsigned char *row = sIn + s * kInBytes + r * 128;
            if constexpr (BITS == 4) {
#pragma unroll
                for (int c = 0; c < kG; ++c) pk[c] = *reinterpret_cast<const uint4 *>(row + ((c ^ (r & 7)) << 4));
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->in_empty[s]));   // the values are in registers
            }

            // ---- the operand stage is free again (the MMAs of the tile that used it last are complete)
            if (!wait_or_abort(smem_u32(&ctrl->a_empty[p][sa]), ((uint32_t)(j / C::kAStages) & 1u) ^ 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT))
                break;
            tc_fence_after();
            // ---- the A operand q sigma rho is fp16.  A row whose scales would take it out of fp16's normal range (a very
            // ---- small or very large vector) is carried times a power of two instead, which the epilogue takes out again
            // ---- in fp32; every other row has the factor 1 and costs the epilogue nothing.  Both parity groups see the
            // ---- same scales and take the same factor; group 0 posts it.
            float inv;
            const float pw = operand_rescue<kG>(sc, rho, BITS == 4 ? 9000.0f : 500.0f, inv);   // 7 (127) times this stays inside fp16
            if (p == 0) row_scale[(j % C::kScaleSlots) * kTile + r] = inv;
            const uint32_t a_row = tmem_base + ((uint32_t)(q * 32) << 16) + kACol0 + (uint32_t)p * 128u + (uint32_t)sa * 64u;
            const __half2 h1032 = __float2half2_rn(1032.0f);
#pragma unroll
            for (int c = 0; c < kG; ++c) {   // group c: 16 codes of this parity, 8 tensor-memory columns
                const float sig = __half2float(__ushort_as_half((unsigned short)((sc[c >> 1] >> (16 * (c & 1))) & 0xFFFFu)));
                const __half2 s2 = __float2half2_rn(sig * rho * pw);
                uint32_t a_hi[8], a_lo[8];
                auto put = [&](int k, __half2 qq) {   // K pair k of the group: one rounding, and what it left behind
                    const __half2 hi = __hmul2(qq, s2);
                    a_hi[k] = *reinterpret_cast<const uint32_t *>(&hi);
                    if constexpr (kTerms == 2) {
                        const __half2 lo = __hfma2(qq, s2, __hneg2(hi));   // q s - hi: exact, the product has 15 (byte codes: 18) bits
                        a_lo[k] = *reinterpret_cast<const uint32_t *>(&lo);
                    }
                };
                if constexpr (BITS == 4) {
                    const uint32_t words[4] = {pk[c].x, pk[c].y, pk[c].z, pk[c].w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t w = (words[i] ^ 0x88888888u) >> (4 * p);   // nibbles hold q + 8; parity p starts at nibble p
#pragma unroll
                        for (int t = 0; t < 2; ++t) {
                            // nibbles 2t + p and 2t + p + 4 of the word: channels 8w + 2t + p and + 4, both of parity p
                            const uint32_t m = lop3_and_or(w >> (8 * t), 0x000F000Fu, 0x64006400u);   // {1024 + n, 1024 + n'}
                            put(2 * i + t, __hsub2(*reinterpret_cast<const __half2 *>(&m), h1032));       // exact codes
                        }
                    }
                } else {
                    // group c = bytes 32 c .. 32 c + 31 of the row: two 16-byte chunks of the box that holds this half of the row.
                    // Eight channels 8w .. 8w + 7 are two words; the pairs of parity p are bytes (p, p + 4) and (p + 2, p + 6):
                    // the K order of the B operand.
                    const __half2 h1152 = __float2half2_rn(1152.0f);
                    const unsigned char *half_row = row + (c >> 2) * (kInBytes / 2);
#pragma unroll
                    for (int hc = 0; hc < 2; ++hc) {
                        const uint4 pc = *reinterpret_cast<const uint4 *>(half_row + ((uint32_t)((2 * (c & 3) + hc) ^ (r & 7)) << 4));
                        const uint32_t words[4] = {pc.x ^ 0x80808080u, pc.y ^ 0x80808080u, pc.z ^ 0x80808080u, pc.w ^ 0x80808080u};   // bytes hold q + 128
#pragma unroll
                        for (int i = 0; i < 2; ++i) {   // eight channels: words 2 i and 2 i + 1
#pragma unroll
                            for (int t = 0; t < 2; ++t) {
                                const uint32_t sel = (uint32_t)(p + 2 * t) | ((uint32_t)(4 + p + 2 * t) << 8);   // byte p + 2t of each word, to bytes 0 and 2
                                const uint32_t two = __byte_perm(words[2 * i], words[2 * i + 1], sel);
                                const uint32_t m = lop3_and_or(two, 0x00FF00FFu, 0x64006400u);                  // {1024 + b, 1024 + b'}
                                put(4 * hc + 2 * i + t, __hsub2(*reinterpret_cast<const __half2 *>(&m), h1152));   // exact codes
                            }
                        }
                    }
                }
                tmem_st8(a_row + 8u * (uint32_t)c, a_hi);
                if constexpr (kTerms == 2) tmem_st8(a_row + 64u + 8u * (uint32_t)c, a_lo);
            }
            if constexpr (BITS == 8) {   // the packed rows were read group by group: only now is their stage free
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->in_empty[s]));
            }
            tmem_st_wait();
            tc_fence_before();
            __threadfence_block();   // the row scales, for the epilogue that follows this tile's accumulator
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->a_full[p][sa]));
        }
    } else {
        // =========================== epilogue: E, O -> x^ -> TMA store ===========================
        const int q = warp & 3;
        const int ch = (warp - 10) >> 2;                            // this warp's half of the column pairs: n in [64 ch, 64 ch + 64)
        unsigned char *stg_base = sOut + (warp - 10) * kOutWarpBytes;   // per chunk: two [32 rows][64 B] boxes
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        TileCursor cur(tile_begin, tps);
        for (int j = 0; j < n_my; ++j, cur.advance(1)) {
            if (!wait_or_abort(smem_u32(&ctrl->acc_full), (uint32_t)j & 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT)) break;
            tc_fence_after();
            const int64_t seg = cur.seg;
            const int row_in_seg = (int)cur.row_in_segment() + q * 32;
            const bool tail = seg >= prm.n_full;
            const CUtensorMap *tm = tail ? &maps.tail : &maps.out;
            const int segc = tail ? 0 : (int)seg;
            const float row_inv = row_scale[(j % C::kScaleSlots) * kTile + q * 32 + lane];
            const bool rescale = __any_sync(0xFFFFFFFFu, row_inv != 1.0f);   // rare: a row outside the operand's comfort zone
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {   // 32 column pairs at a time: outputs n0 .. n0 + 31 and 128 + n0 ..
                const int n0 = 64 * ch + 32 * cc;
                unsigned char *stg = stg_base + cc * (2 * 32 * 64);
                uint32_t e[32], o[32];
                tmem_ld32(lane_addr + (uint32_t)n0, e);
                tmem_ld32(lane_addr + (uint32_t)(kHalf + n0), o);
                tmem_ld_wait();
                if (rescale) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        e[i] = __float_as_uint(__uint_as_float(e[i]) * row_inv);
                        o[i] = __float_as_uint(__uint_as_float(o[i]) * row_inv);
                    }
                }
                if (cc == 1) {   // the last values are in registers: hand the accumulator back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctrl->acc_empty));
                }
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the stores of this chunk's boxes one tile ago have read them
                __syncwarp();
#pragma unroll
                for (int k = 0; k < 4; ++k) {   // 16-byte chunk k of each box row: 8 outputs
                    const uint4 fl = ctrl->flip[(n0 >> 3) + k];   // warp-uniform address: a broadcast
                    const uint32_t f[4] = {fl.x, fl.y, fl.z, fl.w};
                    uint32_t lo[4], hi[4];
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        const int i = 8 * k + 2 * v;
                        const float e0 = __uint_as_float(e[i]), e1 = __uint_as_float(e[i + 1]);
                        const float o0 = __uint_as_float(o[i]), o1 = __uint_as_float(o[i + 1]);
                        lo[v] = narrow2<BF16OUT>(e0 + o0, e1 + o1);          // s_n is already in E and O
                        hi[v] = narrow2<BF16OUT>(e0 - o0, e1 - o1) ^ f[v];   // times s_n s_{n+128}
                    }
                    const uint32_t off = (uint32_t)(lane * 64 + ((k ^ ((lane >> 1) & 3)) << 4));   // 64-byte swizzle
                    *reinterpret_cast<uint4 *>(stg + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                    *reinterpret_cast<uint4 *>(stg + 32 * 64 + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                    tma_store_3d(tm, n0, row_in_seg, segc, smem_u32(stg));
                    tma_store_3d(tm, kHalf + n0, row_in_seg, segc, smem_u32(stg + 32 * 64));
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
    // ---- tiles of a lambda row too wide for the fp16 B operand: decoded again in fp32, over what the pipeline stored
    if (ctrl->any_wide && !*abort_flag)
        redo_tiles_fp32<kD, BF16OUT, BITS, kTile>(prm.g, tile_begin, n_my, tps, rpl, reinterpret_cast<float *>(smem));
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
namespace {

template <bool BF16OUT, int BITS>
cudaError_t launch(int64_t N, const GemmParams &g, const uint32_t *sign_xor, cudaStream_t stream)
{
    using C = Cfg<BF16OUT, BITS>;
    static DeviceSlots slots;
    int dev = 0;
    cudaError_t e = current_device_slot(&dev);
    if (e != cudaSuccess) return e;
    int &sms = slots.sms[dev];
    if (sms == 0) {
        int n = 0;
        if ((e = cudaFuncSetAttribute(kvq_decode_umma_d256_kernel<BF16OUT, BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        sms = n;
    }
    if (!tensor_map_encode_fn()) return cudaErrorNotSupported;
    if (N == 0) return cudaSuccess;   // kvq_plan_prepare: the launch attributes are set, there is nothing to run
    if (N >= (int64_t)1 << 31) return cudaErrorInvalidValue;   // tensor-map coordinates are 32-bit

    UmmaDecode256Params prm;
    prm.g = g;
    prm.rpl = g.view.rows ? g.view.rows : g.n_lambda == 1 ? N : g.rows_per_lambda;   // a cache view: one segment per stream
    prm.n_seg = (N + prm.rpl - 1) / prm.rpl;
    prm.n_full = N / prm.rpl;
    prm.phys_rows = g.view.rows ? prm.n_seg * g.view.stride : N;
    if (prm.phys_rows >= (int64_t)1 << 31) return cudaErrorInvalidValue;
    const int64_t seg_stride = g.view.rows ? g.view.stride : prm.rpl;   // rows from one segment's first row to the next's
    unsigned char *out0 = static_cast<unsigned char *>(g.out) + (size_t)(g.view.rows ? g.view.base : 0) * (2 * kD);
    for (int i = 0; i < 128; ++i) prm.sign_xor[i] = sign_xor[i];

    UmmaDecode256Maps maps;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)C::kInRow, (cuuint64_t)prm.phys_rows};
        const cuuint64_t strides[1] = {(cuuint64_t)C::kInRow};
        const cuuint32_t box[2] = {128u, (cuuint32_t)kTile};   // 128 bytes of 128 rows: a whole nibble row, half a byte row
        if (!make_tensor_map(&maps.packed, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, g.packed, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
            return cudaErrorInvalidValue;
    }
    auto out_map = [&](CUtensorMap *tm, void *base, int64_t rows, int64_t segs) -> bool {
        const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)rows, (cuuint64_t)segs};
        const cuuint64_t strides[2] = {(cuuint64_t)(2 * kD), (cuuint64_t)(2 * kD) * (cuuint64_t)(segs > 1 ? seg_stride : rows)};
        const cuuint32_t box[3] = {32u, 32u, 1u};
        return make_tensor_map(tm, BF16OUT ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base, dims, strides, box,
                               CU_TENSOR_MAP_SWIZZLE_64B);
    };
    const int64_t tail_rows = N - prm.n_full * prm.rpl;
    unsigned char *tail_base = out0 + (size_t)prm.n_full * seg_stride * (2 * kD);
    if (prm.n_full > 0 && !out_map(&maps.out, out0, prm.rpl, prm.n_full)) return cudaErrorInvalidValue;
    if (tail_rows > 0 && !out_map(&maps.tail, tail_base, tail_rows, 1)) return cudaErrorInvalidValue;
    if (tail_rows == 0) maps.tail = maps.out;
    if (prm.n_full == 0) maps.out = maps.tail;

    const int64_t tiles = prm.n_seg * ((prm.rpl + kTile - 1) / kTile);
    const int grid = (int)(tiles < sms ? tiles : sms);
    kvq_decode_umma_d256_kernel<BF16OUT, BITS><<<grid, kThreads, C::kSmemBytes, stream>>>(prm, maps);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t umma_decode_d256(bool bf16, int bits, int64_t N, const GemmParams &g, const uint32_t *sign_xor, cudaStream_t stream)
{
    if (bits == 8) return bf16 ? launch<true, 8>(N, g, sign_xor, stream) : launch<false, 8>(N, g, sign_xor, stream);
    return bf16 ? launch<true, 4>(N, g, sign_xor, stream) : launch<false, 4>(N, g, sign_xor, stream);
}

}  // namespace kvq

// Warp-specialised tcgen05 DFT-as-GEMM encode kernel of libkvq (sm_100a): D = 64, 96, 128, 160; fp16 and bf16 input
// (D = 160 with bf16: two x tiles in flight instead of four, and no three-term forms).
//
// The forward path v = lambda (.) M (s (.) x) (Sec. 3.1 Eq. 1-2, Sec. 5.1 item 1) is a dense D x D
// contraction per vector, for any even D: v_c = sum_n W[c, n] x_n with W[c, n] = lambda_c M[c, n] s_n.  The
// codes must agree with an fp64 evaluation on all but 1e-4 of the entries, so W cannot be rounded to 11 bits
// (that leaves 1e-3 of the codes on the wrong side of a rounding).  x is exact in its 16-bit format; W is split into
// two 16-bit terms,
//      fp16 input:  W 2^k = W1 + W2          (two fp16 terms: 22 bits)
//      bf16 input:  W 2^k = W1 + W2          (two bf16 terms: 16 bits; 6e-6 of the codes and 0.2 % of the stored
//                                             scales then differ from the fp64 evaluation, all at rounding ties;
//                                             the calibration pass adds a third term)
// every product x_n W_i[c, n] is exact in fp32, and the terms are summed in fp32: for D <= 128 the two terms are stacked
// along N (one MMA of N = 2 D per K-step fills two halves of the accumulator, which the epilogue adds: an MMA
// instruction costs about 117 cycles whatever N <= 128 it carries and 176 at N = 256, so half the instructions is
// worth more than the flops); D = 160 and the three-term forms accumulate all terms in one accumulator.  A term costs as much energy as the same GEMM in a library (0.6 pJ per flop), and the kernel runs
// at the board's power cap, so a term more is 20 % less throughput.  2^k lifts the small terms clear of fp16's subnormal range; the epilogue undoes it in
// the scale computation, at no cost per element.
//
//   warp 0        producer   one TMA tensor load per K block of 64 elements and tile of 128 vectors (128-byte
//                            swizzle): x lands in shared memory in the tensor core's canonical K-major
//                            layout, several tiles in flight, no thread touches it
//   warp 1        mma        one thread issues D / 16 K-steps (per split term where the terms are not stacked) into
//                            one accumulator stage, then commits once: the epilogue reads it as "accumulator full", the producer as
//                            "x stage free"
//   warps 2-17    epilogue   two sets of eight warps on alternate tiles; thread = (row, half row).  Per group
//                            of 32 channels: tcgen05.ld of the 32 accumulator columns, abs-max, fp16 scale,
//                            round-to-nearest-even codes, nibble pack (Sec. 3.2 steps 3-4, per-group scales
//                            of Sec. 5.6 / 7.1): no shuffle, no shared memory; the codes and scales go
//                            straight to global memory.  The accumulator stage is released as soon as the
//                            values are in registers.  The set that meets the first tile of a new lambda
//                            row rebuilds the B operand (the mma warp waits for it on an mbarrier).
//
//   A [128 vectors, K = D]     x in shared memory (TMA), K-major, 128-byte swizzle, K blocks of 64
//   B [N = D channels, K]      split terms of W 2^k in shared memory, same layout: one region per term, or the
//                              terms stacked as rows [0, D) and [D, 2 D) of every K block (D <= 128, two terms)
//   D [128, D or 2 D]          fp32 accumulator in tensor memory, two to four stages
//
// Every wait on an mbarrier is bounded: on a time-out the role records the reason in the status word,
// raises the CTA's abort flag and leaves its loop; the CTA then frees its tensor memory and returns.
#include "kvq_internal.h"
#include "kvq_umma.cuh"

namespace kvq {

namespace {

constexpr int kTile = 128;                 // vectors per tile = MMA M
constexpr int kGroup = 32;
constexpr int kThreads = 576;              // producer, mma, 16 epilogue warps
constexpr int kEpiWarps = 16;
constexpr int kBlockBytes = kTile * 128;   // one K block of the x tile: 128 rows x 128 B
constexpr int kCtrlBytes = 4608;            // barriers and flags, then the row maxima the two half-row threads trade
constexpr int kSmemLimit = 232448;         // 227 KB of dynamic shared memory per CTA
constexpr uint32_t kTmemCols = 512;
// "Accumulator full" barriers form a ring of four indexed by TILE, whatever the number of accumulator stages: the producer
// takes tile j - kInStages's as "x stage free", and a parity wait only tells a phase from its neighbours, so the barrier it
// waits on must not be able to complete another phase before the producer has loaded tile j.
constexpr int kFullBars = 4;


// THREE: a third bf16 term of W.  The calibration pass takes it (it runs once; its result is compared at 1e-6 of the
// vector norm), and so do byte codes, whose step is 18 times finer than that of 4-bit codes.
template <int D, bool BF16, bool THREE = false>
struct Cfg {
    static_assert(D % 32 == 0 && D >= 64 && D <= 160, "head dim not built");
    static constexpr int G = D / kGroup;
    static constexpr int kSplit = (BF16 && THREE) ? 3 : 2;
    static constexpr int kKSteps = D / 16;
    static constexpr int kKBlocks = (D + 63) / 64;              // K blocks of 64 elements (the last one may be half used)
    static constexpr int kXBytes = kKBlocks * kBlockBytes;      // one x tile
    // Two terms and D <= 128: the terms are STACKED along N, rows [0, D) of a K block the first term's, rows [D, 2 D) the
    // second's, and one MMA of N = 2 D computes x W_hi into accumulator columns [0, D) and x W_lo into [D, 2 D); the
    // epilogue adds the two.  An MMA of M 128, N 128, K 16 costs about 120 cycles here, one of N = 256 about 176 (measured,
    // both operands in shared memory, accumulating into one tile; the nominal rates are 68 and 135): the per-instruction
    // overhead is paid once for both terms, and the x tile is read from shared memory once instead of twice.
    static constexpr bool kStack = kSplit == 2 && D <= 128;
    static constexpr int kNmma = kStack ? 2 * D : D;            // N of one MMA
    static constexpr int kBBlock = kNmma * 128;                 // one K block of B: kNmma rows x 128 B
    static constexpr int kBTerm = kStack ? D * 128 : kKBlocks * kBBlock;   // from one term's row c to the next term's
    static constexpr int kBBytes = kSplit * kKBlocks * D * 128;
    static constexpr int kRoom = (kSmemLimit - 1024 - kCtrlBytes - kBBytes) / kXBytes;
    static constexpr int kInStages = kRoom < 4 ? kRoom : 4;     // x tiles in flight
    static_assert(kInStages >= 2 && kInStages <= kFullBars, "this head dim and input type do not fit shared memory");
    static constexpr int kSmemBytes = kBBytes + kInStages * kXBytes + kCtrlBytes + 1024;
    static constexpr uint32_t kAccStride = kStack ? 2 * D : D <= 128 ? 128 : 160;
    static constexpr int kAccStages = 512 / (int)kAccStride < 4 ? 512 / (int)kAccStride : 4;   // accumulators in tensor memory
    static constexpr uint32_t kIdesc = umma_idesc_m128(kNmma, BF16);
    static constexpr int kGroupsPerPart = (G + 1) / 2;          // groups of the first half row; the second takes the rest
};

struct Ctrl {
    uint64_t in_full[4];
    uint64_t acc_full[kFullBars], acc_empty[4];
    uint64_t b_first, b_ready;
    uint64_t pair[2][4];        // one scale per vector: the two warps that share 32 rows of a set meet here, once per tile
    uint32_t tmem_base;
    volatile uint32_t abort;
    uint32_t pad[2];
    float rowmax[2][2][2][kTile];   // [tile parity within the set][set][half row][row]
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

// 2^k for a lambda row: the power of two that brings max_c lambda_c max|table entry| (sqrt(2 / D) without a rotation) into [2^13, 2^14), so that
// the first split term of W 2^k stays below fp16's maximum and the later ones above its subnormals.
// Every lane of the warp gets the same value.
template <int D>
__device__ __forceinline__ float lift_of(const float *__restrict__ lam, float table_max, int lane)
{
    float mx = lam ? 0.0f : 1.0f;   // no lambda row (calibration): lambda = 1
#pragma unroll
    for (int p = 0; p < (D / 4 + 31) / 32; ++p) {
        const int i = lane + 32 * p;
        if (lam && i < D / 4) {
            const float4 l = __ldg(reinterpret_cast<const float4 *>(lam) + i);
            mx = fmaxf(mx, fmaxf(fmaxf(fabsf(l.x), fabsf(l.y)), fmaxf(fabsf(l.z), fabsf(l.w))));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    mx = fminf(fmaxf(mx * table_max, 1e-30f), 1e30f);   // table_max: largest |entry| of the table
    const int e = (int)((__float_as_uint(mx) >> 23) & 0xFFu) - 127;      // floor(log2 mx)
    return __uint_as_float((uint32_t)(127 + 13 - e) << 23);
}

// Rows [c0, c1) of every split term of the B operand, by one warp: a lane reads four table entries
// e0[c][4 i .. 4 i + 3] (coalesced rows), scales them by lambda_c 2^k, peels off 16-bit terms and writes
// 8 bytes of each term's swizzled row.
// One quad of row c of every split term: the four table entries m scaled by f = lambda_c 2^k, 16-bit terms peeled
// off one after the other, 8 bytes of each term's swizzled row written.
template <int D, bool BF16, bool THREE>
__device__ __forceinline__ void build_b_quad(unsigned char *sB, float4 m, float f, int c, int i)
{
    using C = Cfg<D, BF16, THREE>;
    float w[4] = {m.x * f, m.y * f, m.z * f, m.w * f};
    const int ch = i >> 1;   // 16-byte chunk of the K-major row: K block ch / 8, chunk ch % 8
    const uint32_t off = (uint32_t)((ch >> 3) * C::kBBlock + c * 128 + (((ch & 7) ^ (c & 7)) << 4) + ((i & 1) ? 8 : 0));
#pragma unroll
    for (int t = 0; t < C::kSplit; ++t) {
        const uint32_t lo = narrow2<BF16>(w[0], w[1]), hi = narrow2<BF16>(w[2], w[3]);
        *reinterpret_cast<uint2 *>(sB + t * C::kBTerm + off) = make_uint2(lo, hi);
        if (t + 1 < C::kSplit) {   // what the 16-bit term left behind (exact in fp32)
            const float2 a = widen2<BF16>(lo), b = widen2<BF16>(hi);
            w[0] -= a.x, w[1] -= a.y, w[2] -= b.x, w[3] -= b.y;
        }
    }
}

template <int D, bool BF16, bool THREE>
__device__ __forceinline__ void build_b_rows(unsigned char *sB, const float *__restrict__ e0, const float *__restrict__ lam, float lift,
                                             int c0, int c1, int lane)
{
#pragma unroll 4
    for (int c = c0; c < c1; ++c) {
        const float f = lam ? __ldg(lam + c) * lift : lift;
#pragma unroll
        for (int p = 0; p < (D / 4 + 31) / 32; ++p) {
            const int i = lane + 32 * p;
            if (i < D / 4) build_b_quad<D, BF16, THREE>(sB, __ldg(reinterpret_cast<const float4 *>(e0 + (size_t)c * D) + i), f, c, i);
        }
    }
}

// The first build of a CTA: a warp's D / 16 table rows and their lambda entries are requested at kernel entry, all at
// once, and turned into B rows once the lift is known: one round trip to L2 instead of one per batch of rows.
template <int D, bool BF16, bool THREE>
struct FirstRows {
    static constexpr int kRows = D / 16, kPasses = (D / 4 + 31) / 32;
    float4 m[kRows][kPasses];
    float lam_c[kRows];
    __device__ __forceinline__ void load(const float *__restrict__ e0, const float *__restrict__ lam, int c0, int lane)
    {
#pragma unroll
        for (int k = 0; k < kRows; ++k) {
#pragma unroll
            for (int p = 0; p < kPasses; ++p) {
                const int i = lane + 32 * p;
                m[k][p] = i < D / 4 ? __ldg(reinterpret_cast<const float4 *>(e0 + (size_t)(c0 + k) * D) + i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            }
            lam_c[k] = lam ? __ldg(lam + c0 + k) : 1.0f;
        }
    }
    __device__ __forceinline__ void build(unsigned char *sB, float lift, int c0, int lane) const
    {
#pragma unroll
        for (int k = 0; k < kRows; ++k)
#pragma unroll
            for (int p = 0; p < kPasses; ++p) {
                const int i = lane + 32 * p;
                if (i < D / 4) build_b_quad<D, BF16, THREE>(sB, m[k][p], lam_c[k] * lift, c0 + k, i);
            }
    }
};

// The mma role's wait for the CTA's first B operand: the one wait whose limit the host may shorten
// (kvq_plan_set_wait_limit), because the waiting thread has issued nothing yet and can leave at once.  A shortened limit
// counts looks at the barrier that do not block, so that "one poll" is over before the operand can possibly be there.
__device__ __forceinline__ bool wait_first_operand(uint32_t bar, volatile uint32_t *abort_flag, uint32_t *status, uint32_t limit)
{
    for (uint32_t it = 0; it < limit; ++it)
        if (mbar_test_wait(bar, 0u)) return true;
    *abort_flag = 1u;
    atomicOr(status, (uint32_t)KVQ_DEV_SLOT_TIMEOUT);
    return false;
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
    RowMap out_map;        // output row of input row r
    float table_max;       // largest |entry| of e0
    int bits;              // 4: nibble pairs; 8: one two's-complement byte per code, scale = absmax / 127
    uint32_t *status;
    uint32_t *amax_bits;        // calibration only: [D] running column maxima as fp32 bit patterns (start at zero)
    uint32_t first_wait_polls;  // polls the mma role gives the first B build before it gives up (kvq_plan_set_wait_limit)
};

// PERVEC: one scale per vector (group = D; Sec. 3.2 step 3, Sec. 4.1) instead of one per 32 channels.
// WIDE: byte codes from bf16 input (three terms of W).
template <int D, bool BF16, bool CALIB, bool PERVEC, bool WIDE>
__global__ void __launch_bounds__(kThreads, 1)
    kvq_encode_umma_kernel(const __grid_constant__ UmmaEncodeParams prm, const __grid_constant__ CUtensorMap tm_x)
{
    using C = Cfg<D, BF16, CALIB || WIDE>;
    constexpr int G = C::G, kInStages = C::kInStages, kAccStages = C::kAccStages;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sB = smem;                                   // kSplit terms
    unsigned char *sIn = sB + C::kBBytes;                       // kInStages x tiles
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(sIn + kInStages * C::kXBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kInStages; ++s) mbar_init(smem_u32(&ctrl->in_full[s]), 1);
        for (int s = 0; s < kFullBars; ++s) mbar_init(smem_u32(&ctrl->acc_full[s]), 1);
        for (int s = 0; s < kAccStages; ++s) mbar_init(smem_u32(&ctrl->acc_empty[s]), kEpiWarps / 2);
        mbar_init(smem_u32(&ctrl->b_first), kEpiWarps);       // first B: all epilogue warps build it
        mbar_init(smem_u32(&ctrl->b_ready), kEpiWarps / 2);   // later rebuilds: the set that owns the tile
        for (int s = 0; s < 2; ++s)
            for (int qq = 0; qq < 4; ++qq) mbar_init(smem_u32(&ctrl->pair[s][qq]), 2);
        ctrl->abort = 0u;
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);

    // ---- tiles: lambda segments of rpl rows, cut into tiles of 128 rows; a contiguous range per CTA
    const int64_t N = prm.N, rpl = prm.rpl;
    const TileShare share(prm.n_seg, rpl, blockIdx.x, gridDim.x);
    const int64_t tps = share.tps, tile_begin = share.begin;
    const int n_my = share.n;

    // ---- B for the CTA's first lambda row: D / 16 rows per epilogue warp.  Table rows and lambda are requested before
    // ---- the set-up barrier, so that their latency runs under it and under the first x loads.
    float first_lift = 1.0f;
    int64_t first_seg = -1;
    if (n_my > 0 && warp >= 2) {
        first_seg = tile_begin / tps;
        const float *lam = CALIB ? nullptr : prm.lambda + (prm.n_lambda == 1 ? 0 : first_seg) * D;
        FirstRows<D, BF16, CALIB || WIDE> rows;
        rows.load(prm.e0, lam, (warp - 2) * (D / 16), lane);
        first_lift = lift_of<D>(lam, prm.table_max, lane);
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        rows.build(sB, first_lift, (warp - 2) * (D / 16), lane);
        fence_proxy_async();   // B is read by the tensor core through the async proxy
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->b_first));
    } else {
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    const uint32_t tmem_base = ctrl->tmem_base;
    volatile uint32_t *abort_flag = &ctrl->abort;
    uint32_t *status = prm.status;
    int issued = 0;   // producer thread: x tiles whose loads have been issued

    if (warp == 0) {
        // =========================== producer ===========================
        if (lane == 0) {
            bool ok = true;
            TileCursor cur(tile_begin, tps);
            for (int j = 0; j < n_my; ++j, cur.advance(1)) {
                const int s = j % kInStages;
                // The x stage is free once the MMAs of the tile that used it last are complete: that tile's accumulator
                // barrier.  (Its next phase is tile j's own, which cannot complete before this load: the parity test holds.)
                if (j >= kInStages) {
                    const int jp = j - kInStages;
                    ok = wait_or_abort(smem_u32(&ctrl->acc_full[jp % kFullBars]), (uint32_t)(jp / kFullBars) & 1u, abort_flag, status,
                                       KVQ_DEV_SLOT_TIMEOUT);
                }
                if (!ok) break;
                const int64_t row0 = cur.seg * rpl + cur.row_in_segment();
                const uint32_t bar = smem_u32(&ctrl->in_full[s]);
                mbar_arrive_expect_tx(bar, C::kXBytes);
#pragma unroll
                for (int kb = 0; kb < C::kKBlocks; ++kb)   // columns past D (last block of D = 96, 160) are filled with zeros
                    tma_load_2d(smem_u32(sIn + s * C::kXBytes + kb * kBlockBytes), &tm_x, 64 * kb, (int)row0, bar);
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
            // A limit shortened by the host (kvq_plan_set_wait_limit) is spent here, straight after the set-up barrier, when
            // the builders have only just begun to store: this thread has issued nothing yet and can leave at once.
            bool first_ok = true;
            if (n_my > 0 && prm.first_wait_polls < kWaitPolls)
                first_ok = wait_first_operand(smem_u32(&ctrl->b_first), abort_flag, status, prm.first_wait_polls);
            // Descriptors differ only in their 14-bit start-address field (bytes >> 4): one base per operand, one add per MMA.
            // The issuing thread is a single instruction stream: what it spends per MMA beyond the issue itself is time
            // the tensor core idles.
            const uint64_t b_desc = smem_desc_sw128(smem_u32(sB));
            const uint64_t a_desc = smem_desc_sw128(smem_u32(sIn));
            const uint32_t b_lo = (uint32_t)b_desc, b_hi = (uint32_t)(b_desc >> 32);
            const uint32_t a_lo = (uint32_t)a_desc, a_hi = (uint32_t)(a_desc >> 32);
            uint32_t builds = 0;
            TileCursor cur(tile_begin, tps);
            for (int j = 0; j < n_my && first_ok; ++j, cur.advance(1)) {
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
                const uint32_t d_tmem = tmem_base + (uint32_t)sc * C::kAccStride;
                const uint32_t a_lo_s = a_lo + (uint32_t)s * (C::kXBytes >> 4);
#pragma unroll
                for (int t = 0; t < (C::kStack ? 1 : C::kSplit); ++t) {   // stacked terms: one MMA per K-step computes both
#pragma unroll
                    for (int ks = 0; ks < C::kKSteps; ++ks) {
                        // (bytes >> 4) of K-step ks inside the x tile and inside a split term
                        const uint32_t a_off = (uint32_t)(ks >> 2) * (kBlockBytes >> 4) + (uint32_t)(ks & 3) * 2u;
                        const uint32_t b_off = (uint32_t)t * (C::kBTerm >> 4) + (uint32_t)(ks >> 2) * (C::kBBlock >> 4) + (uint32_t)(ks & 3) * 2u;
                        const uint64_t ad = ((uint64_t)a_hi << 32) | (uint64_t)(a_lo_s + a_off);
                        const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)(b_lo + b_off);
                        if (t > 0 || ks > 0) umma_f16_ss<true>(d_tmem, ad, bd, C::kIdesc);
                        else umma_f16_ss<false>(d_tmem, ad, bd, C::kIdesc);
                    }
                }
                umma_commit(smem_u32(&ctrl->acc_full[j % kFullBars]));   // to the epilogue; the producer takes it as "x stage free"
            }
        }
    } else {
        // =========================== epilogue: accumulator -> scales, codes, nibbles ===========================
        // Two sets of eight warps take alternate tiles, so that one set's waits (barrier, tensor-memory load)
        // hide behind the other set's arithmetic.  Thread = (row, half row).
        const int set = (warp - 2) >> 3;        // this set takes tiles set, set + 2, ...
        const int q = warp & 3;                 // tensor-memory lane quarter this warp may touch
        const int h = ((warp - 2) >> 2) & 1;    // half of the row
        const int r = q * 32 + lane;            // tile row of this thread
        const int bw = (warp - 2) & 7;          // position within the set: D / 8 rows of B per warp when the set rebuilds B
        const int g0 = h * C::kGroupsPerPart;                                        // this thread's groups: g0 .. g1 - 1
        const int g1 = h == 0 ? C::kGroupsPerPart : G;
        const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        int64_t cached_seg = first_seg;           // B holds this row's table (built above)
        float unlift = 1.0f / first_lift;
        // Group g of this thread's row of accumulator stage sc; with stacked terms the sum of the two terms' columns.
        auto load_group = [&](int sc, int g, uint32_t (&vb)[32]) {
            tmem_ld32(t_addr + (uint32_t)sc * C::kAccStride + (uint32_t)(g * kGroup), vb);
            if constexpr (C::kStack) {
                uint32_t lo[32];
                tmem_ld32(t_addr + (uint32_t)sc * C::kAccStride + (uint32_t)(D + g * kGroup), lo);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) vb[i] = __float_as_uint(__uint_as_float(vb[i]) + __uint_as_float(lo[i]));
            } else {
                tmem_ld_wait();
            }
        };
        float colmax[C::kGroupsPerPart] = {};   // calibration: lane i keeps the running maximum of column i of each of this thread's groups
        TileCursor cur(tile_begin + set, tps);
        for (int j = set; j < n_my; j += 2, cur.advance(2)) {
            __syncwarp();
            const int64_t seg = cur.seg;
            const int64_t off = cur.row_in_segment();

            // ---- a new lambda row.  Every set needs its lift; the set that owns the row's first tile rebuilds B,
            // ---- once every MMA that read the old B is complete (the previous tile's accumulator is full), and
            // ---- tells the mma warp.
            if (seg != cached_seg) {
                const float *lam = CALIB ? nullptr : prm.lambda + (prm.n_lambda == 1 ? 0 : seg) * D;
                const float lift = lift_of<D>(lam, prm.table_max, lane);
                if (j > 0 && cur.first_of_segment()) {
                    if (!wait_or_abort(smem_u32(&ctrl->acc_full[(j - 1) % kFullBars]), (uint32_t)((j - 1) / kFullBars) & 1u,
                                       abort_flag, status, KVQ_DEV_MMA_TIMEOUT))
                        break;
                    build_b_rows<D, BF16, CALIB || WIDE>(sB, prm.e0, lam, lift, bw * (D / 8), (bw + 1) * (D / 8), lane);
                    fence_proxy_async();   // B is read by the tensor core through the async proxy
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctrl->b_ready));
                }
                unlift = 1.0f / lift;
                cached_seg = seg;
            }

            const int sc = j % kAccStages;
            if (!wait_or_abort(smem_u32(&ctrl->acc_full[j % kFullBars]), (uint32_t)(j / kFullBars) & 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT)) break;
            tc_fence_after();

            // ---- rows of the tile that exist: the segment (and with it the tensor) may end inside the tile
            int64_t seg_rows = N - seg * rpl;
            if (seg_rows > rpl) seg_rows = rpl;
            const bool live = off + r < seg_rows;
            const int64_t orow = prm.out_map(seg * rpl + off + r);
            const float Q = prm.bits == 4 ? 7.0f : 127.0f;   // largest code (warp-uniform)
            // ---- one scale per vector: the row's maximum first (this thread's half, then the other half's through
            // ---- shared memory), then a second pass over the accumulator for the codes
            float row_rs = 0.0f;
            bool row_clamp = false;
            if constexpr (PERVEC) {
                float m = 0.0f;
#pragma unroll
                for (int gi = 0; gi < C::kGroupsPerPart; ++gi) {
                    const int g = g0 + gi;
                    if (g < g1) {
                        uint32_t vb[32];
                        load_group(sc, g, vb);
#pragma unroll
                        for (int i = 0; i < 32; ++i) m = fmaxf(m, fabsf(__uint_as_float(vb[i])));
                    }
                }
                const int it = (j - set) >> 1;   // this set's tile count: parity of the pair barrier and of the buffer
                ctrl->rowmax[it & 1][set][h][r] = m;
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->pair[set][q]));
                if (!wait_or_abort(smem_u32(&ctrl->pair[set][q]), (uint32_t)it & 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                m = fmaxf(m, ctrl->rowmax[it & 1][set][h ^ 1][r]);
                const float amax = m * unlift;
                const float sig = fminf(__fdiv_rn(amax, Q), 65504.0f);
                const __half hs = __float2half_rn(sig);
                const float sg = __half2float(hs);
                const float rs1 = sg > 0.0f ? __frcp_rn(sg) : 0.0f;
                row_clamp = !(amax * rs1 < Q + 0.25f);
                row_rs = rs1 * unlift;
                if (live && h == 0) prm.scales[orow] = __half_as_ushort(hs);
            }
#pragma unroll
            for (int gi = 0; gi < C::kGroupsPerPart; ++gi) {
                const int g = g0 + gi;       // warp-uniform
                if (g < g1) {
                    uint32_t vb[32];
                    load_group(sc, g, vb);
                    if (g == g1 - 1) {   // this thread's last group is in registers: hand the accumulator back
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&ctrl->acc_empty[sc]));
                    }
                    if constexpr (CALIB) {
                        // column maxima over the warp's 32 rows (rows past the end were filled with zeros by the TMA load)
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const uint32_t m = __reduce_max_sync(0xFFFFFFFFu, vb[i] & 0x7FFFFFFFu);   // |v| orders like its bits
                            if (lane == i) colmax[gi] = fmaxf(colmax[gi], __uint_as_float(m));
                        }
                        continue;
                    }
                    // ---- scale: sigma = fp16(absmax / 7); codes are taken against the stored value
                    float rs = row_rs;
                    bool clamp = row_clamp;
                    __half hs = __float2half_rn(0.0f);
                    if constexpr (!PERVEC) {
                        float amax = 0.0f;
#pragma unroll
                        for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(__uint_as_float(vb[i])));
                        amax *= unlift;
                        const float sig = fminf(__fdiv_rn(amax, Q), 65504.0f);
                        hs = __float2half_rn(sig);
                        const float sg = __half2float(hs);
                        const float rs1 = sg > 0.0f ? __frcp_rn(sg) : 0.0f;
                        clamp = !(amax * rs1 < Q + 0.25f);   // saturated or subnormal scale: codes could leave [-Q, Q]
                        rs = rs1 * unlift;               // applies to the lifted accumulator values
                    }

                    // ---- round, bias to unsigned codes, pack: 8 nibbles or 4 bytes per word
                    if (prm.bits == 4) {
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
                        if (live) *reinterpret_cast<uint4 *>(prm.packed + orow * (D / 2) + g * 16) = make_uint4(words[0], words[1], words[2], words[3]);
                    } else {
                        uint32_t words[8];
#pragma unroll
                        for (int w = 0; w < 8; ++w) {
                            uint32_t acc = 0;
                            if (!clamp) {
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    acc += __float_as_uint(fmaf(__uint_as_float(vb[4 * w + e]), rs, kMagicRound8)) << (8 * e);
                            } else {
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    acc += __float_as_uint(fminf(fmaxf(__uint_as_float(vb[4 * w + e]) * rs, -127.0f), 127.0f) + kMagicRound8) << (8 * e);
                            }
                            words[w] = (acc - kMagicSum8) ^ 0x80808080u;
                        }
                        if (live) {
                            uint4 *dst = reinterpret_cast<uint4 *>(prm.packed + orow * D + g * 32);
                            dst[0] = make_uint4(words[0], words[1], words[2], words[3]);
                            dst[1] = make_uint4(words[4], words[5], words[6], words[7]);
                        }
                    }
                    if (live) {
                        if constexpr (!PERVEC) prm.scales[orow * G + g] = __half_as_ushort(hs);
                    }
                }
            }
        }
        if constexpr (CALIB) {   // this warp's maxima of its 32 rows of every tile -> the global column maxima
#pragma unroll
            for (int gi = 0; gi < C::kGroupsPerPart; ++gi)
                if (g0 + gi < g1) atomicMax(prm.amax_bits + (g0 + gi) * kGroup + lane, __float_as_uint(colmax[gi] * unlift));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        if (*abort_flag) {
            // Every role has left its loop.  The x tiles whose loads are still in flight were this thread's to issue: give
            // each a bounded chance to land (nobody else may have waited for them), then let tensor-core work that was
            // already issued drain, before the shared and tensor memory go back.
            if (lane == 0)
                for (int j = issued > kInStages ? issued - kInStages : 0; j < issued; ++j)
                    (void)mbar_wait_bounded(smem_u32(&ctrl->in_full[j % kInStages]), (uint32_t)(j / kInStages) & 1u, 1u << 16);
            __nanosleep(20000);
            __syncwarp();
        }
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
namespace {

template <int D, bool BF16, bool CALIB = false, bool PERVEC = false, bool WIDE = false>
cudaError_t launch(int64_t N, const FftParams &f, const float *e0, cudaStream_t stream, uint32_t *amax_bits = nullptr)
{
    using C = Cfg<D, BF16, CALIB || WIDE>;
    static DeviceSlots slots;
    int dev = 0;
    cudaError_t e = current_device_slot(&dev);
    if (e != cudaSuccess) return e;
    int &sms = slots.sms[dev];
    if (sms == 0) {
        int n = 0;
        if ((e = cudaFuncSetAttribute(kvq_encode_umma_kernel<D, BF16, CALIB, PERVEC, WIDE>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        sms = n;
    }
    if (N == 0) return cudaSuccess;   // kvq_plan_prepare: the launch attributes are set, there is nothing to run
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
    prm.out_map = f.out_map;
    prm.table_max = f.table_max;
    prm.bits = f.bits;
    prm.status = f.status;
    prm.amax_bits = amax_bits;
    prm.first_wait_polls = f.first_wait_polls ? f.first_wait_polls : kWaitPolls;

    CUtensorMap tm_x;
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)N};
    const cuuint64_t strides[1] = {(cuuint64_t)(2 * D)};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    if (!make_tensor_map(&tm_x, BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, f.in, dims, strides, box,
                         CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;

    const int64_t tiles = prm.n_seg * ((prm.rpl + kTile - 1) / kTile);
    const int grid = (int)(tiles < sms ? tiles : sms);
    kvq_encode_umma_kernel<D, BF16, CALIB, PERVEC, WIDE><<<grid, kThreads, C::kSmemBytes, stream>>>(prm, tm_x);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

// D = 160 with bf16 input: two bf16 terms of W (120 KB) leave room for two x tiles in flight; the three-term forms
// (calibration, byte codes) do not fit.
bool umma_encode_supported(int D, bool bf16)
{
    (void)bf16;
    return D == 64 || D == 96 || D == 128 || D == 160 || D == 256;
}
bool umma_calibrate_supported(int D, bool bf16) { return umma_encode_supported(D, bf16) && !(D == 160 && bf16); }

// one scale per vector: the row maximum is traded inside a CTA, or across the cluster pair of the D = 256 kernel
bool umma_encode_per_vector_supported(int D, bool bf16) { return umma_encode_supported(D, bf16); }

// byte codes: the code step is 18 times finer than with 4 bits: two bf16 terms of W would leave 2e-4 of the codes on the
// wrong side of a rounding, so bf16 input takes the three-term instantiation (D <= 128: at D = 160 and 256 three terms leave
// no room for x); fp16 input keeps its two terms at every D
bool umma_encode_bits8_supported(int D, bool bf16) { return !(D == 256 && bf16) && !(D == 160 && bf16) && umma_encode_supported(D, bf16); }

cudaError_t umma_encode(int D, bool bf16, bool per_vector, int64_t N, const FftParams &f, const float *e0, cudaStream_t stream)
{
    if (!tensor_map_encode_fn()) return cudaErrorNotSupported;
    if (D == 256) return umma_encode_d256(bf16, per_vector, N, f, e0, stream);   // its own kernel: CTA pairs, x through a ring of K blocks
    if (bf16 && f.bits == 8) {   // three bf16 terms
        switch (D) {
            case 64: return per_vector ? launch<64, true, false, true, true>(N, f, e0, stream) : launch<64, true, false, false, true>(N, f, e0, stream);
            case 96: return per_vector ? launch<96, true, false, true, true>(N, f, e0, stream) : launch<96, true, false, false, true>(N, f, e0, stream);
            case 128: return per_vector ? launch<128, true, false, true, true>(N, f, e0, stream) : launch<128, true, false, false, true>(N, f, e0, stream);
        }
        return cudaErrorInvalidValue;
    }
    if (per_vector) {
        switch (D) {
            case 64: return bf16 ? launch<64, true, false, true>(N, f, e0, stream) : launch<64, false, false, true>(N, f, e0, stream);
            case 96: return bf16 ? launch<96, true, false, true>(N, f, e0, stream) : launch<96, false, false, true>(N, f, e0, stream);
            case 128: return bf16 ? launch<128, true, false, true>(N, f, e0, stream) : launch<128, false, false, true>(N, f, e0, stream);
            case 160: return bf16 ? launch<160, true, false, true>(N, f, e0, stream) : launch<160, false, false, true>(N, f, e0, stream);
        }
        return cudaErrorInvalidValue;
    }
    switch (D) {
        case 64: return bf16 ? launch<64, true>(N, f, e0, stream) : launch<64, false>(N, f, e0, stream);
        case 96: return bf16 ? launch<96, true>(N, f, e0, stream) : launch<96, false>(N, f, e0, stream);
        case 128: return bf16 ? launch<128, true>(N, f, e0, stream) : launch<128, false>(N, f, e0, stream);
        case 160: return bf16 ? launch<160, true>(N, f, e0, stream) : launch<160, false>(N, f, e0, stream);
    }
    return cudaErrorInvalidValue;
}

// Column maxima of |M (s (.) x)| over the N rows of x, accumulated into amax_bits [D] (fp32 bit patterns, zeroed by the
// caller on the same stream): the forward GEMM with lambda = 1 and a reducing epilogue.
cudaError_t umma_calibrate(int D, bool bf16, int64_t N, const FftParams &f, const float *e0, uint32_t *amax_bits, cudaStream_t stream)
{
    if (!tensor_map_encode_fn()) return cudaErrorNotSupported;
    if (D == 256) return umma_calibrate_d256(bf16, N, f, e0, amax_bits, stream);
    switch (D) {
        case 64: return bf16 ? launch<64, true, true>(N, f, e0, stream, amax_bits) : launch<64, false, true>(N, f, e0, stream, amax_bits);
        case 96: return bf16 ? launch<96, true, true>(N, f, e0, stream, amax_bits) : launch<96, false, true>(N, f, e0, stream, amax_bits);
        case 128: return bf16 ? launch<128, true, true>(N, f, e0, stream, amax_bits) : launch<128, false, true>(N, f, e0, stream, amax_bits);
        case 160: return bf16 ? cudaErrorInvalidValue : launch<160, false, true>(N, f, e0, stream, amax_bits);
    }
    return cudaErrorInvalidValue;
}

}  // namespace kvq

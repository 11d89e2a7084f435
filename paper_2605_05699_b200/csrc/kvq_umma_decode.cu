// Warp-specialised tcgen05 DFT-as-GEMM decode kernel of libkvq (sm_100a): D = 64, 96, 128, 160, fp16 or bf16 output.
//
// The inverse path x^ = diag(s) M^T diag(1 / max(lambda, 1e-6)) (q (.) sigma) (Sec. 3.1: the packing of
// Eq. 2 undone, inverse real DFT, signs last; Sec. 5.1 item 1) is a dense D x D contraction per vector, for any even D (the mixed-radix
// head dims need no special case here).  A tile of 128 vectors is one 128 x D x D GEMM on the
// 5th-generation tensor core, a fraction of the time the tile's bytes need to cross HBM, so the kernel's
// job is to keep HBM busy: one persistent CTA per SM runs four roles that hand tiles to one another
// through mbarriers and never wait for one another's latency.
//
//   warp 0        producer   one TMA tensor load per tile: 128 packed rows into a ring of shared-memory
//                            stages, swizzled (or at a pitch) such that row-per-thread reads are free
//                            of bank conflicts
//   warps 2-9     dequant    two groups of four warps that take alternate tiles.  Thread t of a group
//                            owns row t: nibbles -> fp16 codes -> times sigma * rho, two codes per
//                            half2 instruction, stored straight into TENSOR MEMORY as the A operand
//                            (tcgen05.st); the group scales come by plain loads, one tile ahead.
//                            The group that meets the first tile of a new lambda row rebuilds B.
//   warp 1        mma        one thread issues D / 16 K-steps of tcgen05.mma (A from tensor memory, B
//                            from shared memory) into one of two accumulator stages and commits
//   warps 10-17   epilogue   two groups of four warps, alternate tiles.  Thread t reads accumulator
//                            row t (tcgen05.ld), rounds to fp16, writes a swizzled staging tile; one
//                            lane per warp issues the TMA tensor stores (32 rows x 128 B boxes, plus a
//                            64-byte one when D / 32 is odd).  The output tensor maps are
//                            three-dimensional (column, row within lambda segment, segment), so the
//                            hardware clips a tile that ends with its segment or with the tensor: no
//                            per-row tail code.
//
//   A [128 vectors, K = D]   fp16 in tensor memory: lane = vector, D / 2 columns of two codes each
//   B [N = D outputs, K]     fp16 in shared memory, K-major, 128-byte swizzle, K blocks of 64:
//                            W'[n, c] = s_n M[c, n] / max(lambda_c, 1e-6) / rho, rho a power of two
//   D [128, D]               fp32 accumulator in tensor memory, two stages
//
// The K order inside a word of 8 codes is (0,4,1,5,2,6,3,7): that is how the half2 nibble trick
// delivers them, and B is built in the same order, so no instruction is spent on reordering.
//
// Precision: A and B are each rounded once to fp16, accumulation is fp32: about 3e-4 relative L2 per
// vector before the output rounding.  Every wait on an mbarrier is bounded: on a time-out the role
// records the reason in the status word, raises the CTA's abort flag and leaves its loop; the CTA
// then frees its tensor memory and returns.
#include "kvq_decode_fp32.cuh"
#include "kvq_internal.h"
#include "kvq_umma.cuh"

namespace kvq {

namespace {

constexpr int kTile = 128;       // vectors per tile = MMA M
constexpr int kThreads = 576;    // producer, mma, 2 x 4 dequant, 2 x 4 epilogue warps
constexpr int kMaxInStages = 6;  // packed tiles in flight, at most
constexpr int kAccStages = 2;    // accumulators in tensor memory
constexpr int kCtrlBytes = 4608;   // barriers and flags, then eight tiles' worth of per-row output scales
constexpr int kRowScaleSlots = 8;  // a dequant group is never more than seven tiles ahead of the epilogue that reads its slot
constexpr uint32_t kTmemCols = 512;

// BF16OUT: bfloat16 output rounds 8x coarser than fp16, and a result that is off by 1e-4 of the vector's rms already
// lands on the other side of enough rounding boundaries to miss the 1e-3 tolerance.  Both operands are then carried
// in two fp16 terms: a = q sigma rho has 15 significant bits and splits exactly into a_hi + a_lo (one half2 FMA),
// W' = W_hi + W_lo, and x^ = a_hi W_hi + a_lo W_hi + a_hi W_lo accumulates in fp32 (a_lo W_lo is below 1e-7).
// BITS: 4 (nibble pairs) or 8 (one two's-complement byte per code; scale = absmax / 127).  The byte path dequantises
// pairs of neighbouring codes, so its K order is the natural one and the B operand is built to match.
// R2: one radix-2 step of the transform is taken out of the GEMM (plans without a rotation; D = 128, 4-bit codes, either
// output type).  Rows of M are cos / sin(2 pi k n / D), so n -> n + D / 2 multiplies a row by (-1)^k, and in the packing of Eq. 2
// the parity of k is the parity of the channel c.  With E_n / O_n the sums over the even / odd channels (n < D / 2),
//     x^_n = s_n (E_n + O_n),        x^_{n + D/2} = s_{n + D/2} (E_n - O_n):
// two 128 x 64 x 64 GEMMs per tile instead of one 128 x 128 x 128, half the tensor work, and an add, a subtract and half a
// sign flip per output in the epilogue.  The kernel runs at the board's power limit, where tensor flops are what is left to
// save: 147 -> 134 us per 2M-vector launch back to back (bf16 output: 215 -> 192 us).  The half2 nibble trick yields pairs
// (c, c + 4) of equal parity, so routing codes to the two A operands is free.
template <int D, bool BF16OUT, int BITS = 4, bool R2 = false>
struct Cfg {
    static_assert(D % 32 == 0 && D >= 64 && D <= 160, "head dim not built");
    static_assert(!R2 || (D == 128 && BITS == 4), "radix-2 form: D = 128, 4-bit codes");
    static_assert(!BF16OUT || BITS == 4 || D <= 128, "two-term operands with byte codes: shared memory holds them for D <= 128 only");
    static_assert(BITS == 4 || BITS == 8, "code width not built");
    static constexpr int kTerms = BF16OUT ? 2 : 1;         // W_hi (, W_lo); a_hi (, a_lo)
    static constexpr int G = D / 32;                       // groups = 16-byte chunks of a packed row = 32-column accumulator chunks
    static constexpr int kKSteps = D / 16;
    static constexpr int kKBlocks = (D + 63) / 64;         // K blocks of 64 elements (the last one may be half used)
    static constexpr int kBBlock = D * 128;                // bytes of one K block: D rows x 128 B
    static constexpr int kBTerm = kKBlocks * kBBlock;
    static constexpr int kBPart = (D / 2) * 128;           // R2: one parity's operand, D / 2 outputs x D / 2 channels
    static constexpr int kBBytes = R2 ? kTerms * 2 * kBPart : kTerms * kBTerm;   // R2: [term][parity]
    static constexpr int kInRow = D * BITS / 8;            // code bytes per row
    static constexpr int kInBytes = kTile * kInRow;        // bytes one TMA load brings
    static constexpr int kInPitch = (kInBytes + 1023) & ~1023;
    // The packed tile is read row per thread, 16 bytes at a time.  Row pitches of 48 and 80 bytes spread eight
    // consecutive rows over all banks by themselves (96 and 160 bytes over half of them); 32, 64 and 128 bytes need
    // the TMA swizzle of that width.
    static constexpr int kInSwizzleBits = kInRow == 32 ? 1 : kInRow == 64 ? 2 : kInRow == 128 ? 3 : 0;
    static constexpr int kOutWarpBytes = 32 * 2 * D;       // staging of one epilogue warp: G / 2 boxes of 4 KB (+ one of 2 KB)
    static constexpr int kOutBytes = 8 * kOutWarpBytes;
    static constexpr int kRoom = (232448 - 1024 - kCtrlBytes - kBBytes - kOutBytes) / kInPitch;
    static constexpr int kInStages = kRoom < kMaxInStages ? kRoom : kMaxInStages;
    static_assert(kInStages >= (D == 160 && BF16OUT ? 2 : 3), "too few packed tiles in flight");
    static constexpr int kSmemBytes = kBBytes + kInStages * kInPitch + kOutBytes + kCtrlBytes + 1024;
    // tensor memory, D <= 128: two accumulators of D columns, then the A stages of D / 2 columns per term (a_lo 64 columns
    // behind a_hi).  D = 160: an accumulator and an A term of 80 columns in each half of the 512 columns; with two-term
    // operands the two halves hold a_hi and a_lo of ONE stage (the tile is tensor-bound: 3 x 10 K-steps per tile).
    static constexpr uint32_t kAccStride = D <= 128 ? 128 : 256;
    static constexpr int kAStages = BF16OUT ? (D <= 128 ? 2 : 1) : D <= 128 ? 4 : 2;
    // The "A full" / "A free" barriers form a ring of at least two, indexed by tile: the two dequant groups take alternate
    // tiles, and a parity wait only tells a phase from its neighbours, so a barrier must not be shared by both groups.
    // Tile j writes A stage j % kAStages once the MMAs of tile j - kAStages have completed (barrier (j - kAStages) % kABars).
    static constexpr int kABars = kAStages < 2 ? 2 : kAStages;
    static constexpr uint32_t kALo = D <= 128 ? 64 : 256;
    __host__ __device__ static constexpr uint32_t acc_col(int s) { return (uint32_t)s * kAccStride; }
    __host__ __device__ static constexpr uint32_t a_col(int s)
    {
        return D <= 128 ? 256u + 64u * (uint32_t)kTerms * (uint32_t)s : 160u + 256u * (uint32_t)s;
    }
    static constexpr uint32_t kIdesc = umma_idesc_m128(R2 ? D / 2 : D, false);
    static constexpr int kBRows = R2 ? D / 2 : D;          // rows of the plan table that B is built from
};

struct Ctrl {
    uint64_t in_full[kMaxInStages], in_empty[kMaxInStages];
    uint64_t a_full[4], a_empty[4];
    uint64_t acc_full[kAccStages], acc_empty[kAccStages];
    uint64_t b_first;
    uint32_t tmem_base;
    volatile uint32_t abort;
    volatile uint32_t any_wide;   // some lambda row of this CTA's tiles is too wide for the fp16 B operand: redone in fp32 at the end
    float row_scale[kRowScaleSlots][kTile];   // what the epilogue multiplies a row by (1 unless its scales left fp16's comfort zone)
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

// Rows [n0, n1) of the B operand, by one warp: a lane reads four table entries b0[n][4 i .. 4 i + 3] (coalesced
// rows), scales them, trades two values with its neighbour so that each lane holds two K-ordered pairs, and
// writes 8 bytes of the swizzled row.
template <int D, bool BF16OUT, int BITS>
__device__ __forceinline__ void build_b_quad(unsigned char *sB, float4 m, const RecipLambda<D> &rl, int n, int p, int lane)
{
    using C = Cfg<D, BF16OUT, BITS>;
    const bool odd = lane & 1;
    const int i = lane + 32 * p;
    const bool live = i < D / 4;
    auto sat = [](float v) { return fminf(fmaxf(v, -65504.0f), 65504.0f); };
    float vx = sat(m.x * rl.r[p].x), vy = sat(m.y * rl.r[p].y), vz = sat(m.z * rl.r[p].z), vw = sat(m.w * rl.r[p].w);
    const int w = i >> 1;   // word of 8 codes = 16-byte chunk w of the K-major row: K block w / 8, chunk w % 8
    unsigned char *dst = sB + (w >> 3) * C::kBBlock + n * 128 + (((w & 7) ^ (n & 7)) << 4) + (odd ? 8 : 0);
#pragma unroll
    for (int t = 0; t < C::kTerms; ++t) {
        uint2 o;
        if constexpr (BITS == 4) {
            // even lane holds codes 8w .. 8w+3, odd lane 8w+4 .. 8w+7; K order of the word is (0,4,1,5,2,6,3,7)
            const float r0 = __shfl_xor_sync(0xFFFFFFFFu, odd ? vx : vz, 1);
            const float r1 = __shfl_xor_sync(0xFFFFFFFFu, odd ? vy : vw, 1);
            o.x = odd ? narrow2<false>(r0, vz) : narrow2<false>(vx, r0);   // odd: (2, 6)   even: (0, 4)
            o.y = odd ? narrow2<false>(r1, vw) : narrow2<false>(vy, r1);   // odd: (3, 7)   even: (1, 5)
        } else {   // byte codes: natural K order, this lane's four channels side by side
            o.x = narrow2<false>(vx, vy);
            o.y = narrow2<false>(vz, vw);
        }
        if (live) *reinterpret_cast<uint2 *>(dst + t * C::kBTerm) = o;
        if (t + 1 < C::kTerms) {   // what the fp16 term left behind (exact in fp32)
            vx -= __half2float(__float2half_rn(vx)), vy -= __half2float(__float2half_rn(vy));
            vz -= __half2float(__float2half_rn(vz)), vw -= __half2float(__float2half_rn(vw));
        }
    }
}

// Radix-2 form, row n < D / 2 of both parities' operands.  The lane's four channels 4 i .. 4 i + 3 alternate in parity;
// per parity p the even lane assembles the pair (8w + p, 8w + p + 4) and the odd lane (8w + p + 2, 8w + p + 6), each from
// one value of its own and one of its neighbour's: the K order in which the dequant threads write the codes of parity p.
template <int D, int TERMS>
__device__ __forceinline__ void build_b_quad_r2(unsigned char *sB, float4 m, const RecipLambda<D> &rl, int n, int lane)
{
    static_assert(D == 128, "one pass of 32 lanes covers the row");
    constexpr int kPart = (D / 2) * 128;
    const bool odd = lane & 1;
    auto sat = [](float v) { return fminf(fmaxf(v, -65504.0f), 65504.0f); };
    const float v[4] = {sat(m.x * rl.r[0].x), sat(m.y * rl.r[0].y), sat(m.z * rl.r[0].z), sat(m.w * rl.r[0].w)};
    const int w = lane >> 1;   // word of 8 codes; its parity-p codes take bytes 8 w .. 8 w + 7 of the parity's K-major row
#pragma unroll
    for (int p = 0; p < 2; ++p) {
        const float got = __shfl_xor_sync(0xFFFFFFFFu, odd ? v[p] : v[p + 2], 1);
        float w0 = odd ? got : v[p], w1 = odd ? v[p + 2] : got;
        unsigned char *dst = sB + p * kPart + n * 128 + ((((w >> 1) ^ (n & 7))) << 4) + ((w & 1) ? 8 : 0) + (odd ? 4 : 0);
#pragma unroll
        for (int t = 0; t < TERMS; ++t) {
            const uint32_t h = narrow2<false>(w0, w1);
            *reinterpret_cast<uint32_t *>(dst + t * (2 * kPart)) = h;
            if (t + 1 < TERMS) {   // what the fp16 term left behind (exact in fp32)
                const float2 a = widen2<false>(h);
                w0 -= a.x, w1 -= a.y;
            }
        }
    }
}

template <int D, bool BF16OUT, int BITS, bool R2>
__device__ __forceinline__ void build_b_rows(unsigned char *sB, const float *__restrict__ b0, const RecipLambda<D> &rl, int n0, int n1,
                                             int lane)
{
#pragma unroll 4
    for (int n = n0; n < n1; ++n) {
#pragma unroll
        for (int p = 0; p < RecipLambda<D>::kPasses; ++p) {
            const int i = lane + 32 * p;
            float4 m = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (i < D / 4) m = __ldg(reinterpret_cast<const float4 *>(b0 + (size_t)n * D) + i);
            if constexpr (R2) build_b_quad_r2<D, Cfg<D, BF16OUT, BITS, R2>::kTerms>(sB, m, rl, n, lane);
            else build_b_quad<D, BF16OUT, BITS>(sB, m, rl, n, p, lane);
        }
    }
}

// The first build of a CTA: its D / 16 table rows per warp are requested at kernel entry, all at once, and turned
// into B rows here, once lambda has arrived too: one round trip to L2 instead of one per batch of rows.
template <int D, bool BF16OUT, int BITS, bool R2>
struct FirstRows {
    static constexpr int kRows = (R2 ? D / 2 : D) / 16, kPasses = RecipLambda<D>::kPasses;
    float4 m[kRows][kPasses];
    __device__ __forceinline__ void load(const float *__restrict__ b0, int n0, int lane)
    {
#pragma unroll
        for (int k = 0; k < kRows; ++k)
#pragma unroll
            for (int p = 0; p < kPasses; ++p) {
                const int i = lane + 32 * p;
                m[k][p] = i < D / 4 ? __ldg(reinterpret_cast<const float4 *>(b0 + (size_t)(n0 + k) * D) + i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            }
    }
    __device__ __forceinline__ void build(unsigned char *sB, const RecipLambda<D> &rl, int n0, int lane) const
    {
#pragma unroll
        for (int k = 0; k < kRows; ++k)
#pragma unroll
            for (int p = 0; p < kPasses; ++p) {
                if constexpr (R2) build_b_quad_r2<D, Cfg<D, BF16OUT, BITS, R2>::kTerms>(sB, m[k][p], rl, n0 + k, lane);
                else build_b_quad<D, BF16OUT, BITS>(sB, m[k][p], rl, n0 + k, p, lane);
            }
    }
};

// The D / 32 fp16 group scales of one row, as packed 16-bit pairs.
template <int G>
__device__ __forceinline__ void load_row_scales(const uint16_t *__restrict__ sp, uint32_t (&sb)[(G + 1) / 2])
{
    if constexpr (G == 8) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(sp));
        sb[0] = v.x, sb[1] = v.y, sb[2] = v.z, sb[3] = v.w;
    } else if constexpr (G == 4) {
        const uint2 v = __ldg(reinterpret_cast<const uint2 *>(sp));
        sb[0] = v.x, sb[1] = v.y;
    } else if constexpr (G == 2) {
        sb[0] = __ldg(reinterpret_cast<const uint32_t *>(sp));
    } else {   // rows of 6 or 10 bytes are only 2-byte aligned
#pragma unroll
        for (int j = 0; j < (G + 1) / 2; ++j) sb[j] = 0;
#pragma unroll
        for (int j = 0; j < G; ++j) sb[j / 2] |= (uint32_t)__ldg(sp + j) << (16 * (j & 1));
    }
}

}  // namespace

struct UmmaDecodeParams {
    GemmParams g;
    int64_t rpl;        // rows per lambda segment (N when there is one lambda row)
    int64_t n_seg;      // segments
    int64_t n_full;     // segments of exactly rpl rows, covered by the main output maps; a shorter last one uses the tail maps
    int64_t phys_rows;  // rows of the packed / scales arrays (N, or the whole cache for a cache view)
    uint32_t flip2[32]; // radix-2 form: sign-bit masks of s_n s_{n + 64} for the output pairs (n, n + 1), n = 0, 2, .. 62
};

struct UmmaDecodeMaps {
    CUtensorMap packed;            // [N, D / 2] bytes, box 128 rows
    CUtensorMap wide, wide_tail;   // output, boxes of 64 columns x 32 rows (128-byte swizzle)
    CUtensorMap slim, slim_tail;   // output, boxes of 32 columns x 32 rows (64-byte swizzle), used when D / 32 is odd
};

template <int D, bool BF16OUT, int BITS, bool R2>
__global__ void __launch_bounds__(kThreads, 1)
    kvq_decode_umma_kernel(const __grid_constant__ UmmaDecodeParams prm, const __grid_constant__ UmmaDecodeMaps maps)
{
    using C = Cfg<D, BF16OUT, BITS, R2>;
    constexpr int G = C::G, kInStages = C::kInStages;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sB = smem;
    unsigned char *sIn = sB + C::kBBytes;
    unsigned char *sOut = sIn + kInStages * C::kInPitch;
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(sOut + C::kOutBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kInStages; ++s) {
            mbar_init(smem_u32(&ctrl->in_full[s]), 1);
            mbar_init(smem_u32(&ctrl->in_empty[s]), 4);
        }
        for (int s = 0; s < C::kABars; ++s) {
            mbar_init(smem_u32(&ctrl->a_full[s]), 4);
            mbar_init(smem_u32(&ctrl->a_empty[s]), 1);
        }
        for (int s = 0; s < kAccStages; ++s) {
            mbar_init(smem_u32(&ctrl->acc_full[s]), 1);
            mbar_init(smem_u32(&ctrl->acc_empty[s]), 4);
        }
        mbar_init(smem_u32(&ctrl->b_first), 16);   // first B: the sixteen dequant and epilogue warps build it
        ctrl->abort = 0u;
        ctrl->any_wide = 0u;
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);

    // ---- tiles: lambda segments of rpl rows, cut into tiles of 128 rows; a contiguous range of tiles
    // ---- per CTA, so that the B operand is rebuilt as rarely as possible
    const int64_t N = prm.g.N, rpl = prm.rpl;
    const TileShare share(prm.n_seg, rpl, blockIdx.x, gridDim.x);
    const int64_t tps = share.tps, tile_begin = share.begin;
    const int n_my = share.n;
    const int64_t seg_first = n_my > 0 ? tile_begin / tps : 0;
    auto lambda_row = [&](int64_t seg) -> const float * { return prm.g.lambda + prm.g.lambda_index(seg) * D; };

    // ---- B for the first tile's lambda row: the sixteen dequant and epilogue warps build D / 16 rows each while the
    // ---- producer's first loads are in flight; the mma warp waits for all of them.  Table rows and lambda are
    // ---- requested before the set-up barrier, so that their latency runs under it.
    // ---- The dequant warps also request the scales of their first tile here and keep rho, so that neither costs a round
    // ---- trip to L2 after the build.
    float rho_first = 1.0f;
    uint32_t sc_first[(G + 1) / 2];
#pragma unroll
    for (int i = 0; i < (G + 1) / 2; ++i) sc_first[i] = 0u;
    if (n_my > 0 && warp >= 2) {
        FirstRows<D, BF16OUT, BITS, R2> rows;
        rows.load(prm.g.b0, (warp - 2) * (C::kBRows / 16), lane);
        if (warp < 10 && ((warp - 2) >> 2) < n_my) {   // dequant group g's first tile is tile_begin + g
            const TileCursor first(tile_begin + ((warp - 2) >> 2), tps);
            const int64_t row = prm.g.phys_row(first.seg, first.row_in_segment(), rpl) + (warp & 3) * 32 + lane;
            const uint16_t *scales = static_cast<const uint16_t *>(prm.g.scales);
            if (row < prm.phys_rows) {
                if (prm.g.per_vector) {
                    const uint32_t s1 = (uint32_t)__ldg(scales + row);
#pragma unroll
                    for (int i = 0; i < (G + 1) / 2; ++i) sc_first[i] = s1 | (s1 << 16);
                } else {
                    load_row_scales<G>(scales + row * G, sc_first);
                }
            }
        }
        const RecipLambda<D> rl(lambda_row(seg_first), lane);
        rho_first = rl.rho;
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        if (rl.wide) ctrl->any_wide = 1u;
        rows.build(sB, rl, (warp - 2) * (C::kBRows / 16), lane);
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
    uint32_t *status = prm.g.status;

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
                const int64_t row0 = prm.g.phys_row(cur.seg, cur.row_in_segment(), rpl);   // rows past the segment are read and never stored
                const uint32_t bar = smem_u32(&ctrl->in_full[s]);
                mbar_arrive_expect_tx(bar, C::kInBytes);
                tma_load_2d(smem_u32(sIn + s * C::kInPitch), &maps.packed, 0, (int)row0, bar);
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
            for (int j = 0; j < n_mma; ++j) {
                const int sa = j % C::kAStages, sb = j % C::kABars, sc = j % kAccStages;
                if (!wait_or_abort(smem_u32(&ctrl->a_full[sb]), (uint32_t)(j / C::kABars) & 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                if (!wait_or_abort(smem_u32(&ctrl->acc_empty[sc]), ((uint32_t)(j / kAccStages) & 1u) ^ 1u, abort_flag, status,
                                   KVQ_DEV_SLOT_TIMEOUT))
                    break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + C::acc_col(sc);
                const uint32_t a_tmem = tmem_base + C::a_col(sa);
                if constexpr (R2) {   // E = A_even B_even into the first D / 2 accumulator columns, O = A_odd B_odd into the rest
#pragma unroll
                    for (int p = 0; p < 2; ++p) {
#pragma unroll
                        for (int set = 0; set < (BF16OUT ? 3 : 1); ++set) {   // bf16 output: a_hi W_hi + a_lo W_hi + a_hi W_lo
#pragma unroll
                            for (int ks = 0; ks < D / 32; ++ks) {
                                const uint32_t b_set = b_lo + (set == 2 ? (uint32_t)((2 * C::kBPart) >> 4) : 0u) + (uint32_t)p * (C::kBPart >> 4);
                                const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)(b_set + (uint32_t)ks * 2u);
                                const uint32_t dp = d_tmem + (uint32_t)p * (D / 2);
                                const uint32_t ap = a_tmem + (set == 1 ? C::kALo : 0u) + (uint32_t)p * (D / 4) + (uint32_t)ks * 8u;
                                if (set > 0 || ks > 0) umma_f16_ts<true>(dp, ap, bd, C::kIdesc);
                                else umma_f16_ts<false>(dp, ap, bd, C::kIdesc);
                            }
                        }
                    }
                }
                // bf16 output: a_hi W_hi + a_lo W_hi + a_hi W_lo
#pragma unroll
                for (int set = 0; set < (R2 ? 0 : BF16OUT ? 3 : 1); ++set) {
                    const uint32_t a_set = a_tmem + (set == 1 ? C::kALo : 0u);
                    const uint32_t b_set = b_lo + (set == 2 ? (uint32_t)(C::kBTerm >> 4) : 0u);
#pragma unroll
                    for (int ks = 0; ks < C::kKSteps; ++ks) {
                        const uint32_t koff = (uint32_t)(ks >> 2) * (C::kBBlock >> 4) + (uint32_t)(ks & 3) * 2u;   // (bytes >> 4) of K-step ks
                        const uint64_t bd = ((uint64_t)b_hi << 32) | (uint64_t)(b_set + koff);
                        if (set > 0 || ks > 0) umma_f16_ts<true>(d_tmem, a_set + (uint32_t)ks * 8u, bd, C::kIdesc);
                        else umma_f16_ts<false>(d_tmem, a_set, bd, C::kIdesc);
                    }
                }
                umma_commit(smem_u32(&ctrl->acc_full[sc]));
                umma_commit(smem_u32(&ctrl->a_empty[sb]));
            }
        }
    } else if (warp < 10) {
        // =========================== dequant: packed codes -> A in tensor memory ===========================
        const int grp = (warp - 2) >> 2;        // this group takes tiles grp, grp + 2, ...
        const int q = warp & 3;                 // tensor-memory lane quarter this warp may touch
        const int r = q * 32 + lane;            // tile row and tensor-memory lane of this thread
        const uint16_t *scales = static_cast<const uint16_t *>(prm.g.scales);   // D / 32 fp16 scales per row
        const uint32_t swz = C::kInSwizzleBits == 3   ? (uint32_t)(r & 7)
                             : C::kInSwizzleBits == 2 ? (uint32_t)((r >> 1) & 3)
                             : C::kInSwizzleBits == 1 ? (uint32_t)((r >> 2) & 1)
                                                      : 0u;
        int64_t cached_seg = n_my > 0 ? seg_first : -1;   // B holds this row's table (built above)
        float rho = rho_first;

        TileCursor cur(tile_begin + grp, tps), ahead(tile_begin + grp, tps);   // this tile; the tile whose scales are fetched
        uint32_t sc_next[(G + 1) / 2];
        auto fetch_scales = [&](int j) {
#pragma unroll
            for (int i = 0; i < (G + 1) / 2; ++i) sc_next[i] = 0u;
            if (j < n_my) {
                const int64_t row = prm.g.phys_row(ahead.seg, ahead.row_in_segment(), rpl) + r;
                if (row < prm.phys_rows) {
                    if (prm.g.per_vector) {   // one scale per vector: the same value in every group's slot
                        const uint32_t s1 = (uint32_t)__ldg(scales + row);
#pragma unroll
                        for (int i = 0; i < (G + 1) / 2; ++i) sc_next[i] = s1 | (s1 << 16);
                    } else {
                        load_row_scales<G>(scales + row * G, sc_next);
                    }
                }
            }
        };

#pragma unroll
        for (int i = 0; i < (G + 1) / 2; ++i) sc_next[i] = sc_first[i];   // requested before the first B build
        for (int j = grp; j < n_my; j += 2, cur.advance(2)) {
            uint32_t sc[(G + 1) / 2];
#pragma unroll
            for (int i = 0; i < (G + 1) / 2; ++i) sc[i] = sc_next[i];
            ahead.advance(2);
            fetch_scales(j + 2);
            const int64_t seg = cur.seg;

            // ---- a new lambda row: this group needs its rho; the group that meets the row's first tile rebuilds B
            if (seg != cached_seg) {
                const RecipLambda<D> rl(lambda_row(seg), lane);
                rho = rl.rho;
                if (rl.wide) ctrl->any_wide = 1u;
                if (cur.first_of_segment()) {
                    // Every MMA issued so far has read B: the commit of the previous tile (the other group's) covers them
                    // all.  A parity wait can only tell a phase from its neighbours, and the other group may lag by more
                    // than one of its tiles, so first wait for this group's own last tile (its barrier is at most one
                    // phase behind, this group waited on it before writing that tile): MMAs complete in order, so after it
                    // the previous tile's barrier is at most one phase behind too.
                    if (j >= 2 && !wait_or_abort(smem_u32(&ctrl->a_empty[(j - 2) % C::kABars]), (uint32_t)((j - 2) / C::kABars) & 1u,
                                                 abort_flag, status, KVQ_DEV_MMA_TIMEOUT))
                        break;
                    if (!wait_or_abort(smem_u32(&ctrl->a_empty[(j - 1) % C::kABars]), (uint32_t)((j - 1) / C::kABars) & 1u, abort_flag,
                                       status, KVQ_DEV_MMA_TIMEOUT))
                        break;
                    build_b_rows<D, BF16OUT, BITS, R2>(sB, prm.g.b0, rl, q * (C::kBRows / 4), (q + 1) * (C::kBRows / 4), lane);
                    fence_proxy_async();   // B is read by the tensor core through the async proxy
                }
                cached_seg = seg;
            }

            // ---- this tile's packed rows have landed; the A stage is free again
            const int s = j % kInStages, sa = j % C::kAStages, sb = j % C::kABars;
            if (!wait_or_abort(smem_u32(&ctrl->in_full[s]), (uint32_t)(j / kInStages) & 1u, abort_flag, status, KVQ_DEV_LOAD_TIMEOUT)) break;
            const unsigned char *row = sIn + s * C::kInPitch + r * C::kInRow;
            uint4 pk[BITS == 4 ? G : 1];
            if constexpr (BITS == 4) {
#pragma unroll
                for (int c = 0; c < G; ++c) pk[c] = *reinterpret_cast<const uint4 *>(row + (((uint32_t)c ^ swz) << 4));
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->in_empty[s]));   // the values are in registers
            }
            if (j >= C::kAStages) {   // the MMAs that read this A stage last
                const int jp = j - C::kAStages;
                if (!wait_or_abort(smem_u32(&ctrl->a_empty[jp % C::kABars]), (uint32_t)(jp / C::kABars) & 1u, abort_flag, status,
                                   KVQ_DEV_MMA_TIMEOUT))
                    break;
            }
            tc_fence_after();

            // ---- the A operand q sigma rho is fp16.  A row whose scales would take it out of fp16's normal range (a very
            // ---- small or very large vector) is carried times a power of two instead, which the epilogue takes out again
            // ---- in fp32; every other row has the factor 1 and costs the epilogue nothing.
            float inv;
            const float pw = operand_rescue<G>(sc, rho, BITS == 4 ? 9000.0f : 500.0f, inv);   // 7 (127) times this stays inside fp16
            ctrl->row_scale[j & (kRowScaleSlots - 1)][r] = inv;
            // ---- nibbles -> fp16 codes -> times sigma * rho, two codes per instruction
            const uint32_t a_row = tmem_base + ((uint32_t)(q * 32) << 16) + C::a_col(sa);
            const __half2 h1032 = __float2half2_rn(1032.0f);
#pragma unroll
            for (int c = 0; c < G; ++c) {   // chunk c = group c: 32 codes, 16 tensor-memory columns
                const float sig = __half2float(__ushort_as_half((unsigned short)((sc[c >> 1] >> (16 * (c & 1))) & 0xFFFFu)));
                const __half2 s2 = __float2half2_rn(sig * rho * pw);
                uint32_t a[16], al[BF16OUT ? 16 : 1];
                auto put = [&](int k, __half2 q2) {   // K-pair k of the group: one rounding, and what it left behind
                    const __half2 h = __hmul2(q2, s2);
                    a[k] = *reinterpret_cast<const uint32_t *>(&h);
                    if constexpr (BF16OUT) {   // q s2 - h, exact in fp16
                        const __half2 l = __hfma2(q2, s2, __hneg2(h));
                        al[k] = *reinterpret_cast<const uint32_t *>(&l);
                    }
                };
                if constexpr (BITS == 4) {
                    const uint32_t words[4] = {pk[c].x, pk[c].y, pk[c].z, pk[c].w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t u = words[i] ^ 0x88888888u;   // nibbles now hold q + 8
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint32_t m = lop3_and_or(u >> (4 * e), 0x000F000Fu, 0x64006400u);   // {1024 + n_e, 1024 + n_{e+4}}
                            // radix-2 form: pairs 0 and 2 of a word are even channels (first half of a[]), 1 and 3 odd (second half)
                            put(R2 ? 8 * (e & 1) + 2 * i + (e >> 1) : 4 * i + e, __hsub2(*reinterpret_cast<const __half2 *>(&m), h1032));   // exact q
                        }
                    }
                } else {   // 32 byte codes: two 16-byte chunks of the row, pairs of neighbours
                    const __half2 h1152 = __float2half2_rn(1152.0f);
#pragma unroll
                    for (int hc = 0; hc < 2; ++hc) {
                        const uint4 pc = *reinterpret_cast<const uint4 *>(row + (((uint32_t)(2 * c + hc) ^ swz) << 4));
                        const uint32_t words[4] = {pc.x, pc.y, pc.z, pc.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint32_t u = words[i] ^ 0x80808080u;                 // bytes now hold q + 128
                            const uint32_t m01 = __byte_perm(u, 0x64646464u, 0x4140);   // {1024 + b0, 1024 + b1} as fp16 bit patterns
                            const uint32_t m23 = __byte_perm(u, 0x64646464u, 0x4342);
                            put(8 * hc + 2 * i, __hsub2(*reinterpret_cast<const __half2 *>(&m01), h1152));       // exact q
                            put(8 * hc + 2 * i + 1, __hsub2(*reinterpret_cast<const __half2 *>(&m23), h1152));
                        }
                    }
                }
                if constexpr (R2) {   // 8 columns of the even operand, 8 of the odd one
                    const uint32_t ae[8] = {a[0], a[1], a[2], a[3], a[4], a[5], a[6], a[7]};
                    const uint32_t ao[8] = {a[8], a[9], a[10], a[11], a[12], a[13], a[14], a[15]};
                    tmem_st8(a_row + 8u * (uint32_t)c, ae);
                    tmem_st8(a_row + (uint32_t)(D / 4) + 8u * (uint32_t)c, ao);
                    if constexpr (BF16OUT) {
                        const uint32_t le[8] = {al[0], al[1], al[2], al[3], al[4], al[5], al[6], al[7]};
                        const uint32_t lo[8] = {al[8], al[9], al[10], al[11], al[12], al[13], al[14], al[15]};
                        tmem_st8(a_row + C::kALo + 8u * (uint32_t)c, le);
                        tmem_st8(a_row + C::kALo + (uint32_t)(D / 4) + 8u * (uint32_t)c, lo);
                    }
                } else {
                    tmem_st16(a_row + 16u * (uint32_t)c, a);
                    if constexpr (BF16OUT) tmem_st16(a_row + C::kALo + 16u * (uint32_t)c, al);
                }
            }
            if constexpr (BITS == 8) {   // the packed rows were read group by group: only now is their stage free
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->in_empty[s]));
            }
            tmem_st_wait();
            tc_fence_before();
            __threadfence_block();   // the row scales, for the epilogue that follows this tile's accumulator
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->a_full[sb]));
        }
    } else {
        // =========================== epilogue: accumulator -> fp16 -> TMA store ===========================
        const int grp = (warp - 10) >> 2;
        const int q = warp & 3;
        unsigned char *stg = sOut + (warp - 10) * C::kOutWarpBytes;   // this warp's staging tile
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        TileCursor cur(tile_begin + grp, tps);
        for (int j = grp; j < n_my; j += 2, cur.advance(2)) {
            const int sc = j % kAccStages;
            if (!wait_or_abort(smem_u32(&ctrl->acc_full[sc]), (uint32_t)(j / kAccStages) & 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT)) break;
            tc_fence_after();
            if (lane == 0) bulk_wait_read_all();   // this warp's previous stores have read the staging tile
            __syncwarp();
            const float row_inv = ctrl->row_scale[j & (kRowScaleSlots - 1)][q * 32 + lane];
            const bool rescale = __any_sync(0xFFFFFFFFu, row_inv != 1.0f);   // rare: a row outside the operand's comfort zone
            if constexpr (R2) {
#pragma unroll
                for (int h = 0; h < 4; ++h) {   // E and O columns 16 h .. 16 h + 15 -> outputs 16 h .. and D / 2 + 16 h ..
                    uint32_t ev[16], ov[16];
                    tmem_ld16(lane_addr + C::acc_col(sc) + (uint32_t)h * 16u, ev);
                    tmem_ld16(lane_addr + C::acc_col(sc) + (uint32_t)(D / 2) + (uint32_t)h * 16u, ov);
                    tmem_ld_wait();
                    if (rescale) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            ev[i] = __float_as_uint(__uint_as_float(ev[i]) * row_inv);
                            ov[i] = __float_as_uint(__uint_as_float(ov[i]) * row_inv);
                        }
                    }
#pragma unroll
                    for (int k = 0; k < 2; ++k) {   // 16-byte chunk: 8 outputs
                        uint32_t lo[4], hi[4];
#pragma unroll
                        for (int p2 = 0; p2 < 4; ++p2) {
                            const int i = 8 * k + 2 * p2;
                            const float e0 = __uint_as_float(ev[i]), e1 = __uint_as_float(ev[i + 1]);
                            const float o0 = __uint_as_float(ov[i]), o1 = __uint_as_float(ov[i + 1]);
                            lo[p2] = narrow2<BF16OUT>(e0 + o0, e1 + o1);                                     // s_n is already in E and O
                            hi[p2] = narrow2<BF16OUT>(e0 - o0, e1 - o1) ^ prm.flip2[8 * h + 4 * k + p2];     // times s_n s_{n + D/2}
                        }
                        const int chunk = 2 * h + k;   // both halves of the row are 64-column boxes: [32 rows][128 B], 128-byte swizzle
                        *reinterpret_cast<uint4 *>(stg + lane * 128 + ((chunk ^ (lane & 7)) << 4)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                        *reinterpret_cast<uint4 *>(stg + 32 * 128 + lane * 128 + ((chunk ^ (lane & 7)) << 4)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    }
                }
            }
#pragma unroll
            for (int cc = 0; cc < (R2 ? 0 : G); ++cc) {   // 32 accumulator columns = 64 bytes of the output row
                uint32_t v[32];
                tmem_ld32(lane_addr + C::acc_col(sc) + (uint32_t)cc * 32u, v);
                tmem_ld_wait();
                if (rescale) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * row_inv);
                }
                constexpr int kWideBoxes = G / 2;
                const bool wide = (cc >> 1) < kWideBoxes;   // inside a 64-column box, or the last 32-column one
                unsigned char *box = stg + (cc >> 1) * (32 * 128);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    uint4 o;
                    o.x = narrow2<BF16OUT>(__uint_as_float(v[8 * k]), __uint_as_float(v[8 * k + 1]));
                    o.y = narrow2<BF16OUT>(__uint_as_float(v[8 * k + 2]), __uint_as_float(v[8 * k + 3]));
                    o.z = narrow2<BF16OUT>(__uint_as_float(v[8 * k + 4]), __uint_as_float(v[8 * k + 5]));
                    o.w = narrow2<BF16OUT>(__uint_as_float(v[8 * k + 6]), __uint_as_float(v[8 * k + 7]));
                    if (wide) {   // [32 rows][128 B], 128-byte swizzle
                        const int chunk = (cc & 1) * 4 + k;
                        *reinterpret_cast<uint4 *>(box + lane * 128 + ((chunk ^ (lane & 7)) << 4)) = o;
                    } else {      // [32 rows][64 B], 64-byte swizzle
                        *reinterpret_cast<uint4 *>(box + lane * 64 + ((k ^ ((lane >> 1) & 3)) << 4)) = o;
                    }
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
                const int segc = tail ? 0 : (int)seg;
                const CUtensorMap *tw = tail ? &maps.wide_tail : &maps.wide;
#pragma unroll
                for (int b = 0; b < G / 2; ++b) tma_store_3d(tw, 64 * b, row_in_seg, segc, smem_u32(stg + b * (32 * 128)));
                if constexpr (G & 1) {
                    const CUtensorMap *ts = tail ? &maps.slim_tail : &maps.slim;
                    tma_store_3d(ts, 64 * (G / 2), row_in_seg, segc, smem_u32(stg + (G / 2) * (32 * 128)));
                }
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
    // ---- tiles of a lambda row too wide for the fp16 B operand: decoded again in fp32, over what the pipeline stored
    if (ctrl->any_wide && !*abort_flag)
        redo_tiles_fp32<D, BF16OUT, BITS, kTile>(prm.g, tile_begin, n_my, tps, rpl, reinterpret_cast<float *>(smem));
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
namespace {

template <int D, bool BF16OUT, int BITS = 4, bool R2 = false>
cudaError_t launch(int64_t N, const GemmParams &g, cudaStream_t stream, const uint32_t *sign_xor = nullptr)
{
    using C = Cfg<D, BF16OUT, BITS, R2>;
    static DeviceSlots slots;
    int dev = 0;
    cudaError_t e = current_device_slot(&dev);
    if (e != cudaSuccess) return e;
    int &sms = slots.sms[dev];
    if (sms == 0) {
        int n = 0;
        if ((e = cudaFuncSetAttribute(kvq_decode_umma_kernel<D, BF16OUT, BITS, R2>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        sms = n;
    }
    if (!tensor_map_encode_fn()) return cudaErrorNotSupported;
    if (N == 0) return cudaSuccess;   // kvq_plan_prepare: the launch attributes are set, there is nothing to run
    if (N >= (int64_t)1 << 31) return cudaErrorInvalidValue;   // tensor-map coordinates are 32-bit

    UmmaDecodeParams prm;
    prm.g = g;
    prm.rpl = g.view.rows ? g.view.rows : g.n_lambda == 1 ? N : g.rows_per_lambda;   // a cache view: one segment per stream
    prm.n_seg = (N + prm.rpl - 1) / prm.rpl;
    prm.n_full = N / prm.rpl;
    prm.phys_rows = g.view.rows ? prm.n_seg * g.view.stride : N;
    if (prm.phys_rows >= (int64_t)1 << 31) return cudaErrorInvalidValue;
    const int64_t seg_stride = g.view.rows ? g.view.stride : prm.rpl;   // rows from one segment's first row to the next's
    unsigned char *out0 = static_cast<unsigned char *>(g.out) + (size_t)(g.view.rows ? g.view.base : 0) * (2 * D);
    for (int m = 0; m < 32; ++m) prm.flip2[m] = R2 && sign_xor ? sign_xor[m] ^ sign_xor[m + D / 4] : 0u;   // words hold two signs each

    UmmaDecodeMaps maps;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)C::kInRow, (cuuint64_t)prm.phys_rows};
        const cuuint64_t strides[1] = {(cuuint64_t)C::kInRow};
        const cuuint32_t box[2] = {(cuuint32_t)C::kInRow, (cuuint32_t)kTile};
        const CUtensorMapSwizzle sw = C::kInSwizzleBits == 3   ? CU_TENSOR_MAP_SWIZZLE_128B
                                      : C::kInSwizzleBits == 2 ? CU_TENSOR_MAP_SWIZZLE_64B
                                      : C::kInSwizzleBits == 1 ? CU_TENSOR_MAP_SWIZZLE_32B
                                                               : CU_TENSOR_MAP_SWIZZLE_NONE;
        if (!make_tensor_map(&maps.packed, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, g.packed, dims, strides, box, sw)) return cudaErrorInvalidValue;
    }
    auto out_map = [&](CUtensorMap *tm, void *base, int64_t rows, int64_t segs, bool wide) -> bool {
        const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)rows, (cuuint64_t)segs};
        const cuuint64_t strides[2] = {(cuuint64_t)(2 * D), (cuuint64_t)(2 * D) * (cuuint64_t)(segs > 1 ? seg_stride : rows)};
        const cuuint32_t box[3] = {wide ? 64u : 32u, 32u, 1u};
        return make_tensor_map(tm, BF16OUT ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base, dims, strides, box,
                               wide ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B);
    };
    const int64_t tail_rows = N - prm.n_full * prm.rpl;
    unsigned char *tail_base = out0 + (size_t)prm.n_full * seg_stride * (2 * D);
    if (prm.n_full > 0 && (!out_map(&maps.wide, out0, prm.rpl, prm.n_full, true) || !out_map(&maps.slim, out0, prm.rpl, prm.n_full, false)))
        return cudaErrorInvalidValue;
    if (tail_rows > 0 && (!out_map(&maps.wide_tail, tail_base, tail_rows, 1, true) || !out_map(&maps.slim_tail, tail_base, tail_rows, 1, false)))
        return cudaErrorInvalidValue;
    if (tail_rows == 0) maps.wide_tail = maps.wide, maps.slim_tail = maps.slim;
    if (prm.n_full == 0) maps.wide = maps.wide_tail, maps.slim = maps.slim_tail;

    const int64_t tiles = prm.n_seg * ((prm.rpl + kTile - 1) / kTile);
    const int grid = (int)(tiles < sms ? tiles : sms);
    kvq_decode_umma_kernel<D, BF16OUT, BITS, R2><<<grid, kThreads, C::kSmemBytes, stream>>>(prm, maps);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool umma_decode_supported(int D, bool bf16)
{
    (void)bf16;
    return D == 256 || D == 64 || D == 96 || D == 128 || D == 160;
}

// byte codes: every kernel but the D = 160 bf16 form (and the dense D = 256 kernel of rotated plans, which the caller excludes)
bool umma_decode_bits8_supported(int D, bool bf16) { return !(D == 160 && bf16) && umma_decode_supported(D, bf16); }

cudaError_t umma_decode(int D, bool bf16, int bits, int64_t N, const GemmParams &g, const uint32_t *sign_xor, cudaStream_t stream,
                        bool radix2)
{
    // the radix-2 form needs the transform's even / odd structure: the caller asks for it on plans without a rotation
    if (radix2 && D == 128 && bits == 4 && sign_xor)
        return bf16 ? launch<128, true, 4, true>(N, g, stream, sign_xor) : launch<128, false, 4, true>(N, g, stream, sign_xor);
    if (D == 256 && sign_xor) return umma_decode_d256(bf16, bits, N, g, sign_xor, stream);   // its own kernel: radix-2 split, split operands for bf16
    if (bits == 8) {
        switch (D) {
            case 64: return bf16 ? launch<64, true, 8>(N, g, stream) : launch<64, false, 8>(N, g, stream);
            case 96: return bf16 ? launch<96, true, 8>(N, g, stream) : launch<96, false, 8>(N, g, stream);
            case 128: return bf16 ? launch<128, true, 8>(N, g, stream) : launch<128, false, 8>(N, g, stream);
            case 160: return bf16 ? cudaErrorInvalidValue : launch<160, false, 8>(N, g, stream);
        }
        return cudaErrorInvalidValue;
    }
    switch (D) {
        case 64: return bf16 ? launch<64, true>(N, g, stream) : launch<64, false>(N, g, stream);
        case 96: return bf16 ? launch<96, true>(N, g, stream) : launch<96, false>(N, g, stream);
        case 128: return bf16 ? launch<128, true>(N, g, stream) : launch<128, false>(N, g, stream);
        case 160: return bf16 ? launch<160, true>(N, g, stream) : launch<160, false>(N, g, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace kvq

// Warp-specialised tcgen05 DFT-as-GEMM encode kernel of libkvq (sm_100a) for D = 256, fp16 or bf16 input.
//
// Same contraction and the same split of W into 16-bit terms as kvq_umma_encode.cu (v = lambda (.) M (s (.) x),
// Sec. 3.1 Eq. 1-2, Sec. 5.1 item 1; W 2^k = W1 + W2, a third term for bf16 in the calibration pass), with the two changes
// that D = 256 forces:
//
//   * the split B operand (2 or 3 x 128 KB) does not fit one CTA's shared memory, so CTAs work in pairs on the
//     same tiles and each computes one half of the channels (four groups): B is [128 channels, K = 256] per
//     term and CTA.  The two CTAs of a pair share nothing and never wait for each other; the x tile is read
//     twice (the second read hits L2).
//   * what shared memory is left holds little more than one x tile next to B, so x moves through a ring
//     of K blocks (64 columns x 128 rows, 16 KB): the mma thread issues the K steps of a block for every term
//     as soon as the block has landed and releases it with a commit of its own.
//
// Roles as in kvq_umma_encode.cu: producer (TMA), one mma thread, two epilogue sets of eight warps on
// alternate tiles (thread = (row, two groups)).  With two terms they are stacked along N as there (one MMA of
// N = 256 per K-step and CTA, two accumulator stages of 256 columns, the epilogue adds the halves); the three-term
// calibration form keeps four stages of 128 columns.  Byte codes (fp16 input) are a run-time switch of the epilogue.
// Every wait is bounded.
#include "kvq_internal.h"
#include "kvq_umma.cuh"

namespace kvq {

namespace {

constexpr int kTile = 128;                 // vectors per tile = MMA M
constexpr int kGroup = 32;
constexpr int kThreads = 576;              // producer, mma, 16 epilogue warps
constexpr int kEpiWarps = 16;
constexpr int kBlockBytes = kTile * 128;   // one K block of the x tile: 128 rows x 128 B
constexpr int kCtrlBytes = 256;
constexpr int kSmemLimit = 232448;         // 227 KB of dynamic shared memory per CTA
constexpr uint32_t kTmemCols = 512;


constexpr int kD = 256;
constexpr int kG = kD / kGroup;            // 8 scales per row
constexpr int kHalfN = 128;                // channels per CTA = MMA N
constexpr int kKBlocks = kD / 64;          // 4 K blocks per tile
constexpr int kBTermBytes = kKBlocks * kHalfN * 128;   // one split term of B: 128 rows x K = 256, 64 KB
constexpr int kMaxRing = 6;

// CALIB: the calibration pass keeps a third bf16 term (it runs once; its result is compared at 1e-6 of the vector norm)
// PERVEC: one scale per vector.  A row's 256 channels sit in two CTAs, so the pair runs as a thread-block cluster and
// the four half-row maxima of a row (two warps in each CTA) meet in both CTAs' shared memory.
template <bool BF16, bool CALIB = false, bool PERVEC = false>
struct Cfg {
    static constexpr int kSplit = (BF16 && CALIB) ? 3 : 2;
    static constexpr int kBBytes = kSplit * kBTermBytes;
    // Two terms: STACKED along N, rows [0, 128) of a K block the first term's, rows [128, 256) the second's, so that one
    // MMA of N = 256 computes x W_hi into accumulator columns [0, 128) and x W_lo into [128, 256); the epilogue adds the
    // two.  An MMA of M 128, N 128, K 16 costs about 120 cycles here, one of N = 256 about 176 (measured, operands in
    // shared memory): the per-instruction overhead is paid once for both terms and x is read once instead of twice.
    static constexpr bool kStack = kSplit == 2;
    static constexpr int kNmma = kStack ? 2 * kHalfN : kHalfN;
    static constexpr int kBBlock = kNmma * 128;                          // one K block of B: kNmma rows x 128 B
    static constexpr int kBTerm = kStack ? kHalfN * 128 : kBTermBytes;   // from one term's row c to the next term's
    static constexpr uint32_t kAccStride = kNmma;                        // tensor-memory columns per accumulator
    static constexpr int kAccStages = 512 / kNmma;                       // 2 (stacked) or 4
    static constexpr int kMaxBytes = PERVEC ? 2 * 2 * 4 * kTile * (int)sizeof(float) : 0;   // [tile parity][set][party][row]
    static constexpr int kRoom = (kSmemLimit - 1024 - kCtrlBytes - kMaxBytes - kBBytes) / kBlockBytes;
    static constexpr int kRing = kRoom < kMaxRing ? kRoom : kMaxRing;   // K blocks of x in flight: 6 (2 next to a three-term B)
    static_assert(kRing >= 2, "no room for the x ring");
    static constexpr int kSmemBytes = kBBytes + kRing * kBlockBytes + kCtrlBytes + kMaxBytes + 1024;
    static constexpr uint32_t kIdesc = umma_idesc_m128(kNmma, BF16);
};

struct Ctrl {
    uint64_t in_full[kMaxRing], in_empty[kMaxRing];
    uint64_t acc_full[4], acc_empty[4];
    uint64_t b_first, b_ready;
    uint64_t quad[2][4];        // one scale per vector: the four warps (two per CTA of the pair) that share 32 rows of a set
    uint32_t tmem_base;
    volatile uint32_t abort;
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

// ---- thread-block cluster of two CTAs: the partner's shared memory and barriers (one scale per vector only)
__device__ __forceinline__ uint32_t cluster_map(uint32_t smem_addr, uint32_t cta_rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(cta_rank));
    return r;
}
__device__ __forceinline__ void cluster_st_f32(uint32_t cluster_addr, float v)
{
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}
__device__ __forceinline__ void cluster_mbar_arrive(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// wait_or_abort with cluster-scope acquire: the values the partner CTA stored before its arrive are visible afterwards
__device__ __forceinline__ bool wait_cluster_or_abort(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t *status,
                                                      uint32_t reason)
{
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if (it > 32) {
            if (*abort_flag) return false;
            __nanosleep(32);
        }
    }
    *abort_flag = 1u;
    atomicOr(status, reason);
    return false;
}

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

// Rows [c0, c1) of every split term of this CTA's half of the B operand (channel 128 half + c), by one warp: a lane
// reads four table entries per pass (coalesced rows), scales them by lambda_c 2^k, peels off 16-bit terms and
// writes 8 bytes of each term's swizzled row.
template <bool BF16, bool CALIB>
__device__ __forceinline__ void build_b_rows(unsigned char *sB, const float *__restrict__ e0, const float *__restrict__ lam, float lift,
                                             int half, int c0, int c1, int lane)
{
    using C = Cfg<BF16, CALIB>;
#pragma unroll 2   // (eight rows in flight were tried: slower, 60.3 against 55.9 us at 212,992 vectors and 52 lambda rows)
    for (int c = c0; c < c1; ++c) {
        const int cg = half * kHalfN + c;
        const float f = lam ? __ldg(lam + cg) * lift : lift;
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            const int i = lane + 32 * p;
            const float4 m = __ldg(reinterpret_cast<const float4 *>(e0 + (size_t)cg * kD) + i);
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
    }
}

}  // namespace

struct UmmaEncode256Params {
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
    uint32_t *status;
    uint32_t *amax_bits;        // calibration only: [D] running column maxima as fp32 bit patterns (start at zero)
    int bits;                   // 4: nibble pairs; 8 (fp16 input): one two's-complement byte per code, scale = absmax / 127
};

template <bool BF16, bool CALIB, bool PERVEC>
__device__ __forceinline__ void encode_d256_body(const UmmaEncode256Params &prm, const CUtensorMap &tm_x)
{
    using C = Cfg<BF16, CALIB, PERVEC>;
    constexpr int kRing = C::kRing;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *sB = smem;                                   // kSplit terms
    unsigned char *sIn = sB + C::kBBytes;                       // ring of K blocks of x
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(sIn + kRing * kBlockBytes);
    float *rowmax = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(ctrl) + kCtrlBytes);   // PERVEC: [parity][set][party][row]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int half = blockIdx.x & 1;            // which 128 channels this CTA computes
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kRing; ++s) {
            mbar_init(smem_u32(&ctrl->in_full[s]), 1);
            mbar_init(smem_u32(&ctrl->in_empty[s]), 1);
        }
        for (int s = 0; s < C::kAccStages; ++s) {
            mbar_init(smem_u32(&ctrl->acc_full[s]), 1);
            mbar_init(smem_u32(&ctrl->acc_empty[s]), kEpiWarps / 2);
        }
        mbar_init(smem_u32(&ctrl->b_first), kEpiWarps);       // first B: all epilogue warps build it
        mbar_init(smem_u32(&ctrl->b_ready), kEpiWarps / 2);   // later rebuilds: the set that owns the tile
        for (int s = 0; s < 2; ++s)
            for (int qq = 0; qq < 4; ++qq) mbar_init(smem_u32(&ctrl->quad[s][qq]), 4);
        ctrl->abort = 0u;
        mbar_init_fence();
    }
    if (warp == 0) tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if constexpr (PERVEC) cluster_sync_all();   // the partner's barriers exist before anyone arrives on them
    const uint32_t tmem_base = ctrl->tmem_base;
    volatile uint32_t *abort_flag = &ctrl->abort;
    uint32_t *status = prm.status;

    // ---- tiles: lambda segments of rpl rows, cut into tiles of 128 rows; a contiguous range per CTA pair
    const int64_t N = prm.N, rpl = prm.rpl;
    const TileShare share(prm.n_seg, rpl, (unsigned)pair, (unsigned)n_pairs);
    const int64_t tps = share.tps, tile_begin = share.begin;
    const int n_my = share.n;

    if (warp == 0) {
        // =========================== producer ===========================
        if (lane == 0) {
            int issued = 0;
            bool ok = true;
            TileCursor cur(tile_begin, tps);
            for (int j = 0; j < n_my && ok; ++j, cur.advance(1)) {
                const int64_t row0 = cur.seg * rpl + cur.row_in_segment();
#pragma unroll
                for (int kb = 0; kb < kKBlocks; ++kb) {
                    const int u = kKBlocks * j + kb, s = u % kRing;
                    ok = wait_or_abort(smem_u32(&ctrl->in_empty[s]), ((uint32_t)(u / kRing) & 1u) ^ 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT);
                    if (!ok) break;
                    const uint32_t bar = smem_u32(&ctrl->in_full[s]);
                    mbar_arrive_expect_tx(bar, kBlockBytes);
                    tma_load_2d(smem_u32(sIn + s * kBlockBytes), &tm_x, 64 * kb, (int)row0, bar);
                    issued = u + 1;
                }
            }
            if (!ok) {
                // give this thread's own copies in flight a bounded chance to land before the CTA goes away
                for (int u = issued > kRing ? issued - kRing : 0; u < issued; ++u)
                    (void)mbar_wait_bounded(smem_u32(&ctrl->in_full[u % kRing]), (uint32_t)(u / kRing) & 1u, 1u << 16);
            }
        }
    } else if (warp == 1) {
        // =========================== mma issuer ===========================
        if (lane == 0) {
            // Descriptors differ only in their 14-bit start-address field (bytes >> 4): one base per operand, one add per MMA.
            const uint64_t b_desc = smem_desc_sw128(smem_u32(sB));
            const uint64_t a_desc = smem_desc_sw128(smem_u32(sIn));
            const uint32_t b_lo = (uint32_t)b_desc, b_hi = (uint32_t)(b_desc >> 32);
            const uint32_t a_lo = (uint32_t)a_desc, a_hi = (uint32_t)(a_desc >> 32);
            uint32_t builds = 0;
            bool ok = true;
            TileCursor cur(tile_begin, tps);
            for (int j = 0; j < n_my && ok; ++j, cur.advance(1)) {
                const int sc = j % C::kAccStages;
                if (j == 0) {   // all epilogue warps build the first B while the first x blocks are in flight
                    if (!wait_or_abort(smem_u32(&ctrl->b_first), 0u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                } else if (cur.first_of_segment()) {   // an epilogue set rebuilds B for this lambda row
                    if (!wait_or_abort(smem_u32(&ctrl->b_ready), builds & 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                    ++builds;
                }
                if (!wait_or_abort(smem_u32(&ctrl->acc_empty[sc]), ((uint32_t)(j / C::kAccStages) & 1u) ^ 1u, abort_flag, status,
                                   KVQ_DEV_SLOT_TIMEOUT))
                    break;
                const uint32_t d_tmem = tmem_base + (uint32_t)sc * C::kAccStride;
#pragma unroll
                for (int kb = 0; kb < kKBlocks; ++kb) {
                    const int u = kKBlocks * j + kb, s = u % kRing;
                    if (!wait_or_abort(smem_u32(&ctrl->in_full[s]), (uint32_t)(u / kRing) & 1u, abort_flag, status, KVQ_DEV_LOAD_TIMEOUT)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_lo_s = a_lo + (uint32_t)s * (kBlockBytes >> 4);
#pragma unroll
                    for (int t = 0; t < (C::kStack ? 1 : C::kSplit); ++t) {   // stacked terms: one MMA per K-step computes both
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {   // the four K steps of this block
                            const uint64_t ad = ((uint64_t)a_hi << 32) | (uint64_t)(a_lo_s + (uint32_t)ks * 2u);
                            const uint64_t bd = ((uint64_t)b_hi << 32) |
                                                (uint64_t)(b_lo + (uint32_t)t * (C::kBTerm >> 4) + (uint32_t)kb * (C::kBBlock >> 4) + (uint32_t)ks * 2u);
                            if (kb > 0 || t > 0 || ks > 0) umma_f16_ss<true>(d_tmem, ad, bd, C::kIdesc);
                            else umma_f16_ss<false>(d_tmem, ad, bd, C::kIdesc);
                        }
                    }
                    umma_commit(smem_u32(&ctrl->in_empty[s]));   // the tensor core has read this block of x
                }
                if (ok) umma_commit(smem_u32(&ctrl->acc_full[sc]));
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
        const int bw = (warp - 2) & 7;          // position within the set: 16 rows of B per warp when the set rebuilds B
        const int g0 = 2 * h;                   // this thread's groups within the CTA's four: g0, g0 + 1
        const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        // Group g (of this CTA's four) of this thread's row of accumulator stage sc; with stacked terms the sum of the two
        // terms' columns.
        auto load_group = [&](int sc, int g, uint32_t (&vb)[32]) {
            tmem_ld32(t_addr + (uint32_t)sc * C::kAccStride + (uint32_t)(g * kGroup), vb);
            if constexpr (C::kStack) {
                uint32_t lo[32];
                tmem_ld32(t_addr + (uint32_t)sc * C::kAccStride + (uint32_t)(kHalfN + g * kGroup), lo);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) vb[i] = __float_as_uint(__uint_as_float(vb[i]) + __uint_as_float(lo[i]));
            } else {
                tmem_ld_wait();
            }
        };
        int64_t cached_seg = -1;
        float unlift = 1.0f;
        if (n_my > 0) {   // B for the CTA's first lambda row: D / 16 rows per warp, all sixteen warps
            TileCursor first(tile_begin, tps);
            const float *lam = CALIB ? nullptr : prm.lambda + (prm.n_lambda == 1 ? 0 : first.seg) * kD;
            const float lift = lift_of<kD>(lam, prm.table_max, lane);
            build_b_rows<BF16, CALIB>(sB, prm.e0, lam, lift, half, (warp - 2) * 8, (warp - 1) * 8, lane);
            fence_proxy_async();   // B is read by the tensor core through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->b_first));
            unlift = 1.0f / lift;
            cached_seg = first.seg;
        }
        float colmax[2] = {};   // calibration: lane i keeps the running maximum of column i of each of this thread's groups
        TileCursor cur(tile_begin + set, tps);
        for (int j = set; j < n_my; j += 2, cur.advance(2)) {
            __syncwarp();
            const int64_t seg = cur.seg;
            const int64_t off = cur.row_in_segment();

            // ---- a new lambda row.  Every set needs its lift; the set that owns the row's first tile rebuilds B,
            // ---- once every MMA that read the old B is complete (the previous tile's accumulator is full), and
            // ---- tells the mma warp.
            if (seg != cached_seg) {
                const float *lam = CALIB ? nullptr : prm.lambda + (prm.n_lambda == 1 ? 0 : seg) * kD;
                const float lift = lift_of<kD>(lam, prm.table_max, lane);
                if (j > 0 && cur.first_of_segment()) {
                    if (!wait_or_abort(smem_u32(&ctrl->acc_full[(j - 1) % C::kAccStages]), (uint32_t)((j - 1) / C::kAccStages) & 1u,
                                       abort_flag, status, KVQ_DEV_MMA_TIMEOUT))
                        break;
                    build_b_rows<BF16, CALIB>(sB, prm.e0, lam, lift, half, bw * 16, (bw + 1) * 16, lane);
                    fence_proxy_async();   // B is read by the tensor core through the async proxy
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctrl->b_ready));
                }
                unlift = 1.0f / lift;
                cached_seg = seg;
            }

            const int sc = j % C::kAccStages;
            if (!wait_or_abort(smem_u32(&ctrl->acc_full[sc]), (uint32_t)(j / C::kAccStages) & 1u, abort_flag, status, KVQ_DEV_MMA_TIMEOUT)) break;
            tc_fence_after();

            // ---- rows of the tile that exist: the segment (and with it the tensor) may end inside the tile
            int64_t seg_rows = N - seg * rpl;
            if (seg_rows > rpl) seg_rows = rpl;
            const bool live = off + r < seg_rows;
            const int64_t orow = prm.out_map(seg * rpl + off + r);
            const float Q = prm.bits == 4 ? 7.0f : 127.0f;   // largest code (warp-uniform)
            // ---- one scale per vector: this thread's maximum over its 64 channels goes to both CTAs of the pair; the four
            // ---- parties of a row (two half-row threads in each CTA) meet on a four-arrival barrier in each CTA, once per
            // ---- tile; buffers alternate with the tile parity, so a party cannot overwrite what another still reads
            float row_rs = 0.0f;
            bool row_clamp = false;
            if constexpr (PERVEC) {
                float m = 0.0f;
#pragma unroll
                for (int gi = 0; gi < 2; ++gi) {
                    uint32_t vb[32];
                    load_group(sc, g0 + gi, vb);
#pragma unroll
                    for (int i = 0; i < 32; ++i) m = fmaxf(m, fabsf(__uint_as_float(vb[i])));
                }
                const int it = (j - set) >> 1;                       // this set's tile count
                float *slot = rowmax + (((it & 1) * 2 + set) * 4) * kTile;   // [party][row] of this buffer
                const int party = 2 * half + h;
                slot[party * kTile + r] = m;
                cluster_st_f32(cluster_map(smem_u32(slot + party * kTile + r), (uint32_t)(half ^ 1)), m);
                asm volatile("fence.acq_rel.cluster;" ::: "memory");   // every lane's stores before lane 0's arrives
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&ctrl->quad[set][q]));
                    cluster_mbar_arrive(cluster_map(smem_u32(&ctrl->quad[set][q]), (uint32_t)(half ^ 1)));
                }
                if (!wait_cluster_or_abort(smem_u32(&ctrl->quad[set][q]), (uint32_t)it & 1u, abort_flag, status, KVQ_DEV_SLOT_TIMEOUT)) break;
                m = fmaxf(fmaxf(slot[r], slot[kTile + r]), fmaxf(slot[2 * kTile + r], slot[3 * kTile + r]));
                const float amax = m * unlift;
                const float sig = fminf(__fdiv_rn(amax, Q), 65504.0f);
                const __half hs = __float2half_rn(sig);
                const float sg = __half2float(hs);
                const float rs1 = sg > 0.0f ? __frcp_rn(sg) : 0.0f;
                row_clamp = !(amax * rs1 < Q + 0.25f);
                row_rs = rs1 * unlift;
                if (live && party == 0) prm.scales[orow] = __half_as_ushort(hs);
            }
#pragma unroll
            for (int gi = 0; gi < 2; ++gi) {
                const int g = g0 + gi;       // warp-uniform; group within this CTA's half
                {
                    uint32_t vb[32];
                    load_group(sc, g, vb);
                    if (gi == 1) {   // this thread's last group is in registers: hand the accumulator back
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

                    const int gg = 4 * half + g;   // group within the row
                    if (prm.bits == 8) {   // ---- round, bias to unsigned bytes, pack 4 codes per word
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
                            uint4 *dst = reinterpret_cast<uint4 *>(prm.packed + orow * kD + gg * 32);
                            dst[0] = make_uint4(words[0], words[1], words[2], words[3]);
                            dst[1] = make_uint4(words[4], words[5], words[6], words[7]);
                            if constexpr (!PERVEC) prm.scales[orow * kG + gg] = __half_as_ushort(hs);
                        }
                        continue;
                    }
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
                    if (live) {
                        *reinterpret_cast<uint4 *>(prm.packed + orow * (kD / 2) + gg * 16) = make_uint4(words[0], words[1], words[2], words[3]);
                        if constexpr (!PERVEC) prm.scales[orow * kG + gg] = __half_as_ushort(hs);
                    }
                }
            }
        }
        if constexpr (CALIB) {   // this warp's maxima of its 32 rows of every tile -> the global column maxima
#pragma unroll
            for (int gi = 0; gi < 2; ++gi)
                atomicMax(prm.amax_bits + (4 * half + g0 + gi) * kGroup + lane, __float_as_uint(colmax[gi] * unlift));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        if (*abort_flag) __nanosleep(20000);   // let tensor-core work that was already issued drain
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if constexpr (PERVEC) cluster_sync_all();   // neither CTA leaves while the other may still store into its shared memory
}

template <bool BF16, bool CALIB>
__global__ void __launch_bounds__(kThreads, 1)
    kvq_encode_umma_d256_kernel(const __grid_constant__ UmmaEncode256Params prm, const __grid_constant__ CUtensorMap tm_x)
{
    encode_d256_body<BF16, CALIB, false>(prm, tm_x);
}

// one scale per vector: the same body with the CTA pair as a cluster (launched with a cluster dimension of 2)
template <bool BF16>
__global__ void __launch_bounds__(kThreads, 1)
    kvq_encode_umma_d256_pv_kernel(const __grid_constant__ UmmaEncode256Params prm, const __grid_constant__ CUtensorMap tm_x)
{
    encode_d256_body<BF16, false, true>(prm, tm_x);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
namespace {

template <bool BF16, bool CALIB = false, bool PERVEC = false>
cudaError_t launch(int64_t N, const FftParams &f, const float *e0, cudaStream_t stream, uint32_t *amax_bits = nullptr)
{
    using C = Cfg<BF16, CALIB, PERVEC>;
    auto kern = [] {
        if constexpr (PERVEC) return kvq_encode_umma_d256_pv_kernel<BF16>;
        else return kvq_encode_umma_d256_kernel<BF16, CALIB>;
    }();
    static DeviceSlots slots;
    int dev = 0;
    cudaError_t e = current_device_slot(&dev);
    if (e != cudaSuccess) return e;
    int &sms = slots.sms[dev];
    if (sms == 0) {
        int n = 0;
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        sms = n;
    }
    // one scale per vector: the pair is a cluster of two CTAs, as many pairs as the device holds at once (SMs of a
    // cluster share a GPC); looked up once per device
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    if constexpr (PERVEC) {
        cfg.gridDim = dim3((unsigned)sms, 1, 1);
        cfg.blockDim = dim3(kThreads, 1, 1);
        cfg.dynamicSmemBytes = C::kSmemBytes;
        cfg.stream = stream;
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int &fit = slots.blocks_per_sm[dev];
        if (fit == 0) {
            int n = 0;
            if ((e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg)) != cudaSuccess) return e;
            if (n < 1) return cudaErrorLaunchOutOfResources;
            fit = n;
        }
    }
    if (N == 0) return cudaSuccess;   // kvq_plan_prepare: the launch attributes are set, there is nothing to run
    if (N >= (int64_t)1 << 31) return cudaErrorInvalidValue;   // tensor-map coordinates are 32-bit

    UmmaEncode256Params prm;
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
    prm.status = f.status;
    prm.amax_bits = amax_bits;
    prm.bits = f.bits;

    CUtensorMap tm_x;
    const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)N};
    const cuuint64_t strides[1] = {(cuuint64_t)(2 * kD)};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    if (!make_tensor_map(&tm_x, BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, f.in, dims, strides, box,
                         CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;

    const int64_t tiles = prm.n_seg * ((prm.rpl + kTile - 1) / kTile);
    int64_t pairs = tiles < sms / 2 ? tiles : sms / 2;
    if constexpr (PERVEC) {
        const int fit = slots.blocks_per_sm[dev];   // clusters resident at once
        if (pairs > fit) pairs = fit;
        cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
        e = cudaLaunchKernelEx(&cfg, kern, prm, tm_x);
        count_launch();
        return e != cudaSuccess ? e : cudaGetLastError();
    }
    kern<<<(int)(2 * pairs), kThreads, C::kSmemBytes, stream>>>(prm, tm_x);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t umma_encode_d256(bool bf16, bool per_vector, int64_t N, const FftParams &f, const float *e0, cudaStream_t stream)
{
    if (!tensor_map_encode_fn()) return cudaErrorNotSupported;
    if (per_vector) return bf16 ? launch<true, false, true>(N, f, e0, stream) : launch<false, false, true>(N, f, e0, stream);
    return bf16 ? launch<true>(N, f, e0, stream) : launch<false>(N, f, e0, stream);
}

cudaError_t umma_calibrate_d256(bool bf16, int64_t N, const FftParams &f, const float *e0, uint32_t *amax_bits, cudaStream_t stream)
{
    if (!tensor_map_encode_fn()) return cudaErrorNotSupported;
    return bf16 ? launch<true, true>(N, f, e0, stream, amax_bits) : launch<false, true>(N, f, e0, stream, amax_bits);
}

}  // namespace kvq
